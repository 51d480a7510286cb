// Quadratic ("flash-style") KATA forward on plain fp32 FMAs.
//
// Definition evaluated tile by tile: for a 64-row query tile loop over key tiles j <= i,
//   s = q_t . k_i,  w = s^2 / ||k_i||^2  (causal mask incl. diagonal),  N += w v_i,  D += w,
// epilogue o = N / D.  The query norm is a common factor of N and D and is left out.  No running
// maximum and no rescaling are needed: the weights are polynomial, not exponential.
// This is the fp32 path (and the fallback for shapes the tensor-core kernel does not cover).
#include "kata_common.cuh"

namespace kata {
namespace {

constexpr int QT = 64;   // query rows per CTA
constexpr int KT = 64;   // key rows per tile
constexpr int NTHR = 128;
constexpr int TS = 68;   // row stride of the transposed q/k tiles in shared memory

template <typename T, int D, int DV>
__global__ void __launch_bounds__(NTHR) quad_simt_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                          const T* __restrict__ v, T* __restrict__ out,
                                                          int Tlen, int order, int groups) {
  extern __shared__ __align__(16) float smem[];
  // transposed tiles, row stride TS (=68 floats: 16-byte aligned rows, few bank conflicts on the fill)
  float (*qT)[TS] = reinterpret_cast<float (*)[TS]>(smem);
  float (*kT)[TS] = reinterpret_cast<float (*)[TS]>(smem + D * TS);
  float (*vs)[DV] = reinterpret_cast<float (*)[DV]>(smem + 2 * D * TS);
  float (*W)[KT + 1] = reinterpret_cast<float (*)[KT + 1]>(smem + 2 * D * TS + KT * DV);
  float* rk2 = smem + 2 * D * TS + KT * DV + QT * (KT + 1);

  const int tid = threadIdx.x;
  const int ty = tid >> 3, tx = tid & 7;
  const int qtile = gridDim.x - 1 - blockIdx.x;   // heaviest tiles first
  const size_t bh = blockIdx.y;
  const T* qh = q + bh * (size_t)Tlen * D;
  const T* kh = k + bh * (size_t)Tlen * D;
  const T* vh = v + bh * (size_t)Tlen * DV;
  T* oh = out + bh * (size_t)Tlen * DV;
  const int q0 = qtile * QT;

  for (int idx = tid; idx < QT * D; idx += NTHR) {
    const int r = idx / D, a = idx % D;
    qT[a][r] = (q0 + r < Tlen) ? to_f32(qh[(size_t)(q0 + r) * D + a]) : 0.f;
  }

  constexpr int NJ = DV / 8;
  float acc[4][NJ];
  float dacc[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    dacc[i] = 0.f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) acc[i][j] = 0.f;
  }

  for (int kt = 0; kt <= qtile; ++kt) {
    const int k0 = kt * KT;
    __syncthreads();   // previous tile fully consumed (also orders the qT fill)
    for (int idx = tid; idx < KT * D; idx += NTHR) {
      const int r = idx / D, a = idx % D;
      kT[a][r] = (k0 + r < Tlen) ? to_f32(kh[(size_t)(k0 + r) * D + a]) : 0.f;
    }
    for (int idx = tid; idx < KT * DV; idx += NTHR) {
      const int r = idx / DV, c = idx % DV;
      vs[r][c] = (k0 + r < Tlen) ? to_f32(vh[(size_t)(k0 + r) * DV + c]) : 0.f;
    }
    __syncthreads();
    if (tid < KT) {
      float s = 0.f;
#pragma unroll 8
      for (int a = 0; a < D; ++a) s = fmaf(kT[a][tid], kT[a][tid], s);
      rk2[tid] = (order == 2) ? inv_or_zero(s) : 1.f;
    }
    // scores: 4 x 8 micro-tile per thread; with g feature blocks the weight is the sum of the squared block dots
    float s[4][8], w2[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) w2[i][j] = 0.f;
    const int mblk = D / groups;
    for (int gb = 0; gb < groups; ++gb) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) s[i][j] = 0.f;
#pragma unroll 4
      for (int a = gb * mblk; a < (gb + 1) * mblk; ++a) {
        const float4 qa = *reinterpret_cast<const float4*>(&qT[a][ty * 4]);
        const float4 k0v = *reinterpret_cast<const float4*>(&kT[a][tx * 8]);
        const float4 k1v = *reinterpret_cast<const float4*>(&kT[a][tx * 8 + 4]);
        const float qq[4] = {qa.x, qa.y, qa.z, qa.w};
        const float kk[8] = {k0v.x, k0v.y, k0v.z, k0v.w, k1v.x, k1v.y, k1v.z, k1v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) s[i][j] = fmaf(qq[i], kk[j], s[i][j]);
      }
      if (groups > 1) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) w2[i][j] = fmaf(s[i][j], s[i][j], w2[i][j]);
      }
    }
    __syncthreads();   // rk2 visible
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int r = ty * 4 + i, c = tx * 8 + j;
        const bool live = (k0 + c <= q0 + r) && (k0 + c < Tlen);
        float w = (order == 2) ? (groups > 1 ? w2[i][j] : s[i][j] * s[i][j]) * rk2[c] : s[i][j];
        W[r][c] = live ? w : 0.f;
      }
    __syncthreads();
#pragma unroll 4
    for (int i2 = 0; i2 < KT; ++i2) {
      float wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) wv[i] = W[ty * 4 + i][i2];
#pragma unroll
      for (int i = 0; i < 4; ++i) dacc[i] += wv[i];
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const float vv = vs[i2][tx + 8 * j];
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(wv[i], vv, acc[i][j]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = q0 + ty * 4 + i;
    if (r >= Tlen) continue;
    const float inv = (order == 2) ? (dacc[i] > 0.f ? 1.f / dacc[i] : 0.f)
                                   : (dacc[i] != 0.f ? 1.f / dacc[i] : 0.f);
#pragma unroll
    for (int j = 0; j < NJ; ++j) oh[(size_t)r * DV + tx + 8 * j] = from_f32<T>(acc[i][j] * inv);
  }
}

template <typename T, int D, int DV>
void launch_one(const Problem& p, LaunchCtx& ctx) {
  dim3 grid((p.T + QT - 1) / QT, p.B * p.H);
  constexpr size_t smem = sizeof(float) * (2 * D * TS + KT * DV + QT * (KT + 1) + KT);
  auto kern = quad_simt_kernel<T, D, DV>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  kern<<<grid, NTHR, smem, ctx.stream>>>(static_cast<const T*>(p.q), static_cast<const T*>(p.k),
                                         static_cast<const T*>(p.v), static_cast<T*>(p.out), p.T,
                                         p.feature_order, p.groups);
  note_launch(ctx);
}

template <typename T, int D>
void launch_dv(const Problem& p, LaunchCtx& ctx) {
  switch (p.d_v) {
    case 16: launch_one<T, D, 16>(p, ctx); break;
    case 32: launch_one<T, D, 32>(p, ctx); break;
    default: launch_one<T, D, 64>(p, ctx); break;
  }
}

template <typename T>
void launch_d(const Problem& p, LaunchCtx& ctx) {
  switch (p.d_k) {
    case 16: launch_dv<T, 16>(p, ctx); break;
    case 32: launch_dv<T, 32>(p, ctx); break;
    default: launch_dv<T, 64>(p, ctx); break;
  }
}

}  // namespace

void simt_quadratic(const Problem& p, LaunchCtx& ctx) {
  if (p.dtype == KATA_F32) launch_d<float>(p, ctx);
  else launch_d<__nv_bfloat16>(p, ctx);
}

}  // namespace kata
