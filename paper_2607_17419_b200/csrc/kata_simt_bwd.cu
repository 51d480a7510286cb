// Backward of the quadratic form on plain fp32 FMAs: gradients of L = sum(dout * o) with respect to q, k, v.
//
// With s_g = q_t,g . k_i,g per feature block g, r_i = 1/||k_i||^2 and the causal weights
//   a_ti = r_i sum_g s_g^2   (feature_order 2; the query norm cancels in o and is left out)
//   a_ti = q_t . k_i         (feature_order 1)
// the forward is D_t = sum_i a_ti, o_t = sum_i a_ti v_i / D_t.  Chain rule:
//   g_ti  = dL/da_ti = (dout_t . v_i - dout_t . o_t) / D_t          (0 where D_t = 0)
//   dv_i  = sum_t (a_ti / D_t) dout_t
//   dq_t,g = sum_i e_ti,g k_i,g,   dk_i,g = sum_t e_ti,g q_t,g - 2 r_i k_i,g sum_t g_ti a_ti
//   e_ti,g = 2 g_ti r_i s_g  (order 2; the last term of dk is the derivative of r_i),  e_ti = g_ti (order 1).
// Two kernels, 64 x 64 tiles, no atomics, every sum in a fixed order (bit-reproducible):
//   bwd_q_kernel   one CTA per 64 queries: a first sweep over the key tiles gives D_t and dout_t . o_t (kept in
//                  the workspace), a second sweep accumulates dq;
//   bwd_kv_kernel  one CTA per 64 keys: sweep over the query tiles at or after it, accumulates dk, dv.
#include "kata_common.cuh"

namespace kata {
namespace {

constexpr int TQ = 64;   // rows of a tile (queries or keys)
constexpr int NTHR = 128;
constexpr int TS = 68;   // row stride of the transposed tiles
constexpr int PS = 65;   // row stride of the pair matrices

template <int D, int DV> struct BwdSmem {
  // transposed q, k, dout, v tiles (for the 64 x 64 dot products), one row-major tile (the right-hand side of
  // the accumulation), two pair matrices, per-row and per-key scalars
  static constexpr int FLOATS = 2 * D * TS + 2 * DV * TS + TQ * (D > DV ? D : DV) + 2 * TQ * PS + 8 * TQ;
};

// x[rows0 + r][a] -> dstT[a][r] (and optionally row-major dst[r][a]); rows beyond Tlen read as zero
template <typename T, int W>
__device__ __forceinline__ void load_tile(const T* __restrict__ src, int row0, int Tlen, float (*dstT)[TS], float* dst_rm,
                                          int tid) {
  for (int idx = tid; idx < TQ * W; idx += NTHR) {
    const int r = idx / W, a = idx % W;
    const float x = (row0 + r < Tlen) ? to_f32(src[(size_t)(row0 + r) * W + a]) : 0.f;
    if (dstT != nullptr) dstT[a][r] = x;
    if (dst_rm != nullptr) dst_rm[r * W + a] = x;
  }
}

// 4 x 8 micro-tile of X^T Y over features [a0, a1): out[i][j] = sum_a xT[a][ty*4+i] yT[a][tx*8+j]
__device__ __forceinline__ void dot_tile(float (*xT)[TS], float (*yT)[TS], int a0, int a1, int ty, int tx, float (&out)[4][8]) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) out[i][j] = 0.f;
#pragma unroll 4
  for (int a = a0; a < a1; ++a) {
    const float4 xa = *reinterpret_cast<const float4*>(&xT[a][ty * 4]);
    const float4 y0 = *reinterpret_cast<const float4*>(&yT[a][tx * 8]);
    const float4 y1 = *reinterpret_cast<const float4*>(&yT[a][tx * 8 + 4]);
    const float xx[4] = {xa.x, xa.y, xa.z, xa.w};
    const float yy[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) out[i][j] = fmaf(xx[i], yy[j], out[i][j]);
  }
}

template <typename T, int D, int DV>
__global__ void __launch_bounds__(NTHR) bwd_q_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                      const T* __restrict__ v, const T* __restrict__ dout,
                                                      T* __restrict__ dq, float* __restrict__ stats, int Tlen,
                                                      int order, int groups) {
  extern __shared__ __align__(16) float smem[];
  float (*qT)[TS] = reinterpret_cast<float (*)[TS]>(smem);
  float (*kT)[TS] = reinterpret_cast<float (*)[TS]>(smem + D * TS);
  float (*gT)[TS] = reinterpret_cast<float (*)[TS]>(smem + 2 * D * TS);             // dout tile, transposed
  float (*vT)[TS] = reinterpret_cast<float (*)[TS]>(smem + 2 * D * TS + DV * TS);
  float* krm = smem + 2 * D * TS + 2 * DV * TS;                                      // key tile, row-major [64][D]
  float (*E)[PS] = reinterpret_cast<float (*)[PS]>(krm + TQ * (D > DV ? D : DV));
  float* rk = reinterpret_cast<float*>(E) + 2 * TQ * PS;                             // r_i of the key tile
  float* rowD = rk + TQ;                                                             // D_t, then 1 / D_t
  float* rowM = rowD + TQ;                                                           // sum a c, then dout_t . o_t

  const int tid = threadIdx.x, ty = tid >> 3, tx = tid & 7;
  const int qtile = gridDim.x - 1 - blockIdx.x;
  const size_t bh = blockIdx.y;
  const int q0 = qtile * TQ;
  const T* qh = q + bh * (size_t)Tlen * D;
  const T* kh = k + bh * (size_t)Tlen * D;
  const T* vh = v + bh * (size_t)Tlen * DV;
  const T* gh = dout + bh * (size_t)Tlen * DV;
  const int mblk = D / groups;

  load_tile<T, D>(qh, q0, Tlen, qT, nullptr, tid);
  load_tile<T, DV>(gh, q0, Tlen, gT, nullptr, tid);
  if (tid < TQ) { rowD[tid] = 0.f; rowM[tid] = 0.f; }

  constexpr int NJ = D / 8;
  float acc[4][NJ];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < NJ; ++j) acc[i][j] = 0.f;

  for (int sweep = 0; sweep < 2; ++sweep) {
    for (int kt = 0; kt <= qtile; ++kt) {
      const int k0 = kt * TQ;
      __syncthreads();
      load_tile<T, D>(kh, k0, Tlen, kT, sweep == 1 ? krm : nullptr, tid);
      load_tile<T, DV>(vh, k0, Tlen, vT, nullptr, tid);
      __syncthreads();
      if (tid < TQ) {
        float s = 0.f;
#pragma unroll 8
        for (int a = 0; a < D; ++a) s = fmaf(kT[a][tid], kT[a][tid], s);
        rk[tid] = (order == 2) ? inv_or_zero(s) : 1.f;
      }
      float c[4][8], s[4][8], a2[4][8];
      dot_tile(gT, vT, 0, DV, ty, tx, c);                 // c_ti = dout_t . v_i
      __syncthreads();                                    // rk visible
      if (sweep == 0) {
        // a_ti, then D_t += a, M_t += a c
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) a2[i][j] = 0.f;
        for (int gb = 0; gb < groups; ++gb) {
          dot_tile(qT, kT, gb * mblk, (gb + 1) * mblk, ty, tx, s);
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) a2[i][j] = (order == 2) ? fmaf(s[i][j], s[i][j], a2[i][j]) : s[i][j];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float dsum = 0.f, msum = 0.f;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int r = ty * 4 + i, cc = tx * 8 + j;
            const bool live = (k0 + cc <= q0 + r) && (k0 + cc < Tlen);
            const float a = live ? a2[i][j] * rk[cc] : 0.f;
            dsum += a;
            msum = fmaf(a, c[i][j], msum);
          }
          // the 8 threads of a row sit in one warp quarter: lanes tx = 0..7
          dsum += __shfl_xor_sync(0xffffffffu, dsum, 1); msum += __shfl_xor_sync(0xffffffffu, msum, 1);
          dsum += __shfl_xor_sync(0xffffffffu, dsum, 2); msum += __shfl_xor_sync(0xffffffffu, msum, 2);
          dsum += __shfl_xor_sync(0xffffffffu, dsum, 4); msum += __shfl_xor_sync(0xffffffffu, msum, 4);
          if (tx == 0) { rowD[ty * 4 + i] += dsum; rowM[ty * 4 + i] += msum; }
        }
      } else {
        // e_ti,g = 2 g_ti r_i s_g (order 2) or g_ti (order 1), then dq_t,g += sum_i e_ti,g k_i,g
        for (int gb = 0; gb < groups; ++gb) {
          dot_tile(qT, kT, gb * mblk, (gb + 1) * mblk, ty, tx, s);
          __syncthreads();                                // the previous group's E fully consumed
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int r = ty * 4 + i, cc = tx * 8 + j;
              const bool live = (k0 + cc <= q0 + r) && (k0 + cc < Tlen);
              const float g = (c[i][j] - rowM[r]) * rowD[r];
              const float e = (order == 2) ? 2.f * g * rk[cc] * s[i][j] : g;
              E[r][cc] = live ? e : 0.f;
            }
          __syncthreads();
          // columns of this group only: thread (ty, tx) owns columns tx + 8 j
#pragma unroll 4
          for (int i2 = 0; i2 < TQ; ++i2) {
            float ev[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) ev[i] = E[ty * 4 + i][i2];
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
              const int col = tx + 8 * j;
              if (col / mblk != gb) continue;
              const float kk = krm[i2 * D + col];
#pragma unroll
              for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(ev[i], kk, acc[i][j]);
            }
          }
        }
      }
    }
    if (sweep == 0) {
      __syncthreads();
      if (tid < TQ) {
        const float Dt = rowD[tid];
        const float inv = (order == 2) ? (Dt > 0.f ? 1.f / Dt : 0.f) : (Dt != 0.f ? 1.f / Dt : 0.f);
        const float delta = rowM[tid] * inv;               // dout_t . o_t
        rowD[tid] = inv;
        rowM[tid] = delta;
        if (q0 + tid < Tlen) {
          stats[(bh * Tlen + q0 + tid) * 2] = inv;
          stats[(bh * Tlen + q0 + tid) * 2 + 1] = delta;
        }
      }
    }
  }
  T* dqh = dq + bh * (size_t)Tlen * D;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = q0 + ty * 4 + i;
    if (r >= Tlen) continue;
#pragma unroll
    for (int j = 0; j < NJ; ++j) dqh[(size_t)r * D + tx + 8 * j] = from_f32<T>(acc[i][j]);
  }
}

template <typename T, int D, int DV>
__global__ void __launch_bounds__(NTHR) bwd_kv_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                       const T* __restrict__ v, const T* __restrict__ dout,
                                                       T* __restrict__ dk, T* __restrict__ dv,
                                                       const float* __restrict__ stats, int Tlen, int order, int groups) {
  extern __shared__ __align__(16) float smem[];
  float (*qT)[TS] = reinterpret_cast<float (*)[TS]>(smem);
  float (*kT)[TS] = reinterpret_cast<float (*)[TS]>(smem + D * TS);
  float (*gT)[TS] = reinterpret_cast<float (*)[TS]>(smem + 2 * D * TS);
  float (*vT)[TS] = reinterpret_cast<float (*)[TS]>(smem + 2 * D * TS + DV * TS);
  float* rm = smem + 2 * D * TS + 2 * DV * TS;                                       // query or dout tile, row-major
  float (*E)[PS] = reinterpret_cast<float (*)[PS]>(rm + TQ * (D > DV ? D : DV));
  float (*P)[PS] = E + TQ;
  float* rk = reinterpret_cast<float*>(E) + 2 * TQ * PS;
  float* rowD = rk + TQ;       // 1 / D_t of the query tile
  float* rowM = rowD + TQ;     // dout_t . o_t
  float* keyE = rowM + TQ;     // sum_t g_ti a_ti per key
  float* keyP = keyE + TQ;     // [4 warps][64]: partial sums of one query tile

  const int tid = threadIdx.x, ty = tid >> 3, tx = tid & 7;
  const int ktile = blockIdx.x;                  // the first key tiles see the most queries
  const size_t bh = blockIdx.y;
  const int k0 = ktile * TQ;
  const int n_qtiles = (Tlen + TQ - 1) / TQ;
  const T* qh = q + bh * (size_t)Tlen * D;
  const T* kh = k + bh * (size_t)Tlen * D;
  const T* vh = v + bh * (size_t)Tlen * DV;
  const T* gh = dout + bh * (size_t)Tlen * DV;
  const int mblk = D / groups;

  load_tile<T, D>(kh, k0, Tlen, kT, nullptr, tid);
  load_tile<T, DV>(vh, k0, Tlen, vT, nullptr, tid);
  __syncthreads();
  if (tid < TQ) {
    float s = 0.f;
#pragma unroll 8
    for (int a = 0; a < D; ++a) s = fmaf(kT[a][tid], kT[a][tid], s);
    rk[tid] = (order == 2) ? inv_or_zero(s) : 1.f;
    keyE[tid] = 0.f;
  }

  // outputs: thread (ty, tx) owns key rows ty*4 .. ty*4+3 and columns tx + 8 j
  constexpr int NJK = D / 8, NJV = DV / 8;
  float acck[4][NJK], accv[4][NJV];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int j = 0; j < NJK; ++j) acck[i][j] = 0.f;
#pragma unroll
    for (int j = 0; j < NJV; ++j) accv[i][j] = 0.f;
  }

  for (int qt = ktile; qt < n_qtiles; ++qt) {
    const int q0 = qt * TQ;
    __syncthreads();
    load_tile<T, D>(qh, q0, Tlen, qT, nullptr, tid);
    load_tile<T, DV>(gh, q0, Tlen, gT, rm, tid);           // dout row-major for dv
    if (tid < TQ) {
      const bool in = q0 + tid < Tlen;
      rowD[tid] = in ? stats[(bh * Tlen + q0 + tid) * 2] : 0.f;
      rowM[tid] = in ? stats[(bh * Tlen + q0 + tid) * 2 + 1] : 0.f;
    }
    __syncthreads();
    float c[4][8], s[4][8], a2[4][8];
    dot_tile(gT, vT, 0, DV, ty, tx, c);                   // rows = queries (ty), columns = keys (tx)
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) a2[i][j] = 0.f;
    for (int gb = 0; gb < groups; ++gb) {
      dot_tile(qT, kT, gb * mblk, (gb + 1) * mblk, ty, tx, s);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) a2[i][j] = (order == 2) ? fmaf(s[i][j], s[i][j], a2[i][j]) : s[i][j];
    }
    // P_ti = a_ti / D_t and the per-key sum of g_ti a_ti
    float ke[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) ke[j] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int r = ty * 4 + i, cc = tx * 8 + j;
        const bool live = (k0 + cc <= q0 + r) && (q0 + r < Tlen) && (k0 + cc < Tlen);
        const float a = live ? a2[i][j] * rk[cc] : 0.f;
        const float g = live ? (c[i][j] - rowM[r]) * rowD[r] : 0.f;
        P[r][cc] = a * rowD[r];
        ke[j] = fmaf(g, a, ke[j]);
      }
    // keys tx*8+j: sum over the 16 values of ty (lanes differ in bits 3, 4 inside a warp; 4 warps)
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      ke[j] += __shfl_xor_sync(0xffffffffu, ke[j], 8);
      ke[j] += __shfl_xor_sync(0xffffffffu, ke[j], 16);
    }
    if ((tid & 24) == 0) {
#pragma unroll
      for (int j = 0; j < 8; ++j) keyP[(tid >> 5) * TQ + tx * 8 + j] = ke[j];
    }
    __syncthreads();                                     // P and the partial sums complete; E free
    if (tid < TQ) keyE[tid] += (keyP[tid] + keyP[TQ + tid]) + (keyP[2 * TQ + tid] + keyP[3 * TQ + tid]);
    // dv_i += sum_t P_ti dout_t
#pragma unroll 4
    for (int t = 0; t < TQ; ++t) {
      float pv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) pv[i] = P[t][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < NJV; ++j) {
        const float gg = rm[t * DV + tx + 8 * j];
#pragma unroll
        for (int i = 0; i < 4; ++i) accv[i][j] = fmaf(pv[i], gg, accv[i][j]);
      }
    }
    __syncthreads();                                     // rm (dout) consumed
    load_tile<T, D>(qh, q0, Tlen, nullptr, rm, tid);      // query tile row-major for dk
    for (int gb = 0; gb < groups; ++gb) {
      dot_tile(qT, kT, gb * mblk, (gb + 1) * mblk, ty, tx, s);
      __syncthreads();                                   // rm loaded; previous E consumed
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = ty * 4 + i, cc = tx * 8 + j;
          const bool live = (k0 + cc <= q0 + r) && (q0 + r < Tlen) && (k0 + cc < Tlen);
          const float g = (c[i][j] - rowM[r]) * rowD[r];
          const float e = (order == 2) ? 2.f * g * rk[cc] * s[i][j] : g;
          E[r][cc] = live ? e : 0.f;
        }
      __syncthreads();
#pragma unroll 4
      for (int t = 0; t < TQ; ++t) {
        float ev[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) ev[i] = E[t][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < NJK; ++j) {
          const int col = tx + 8 * j;
          if (col / mblk != gb) continue;
          const float qq = rm[t * D + col];
#pragma unroll
          for (int i = 0; i < 4; ++i) acck[i][j] = fmaf(ev[i], qq, acck[i][j]);
        }
      }
    }
  }
  __syncthreads();
  T* dkh = dk + bh * (size_t)Tlen * D;
  T* dvh = dv + bh * (size_t)Tlen * DV;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int rl = ty * 4 + i, r = k0 + rl;
    if (r >= Tlen) continue;
    const float corr = (order == 2) ? 2.f * rk[rl] * keyE[rl] : 0.f;     // derivative of r_i = 1 / ||k_i||^2
#pragma unroll
    for (int j = 0; j < NJK; ++j) {
      const int col = tx + 8 * j;
      dkh[(size_t)r * D + col] = from_f32<T>(acck[i][j] - corr * kT[col][rl]);
    }
#pragma unroll
    for (int j = 0; j < NJV; ++j) dvh[(size_t)r * DV + tx + 8 * j] = from_f32<T>(accv[i][j]);
  }
}

template <typename T, int D, int DV>
void launch_one(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* stats, LaunchCtx& ctx) {
  constexpr size_t smem = sizeof(float) * BwdSmem<D, DV>::FLOATS;
  auto kq = bwd_q_kernel<T, D, DV>;
  auto kkv = bwd_kv_kernel<T, D, DV>;
  if (cudaFuncSetAttribute(kq, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
      cudaFuncSetAttribute(kkv, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  dim3 grid((p.T + TQ - 1) / TQ, p.B * p.H);
  kq<<<grid, NTHR, smem, ctx.stream>>>(static_cast<const T*>(p.q), static_cast<const T*>(p.k), static_cast<const T*>(p.v),
                                       static_cast<const T*>(dout), static_cast<T*>(dq), stats, p.T, p.feature_order,
                                       p.groups);
  note_launch(ctx);
  kkv<<<grid, NTHR, smem, ctx.stream>>>(static_cast<const T*>(p.q), static_cast<const T*>(p.k), static_cast<const T*>(p.v),
                                        static_cast<const T*>(dout), static_cast<T*>(dk), static_cast<T*>(dv), stats, p.T,
                                        p.feature_order, p.groups);
  note_launch(ctx);
}

template <typename T, int D>
void launch_dv(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* stats, LaunchCtx& ctx) {
  switch (p.d_v) {
    case 16: launch_one<T, D, 16>(p, dout, dq, dk, dv, stats, ctx); break;
    case 32: launch_one<T, D, 32>(p, dout, dq, dk, dv, stats, ctx); break;
    default: launch_one<T, D, 64>(p, dout, dq, dk, dv, stats, ctx); break;
  }
}

template <typename T>
void launch_d(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* stats, LaunchCtx& ctx) {
  switch (p.d_k) {
    case 16: launch_dv<T, 16>(p, dout, dq, dk, dv, stats, ctx); break;
    case 32: launch_dv<T, 32>(p, dout, dq, dk, dv, stats, ctx); break;
    default: launch_dv<T, 64>(p, dout, dq, dk, dv, stats, ctx); break;
  }
}

}  // namespace

size_t simt_bwd_workspace_elems(int BH, int T) { return (size_t)BH * T * 2; }

// stats: [BH][T][2] floats of scratch (1 / D_t and dout_t . o_t)
void simt_bwd_quadratic(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* stats, LaunchCtx& ctx) {
  if (p.dtype == KATA_F32) launch_d<float>(p, dout, dq, dk, dv, stats, ctx);
  else launch_d<__nv_bfloat16>(p, dout, dq, dk, dv, stats, ctx);
}

}  // namespace kata
