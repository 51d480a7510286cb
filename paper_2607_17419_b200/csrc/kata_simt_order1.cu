// feature_order = 1: normalised causal linear attention whose features are the rows of q,k as given
// (the "already-feature-mapped inputs" of the associative-scan appendix), state S in R^{d_k x d_v},
// Z in R^{d_k}.  Same three-stage pipeline as the second-order path: chunk-local states
// S_loc = K_[c]^T V_[c], Z_loc = 1^T K_[c]; log-depth exclusive prefix; chunk output
// N = Q S_pre + tril(Q K^T) V, D = Q Z_pre + tril(Q K^T) 1, O = N / D.  fp32 FMAs throughout.
#include "kata_common.cuh"

namespace kata {
namespace {

constexpr int C = kChunk;
constexpr int NTHR = 256;
constexpr int TS = 68;

template <int D, int DV> struct O1 {
  static constexpr size_t STATE_ELEMS = (size_t)D * DV + D;
  static constexpr int SMEM_FLOATS = 2 * D * TS + C * (D + 4) + C * DV + C * (C + 1) + D * DV + D + C;
};

template <typename T, int D, int DV>
__global__ void __launch_bounds__(NTHR) order1_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                       const T* __restrict__ v, T* __restrict__ out, int Tlen,
                                                       int n_chunks, int chunks_per_group, int n_groups,
                                                       const float* __restrict__ init_state,
                                                       float* __restrict__ final_state, int write_out) {
  extern __shared__ __align__(16) float smem[];
  constexpr int RS = D + 4;
  float (*qT)[TS] = reinterpret_cast<float (*)[TS]>(smem);
  float (*kT)[TS] = reinterpret_cast<float (*)[TS]>(smem + D * TS);
  float (*ks)[RS] = reinterpret_cast<float (*)[RS]>(smem + 2 * D * TS);
  float (*vs)[DV] = reinterpret_cast<float (*)[DV]>(smem + 2 * D * TS + C * RS);
  float (*P)[C + 1] = reinterpret_cast<float (*)[C + 1]>(smem + 2 * D * TS + C * RS + C * DV);
  float (*Ss)[DV] = reinterpret_cast<float (*)[DV]>(smem + 2 * D * TS + C * RS + C * DV + C * (C + 1));
  float* Zs = smem + 2 * D * TS + C * RS + C * DV + C * (C + 1) + D * DV;
  float* Dn = Zs + D;

  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const size_t bh = blockIdx.x;
  const int grp = blockIdx.y;
  constexpr size_t E = O1<D, DV>::STATE_ELEMS;

  if (init_state != nullptr && grp > 0) {
    const float* src = init_state + (bh * n_groups + (grp - 1)) * E;
    for (int i = tid; i < D * DV; i += NTHR) (&Ss[0][0])[i] = src[i];
    for (int i = tid; i < D; i += NTHR) Zs[i] = src[D * DV + i];
  } else {
    for (int i = tid; i < D * DV; i += NTHR) (&Ss[0][0])[i] = 0.f;
    for (int i = tid; i < D; i += NTHR) Zs[i] = 0.f;
  }

  const T* qh = q + bh * (size_t)Tlen * D;
  const T* kh = k + bh * (size_t)Tlen * D;
  const T* vh = v + bh * (size_t)Tlen * DV;
  T* oh = out + bh * (size_t)Tlen * DV;
  const int c_begin = grp * chunks_per_group;
  const int c_end = min(n_chunks, c_begin + chunks_per_group);
  constexpr int NJ = DV / 16;

  for (int c = c_begin; c < c_end; ++c) {
    const int t0 = c * C;
    __syncthreads();
    for (int idx = tid; idx < C * D; idx += NTHR) {
      const int r = idx / D, a = idx % D;
      const bool ok = t0 + r < Tlen;
      const float kv = ok ? to_f32(kh[(size_t)(t0 + r) * D + a]) : 0.f;
      qT[a][r] = (ok && write_out) ? to_f32(qh[(size_t)(t0 + r) * D + a]) : 0.f;
      kT[a][r] = kv;
      ks[r][a] = kv;
    }
    for (int idx = tid; idx < C * DV; idx += NTHR) {
      const int r = idx / DV, cc = idx % DV;
      vs[r][cc] = (t0 + r < Tlen) ? to_f32(vh[(size_t)(t0 + r) * DV + cc]) : 0.f;
    }
    __syncthreads();
    if (write_out) {
      // scores P = tril(Q K^T): 4x4 micro-tile per thread
      {
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
        for (int a = 0; a < D; ++a) {
          const float4 qa = *reinterpret_cast<const float4*>(&qT[a][ty * 4]);
          const float4 ka = *reinterpret_cast<const float4*>(&kT[a][tx * 4]);
          const float qq[4] = {qa.x, qa.y, qa.z, qa.w};
          const float kk[4] = {ka.x, ka.y, ka.z, ka.w};
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = fmaf(qq[i], kk[j], s[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = ty * 4 + i, i2 = tx * 4 + j;
            P[t][i2] = (i2 <= t) ? s[i][j] : 0.f;
          }
      }
      __syncthreads();
      // N = P V + Q S, D = P 1 + Q Z
      float acc[4][NJ];
      float dn[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        dn[i] = 0.f;
#pragma unroll
        for (int j = 0; j < NJ; ++j) acc[i][j] = 0.f;
      }
      for (int i2 = 0; i2 < C; ++i2) {
        float w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          w[i] = P[ty * 4 + i][i2];
          dn[i] += w[i];
        }
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          const float vv = vs[i2][tx + 16 * j];
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(w[i], vv, acc[i][j]);
        }
      }
      for (int a = 0; a < D; ++a) {
        const float4 qa = *reinterpret_cast<const float4*>(&qT[a][ty * 4]);
        const float qq[4] = {qa.x, qa.y, qa.z, qa.w};
        const float z = Zs[a];
#pragma unroll
        for (int i = 0; i < 4; ++i) dn[i] = fmaf(qq[i], z, dn[i]);
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          const float sv = Ss[a][tx + 16 * j];
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(qq[i], sv, acc[i][j]);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = t0 + ty * 4 + i;
        if (t >= Tlen) continue;
        const float inv = dn[i] != 0.f ? 1.f / dn[i] : 0.f;
#pragma unroll
        for (int j = 0; j < NJ; ++j) oh[(size_t)t * DV + tx + 16 * j] = from_f32<T>(acc[i][j] * inv);
      }
      __syncthreads();   // all reads of S, Z done before the update
    }
    const bool need_update = (c + 1 < c_end) || (final_state != nullptr);
    if (need_update) {
      if (ty < D / 4) {
        float acc[4][NJ];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < NJ; ++j) acc[i][j] = 0.f;
        for (int t = 0; t < C; ++t) {
          const float4 ka = *reinterpret_cast<const float4*>(&ks[t][ty * 4]);
          const float kk[4] = {ka.x, ka.y, ka.z, ka.w};
#pragma unroll
          for (int j = 0; j < NJ; ++j) {
            const float vv = vs[t][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(kk[i], vv, acc[i][j]);
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < NJ; ++j) Ss[ty * 4 + i][tx + 16 * j] += acc[i][j];
      }
      if (tid >= NTHR - D) {
        const int a = tid - (NTHR - D);
        float z = 0.f;
        for (int t = 0; t < C; ++t) z += ks[t][a];
        Zs[a] += z;
      }
    }
  }
  if (final_state != nullptr) {
    __syncthreads();
    float* dst = final_state + (bh * n_groups + grp) * E;
    for (int i = tid; i < D * DV; i += NTHR) dst[i] = (&Ss[0][0])[i];
    for (int i = tid; i < D; i += NTHR) dst[D * DV + i] = Zs[i];
  }
  (void)Dn;
}

template <int D, int DV>
__global__ void order1_export_kernel(const float* __restrict__ incl, float* __restrict__ s_pre,
                                     float* __restrict__ z_pre, int n_chunks) {
  constexpr size_t E = O1<D, DV>::STATE_ELEMS;
  const int c = blockIdx.x;
  const size_t bh = blockIdx.y;
  float* sp = s_pre + (bh * n_chunks + c) * (size_t)D * DV;
  float* zp = z_pre + (bh * n_chunks + c) * (size_t)D;
  const float* src = incl + (bh * n_chunks + (c > 0 ? c - 1 : 0)) * E;
  for (int i = threadIdx.x; i < D * DV; i += blockDim.x) sp[i] = c > 0 ? src[i] : 0.f;
  for (int i = threadIdx.x; i < D; i += blockDim.x) zp[i] = c > 0 ? src[D * DV + i] : 0.f;
}

template <typename T, int D, int DV>
void run(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, float* s_pre, float* z_pre,
         LaunchCtx& ctx) {
  auto kern = order1_kernel<T, D, DV>;
  constexpr size_t smem = sizeof(float) * O1<D, DV>::SMEM_FLOATS;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  const T* q = static_cast<const T*>(p.q);
  const T* k = static_cast<const T*>(p.k);
  const T* v = static_cast<const T*>(p.v);
  T* o = static_cast<T*>(p.out);
  const int BH = p.B * p.H;
  if (!use_scan) {
    kern<<<dim3(BH, 1), NTHR, smem, ctx.stream>>>(q, k, v, o, p.T, plan.n_chunks, plan.n_chunks, 1, nullptr,
                                                 nullptr, 1);
    note_launch(ctx);
    return;
  }
  const int NG = plan.n_groups;
  constexpr size_t E = O1<D, DV>::STATE_ELEMS;
  float* bufA = ws;
  float* bufB = ws + (size_t)BH * NG * E;
  const float* incl = bufA;
  if (NG > 1) {
    kern<<<dim3(BH, NG - 1), NTHR, smem, ctx.stream>>>(q, k, v, o, p.T, plan.n_chunks, plan.chunks_per_group, NG,
                                                      nullptr, bufA, 0);
    note_launch(ctx);
    incl = scan_group_states(bufA, bufB, BH, NG, NG - 1, E, ctx);
  }
  kern<<<dim3(BH, NG), NTHR, smem, ctx.stream>>>(q, k, v, o, p.T, plan.n_chunks, plan.chunks_per_group, NG, incl,
                                                nullptr, 1);
  note_launch(ctx);
  if (s_pre != nullptr && z_pre != nullptr) {
    order1_export_kernel<D, DV><<<dim3(plan.n_chunks, BH), 256, 0, ctx.stream>>>(incl, s_pre, z_pre, plan.n_chunks);
    note_launch(ctx);
  }
}

template <typename T, int D>
void run_dv(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, float* s_pre, float* z_pre,
            LaunchCtx& ctx) {
  switch (p.d_v) {
    case 16: run<T, D, 16>(p, plan, use_scan, ws, s_pre, z_pre, ctx); break;
    case 32: run<T, D, 32>(p, plan, use_scan, ws, s_pre, z_pre, ctx); break;
    default: run<T, D, 64>(p, plan, use_scan, ws, s_pre, z_pre, ctx); break;
  }
}

template <typename T>
void run_d(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, float* s_pre, float* z_pre,
           LaunchCtx& ctx) {
  switch (p.d_k) {
    case 16: run_dv<T, 16>(p, plan, use_scan, ws, s_pre, z_pre, ctx); break;
    case 32: run_dv<T, 32>(p, plan, use_scan, ws, s_pre, z_pre, ctx); break;
    default: run_dv<T, 64>(p, plan, use_scan, ws, s_pre, z_pre, ctx); break;
  }
}

}  // namespace

size_t order1_state_elems(int d_k, int d_v) { return (size_t)d_k * d_v + d_k; }

void order1_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, float* s_pre,
                    float* z_pre, LaunchCtx& ctx) {
  if (p.dtype == KATA_F32) run_d<float>(p, plan, use_scan, ws, s_pre, z_pre, ctx);
  else run_d<__nv_bfloat16>(p, plan, use_scan, ws, s_pre, z_pre, ctx);
}

}  // namespace kata
