// O(T) backward of the KATA forward on plain fp32 FMAs: two sweeps over the chunk axis that carry linear states
// (table "Training-step latency versus sequence length": the two-pass linear-state backward).
//
// With x_hat = x / ||x||, s_ti = q_hat_t . k_hat_i, w_ti = s_ti^2 (i <= t), N_t = sum_i w_ti v_i, D_t = sum_i w_ti,
// o_t = N_t / D_t and g_t = dL/do_t, the chain rule through the definition gives
//   u_t = g_t / D_t,  c_t = (g_t . o_t) / D_t,  dL/dw_ti = u_t . v_i - c_t,
//   dv_i     = sum_{t>=i} w_ti u_t,
//   dq_hat_t = 2 sum_{i<=t} s_ti (u_t . v_i - c_t) k_hat_i,   dk_hat_i = 2 sum_{t>=i} s_ti (u_t . v_i - c_t) q_hat_t,
//   dx = (dx_hat - x_hat (x_hat . dx_hat)) / ||x||.
// Every sum over the tokens outside the current chunk is a contraction with a running state over the symmetric
// feature pairs f = (a <= b):
//   forward sweep   S[f] = sum_i k_hat_ia k_hat_ib [v_i, 1]:   [N_t, D_t] = sum_f m_f q_hat_ta q_hat_tb S[f]  (m = 1 on the
//                   diagonal, 2 off it),   dq_hat_t = 2 G_t q_hat_t  with  G_t[a,b] = S[f(a,b)] . [u_t, -c_t];
//   reverse sweep   R[f] = sum_t q_hat_ta q_hat_tb [u_t, c_t]:  dv_i = sum_f m_f k_hat_ia k_hat_ib R[f][0..],
//                   dk_hat_i = 2 G_i k_hat_i  with  G_i[a,b] = R[f(a,b)] . [v_i, -1].
// Both sweeps are one kernel: "readers" X (queries forward, keys in reverse) read the state that the "writers" Y of
// the chunks already passed have built, and the tokens of the current chunk through the C x C causal scores.
//
// One CTA owns one head and 8 of the value columns; the state [n_f][8 + 1] lives in shared memory.  c_t needs all
// value columns: each slice uses its own part of g_t . o_t in the forward sweep (the gradient is linear in c_t) and
// the reverse sweep adds the parts up.  Partial dq_hat / dk_hat of the slices go to the workspace and are added in a
// fixed order by the kernel that also takes them through the normalisation: results are bit-reproducible.
#include "kata_common.cuh"

namespace kata {
namespace {

constexpr int C = kChunk;          // 64 tokens per chunk
constexpr int NT = 512;            // threads: 64 reader rows x 8 groups
constexpr int VS = 8;              // value columns per CTA
constexpr int AS = 12;             // floats per state row: 8 value columns, the normaliser column, padding

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float x);
template <> __device__ __forceinline__ void stf<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// x_hat = x / ||x|| and 1 / ||x|| per row (0 for a zero row); one warp per row.
template <typename T>
__global__ void __launch_bounds__(256) bwdc_normalise_kernel(const T* __restrict__ x, float* __restrict__ xn,
                                                             float* __restrict__ rnorm, size_t rows, int d) {
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  float a0 = lane < d ? ldf(x + row * d + lane) : 0.f;
  float a1 = lane + 32 < d ? ldf(x + row * d + lane + 32) : 0.f;
  float ss = a0 * a0 + a1 * a1;
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
  const float r = ss > 0.f ? rsqrtf(ss) : 0.f;
  // one Newton step: rsqrtf is good to 2 ulp, the gradients are checked to 1e-4
  const float rr = ss > 0.f ? r * (1.5f - 0.5f * ss * r * r) : 0.f;
  if (lane < d) xn[row * d + lane] = a0 * rr;
  if (lane + 32 < d) xn[row * d + lane + 32] = a1 * rr;
  if (lane == 0) rnorm[row] = rr;
}

__device__ __forceinline__ int pair_index(int a, int b, int d) {   // a <= b: row-major upper triangle
  return a * d - (a * (a - 1)) / 2 + (b - a);
}

__host__ __device__ inline size_t sweep_smem_floats(int d) {
  const size_t nf = (size_t)d * (d + 1) / 2;
  return nf * AS + (size_t)d * (C + 1) + (size_t)C * d + (size_t)C * C + 2 * (size_t)C * AS + 8 * (size_t)C * 9 + (size_t)C * VS;
}

// One sweep over the chunk axis.  REVERSE = false: readers X = q_hat, writers Y = k_hat, W = [v, 1]; writes u, the
// slice's part of c and the slice's part of dq_hat.  REVERSE = true: chunks in descending order, readers X = k_hat,
// writers Y = q_hat, W = [u, c]; writes dv and the slice's part of dk_hat.
template <typename T, bool REVERSE>
__global__ void __launch_bounds__(NT) bwdc_sweep_kernel(const float* __restrict__ xn, const float* __restrict__ yn,
                                                        const T* __restrict__ v, const T* __restrict__ g,
                                                        float* __restrict__ u32, float* __restrict__ cpart,
                                                        float* __restrict__ part, T* __restrict__ dv_out, int Tlen, int d,
                                                        int dv, int nsl) {
  extern __shared__ __align__(16) float smem[];
  const int nf = d * (d + 1) / 2;
  float* A9 = smem;
  float* xT = A9 + (size_t)nf * AS;
  float* ys = xT + d * (C + 1);
  float* sT = ys + C * d;
  float* W9s = sT + C * C;
  float* coefs = W9s + C * AS;
  float* red = coefs + C * AS;
  float* aux = red + 8 * C * 9;
  unsigned short* pab = reinterpret_cast<unsigned short*>(aux + C * VS);

  const int tid = threadIdx.x, t = tid & (C - 1), grp = tid >> 6;
  const size_t bh = blockIdx.x / nsl;
  const int slice = blockIdx.x % nsl;
  const size_t head = bh * (size_t)Tlen;

  for (int i = tid; i < nf * AS; i += NT) A9[i] = 0.f;
  for (int a = tid; a < d; a += NT)
    for (int b = a; b < d; ++b) pab[pair_index(a, b, d)] = (unsigned short)(a | (b << 8));
  __syncthreads();

  const int n_chunks = (Tlen + C - 1) / C;
  const int nfg = (nf + 7) / 8;
  const int na = d / 8;
  for (int it = 0; it < n_chunks; ++it) {
    const int ch = REVERSE ? n_chunks - 1 - it : it;
    const int t0 = ch * C;
    // ---- the chunk: reader rows transposed, writer rows, [W, 1 or c] of the writers, g or v of the readers ----
    for (int idx = tid; idx < C * d; idx += NT) {
      const int row = idx / d, col = idx - row * d;
      const bool in = t0 + row < Tlen;
      xT[col * (C + 1) + row] = in ? xn[(head + t0 + row) * d + col] : 0.f;
      ys[idx] = in ? yn[(head + t0 + row) * d + col] : 0.f;
    }
    for (int idx = tid; idx < C * 9; idx += NT) {
      const int row = idx / 9, c = idx - row * 9;
      const bool in = t0 + row < Tlen;
      float w = 0.f;
      if (in) {
        if (!REVERSE) {
          w = c < VS ? ldf(v + (head + t0 + row) * dv + slice * VS + c) : 1.f;
        } else if (c < VS) {
          w = u32[(head + t0 + row) * dv + slice * VS + c];
        } else {
          for (int s = 0; s < nsl; ++s) w += cpart[(bh * nsl + s) * (size_t)Tlen + t0 + row];
        }
      }
      W9s[row * AS + c] = w;
    }
    for (int idx = tid; idx < C * VS; idx += NT) {
      const int row = idx / VS, c = idx - row * VS;
      const bool in = t0 + row < Tlen;
      aux[idx] = in ? ldf((REVERSE ? v : g) + (head + t0 + row) * dv + slice * VS + c) : 0.f;
    }
    __syncthreads();
    // ---- causal scores of the chunk, [yi][t] ----
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
      const int yi = grp * 8 + j;
      float s = 0.f;
      for (int e = 0; e < d; ++e) s = fmaf(xT[e * (C + 1) + t], ys[yi * d + e], s);
      const bool keep = REVERSE ? yi >= t : yi <= t;
      sT[yi * C + t] = keep ? s : 0.f;
    }
    // ---- [N | D] (forward) or [dv | .] (reverse) of reader t: this group's features and writers ----
    float acc[9];
#pragma unroll
    for (int c = 0; c < 9; ++c) acc[c] = 0.f;
    {
      const int f1 = min(nf, (grp + 1) * nfg);
      for (int f = grp * nfg; f < f1; ++f) {
        const unsigned ab = pab[f];
        const int a = ab & 255, b = ab >> 8;
        float p = xT[a * (C + 1) + t] * xT[b * (C + 1) + t];
        if (a != b) p *= 2.f;
        const float4 s0 = *reinterpret_cast<const float4*>(A9 + (size_t)f * AS);
        const float4 s1 = *reinterpret_cast<const float4*>(A9 + (size_t)f * AS + 4);
        const float s2 = A9[(size_t)f * AS + 8];
        acc[0] = fmaf(p, s0.x, acc[0]); acc[1] = fmaf(p, s0.y, acc[1]); acc[2] = fmaf(p, s0.z, acc[2]); acc[3] = fmaf(p, s0.w, acc[3]);
        acc[4] = fmaf(p, s1.x, acc[4]); acc[5] = fmaf(p, s1.y, acc[5]); acc[6] = fmaf(p, s1.z, acc[6]); acc[7] = fmaf(p, s1.w, acc[7]);
        acc[8] = fmaf(p, s2, acc[8]);
      }
#pragma unroll 1
      for (int j = 0; j < 8; ++j) {
        const int yi = grp * 8 + j;
        const float s = sT[yi * C + t];
        const float w = s * s;
#pragma unroll
        for (int c = 0; c < 9; ++c) acc[c] = fmaf(w, W9s[yi * AS + c], acc[c]);
      }
    }
#pragma unroll
    for (int c = 0; c < 9; ++c) red[(grp * C + t) * 9 + c] = acc[c];
    __syncthreads();
    // ---- the coefficients [u, -c] (forward) or [v, -1] (reverse) of reader t ----
    if (tid < C) {
      float r9[9];
#pragma unroll
      for (int c = 0; c < 9; ++c) {
        float s = 0.f;
#pragma unroll
        for (int gq = 0; gq < 8; ++gq) s += red[(gq * C + tid) * 9 + c];
        r9[c] = s;
      }
      const bool in = t0 + tid < Tlen;
      if (!REVERSE) {
        const float invD = r9[8] > 0.f ? 1.f / r9[8] : 0.f;
        float cp = 0.f;
#pragma unroll
        for (int c = 0; c < VS; ++c) {
          const float gg = aux[tid * VS + c];
          const float u = gg * invD;
          cp = fmaf(gg, r9[c] * invD, cp);
          coefs[tid * AS + c] = u;
          if (in) u32[(head + t0 + tid) * dv + slice * VS + c] = u;
        }
        cp *= invD;
        coefs[tid * AS + 8] = -cp;
        if (in) cpart[(bh * nsl + slice) * (size_t)Tlen + t0 + tid] = cp;
      } else {
#pragma unroll
        for (int c = 0; c < VS; ++c) {
          coefs[tid * AS + c] = aux[tid * VS + c];
          if (in) stf(dv_out + (head + t0 + tid) * dv + slice * VS + c, r9[c]);
        }
        coefs[tid * AS + 8] = slice == 0 ? -1.f : 0.f;
      }
    }
    __syncthreads();
    float cf[9];
#pragma unroll
    for (int c = 0; c < 9; ++c) cf[c] = coefs[t * AS + c];
    // ---- dL/ds of the chunk: z_ti = 2 s_ti (W_i . coef_t), in place of the scores ----
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
      const int yi = grp * 8 + j;
      float dot = 0.f;
#pragma unroll
      for (int c = 0; c < 9; ++c) dot = fmaf(W9s[yi * AS + c], cf[c], dot);
      sT[yi * C + t] = 2.f * sT[yi * C + t] * dot;
    }
    __syncthreads();
    // ---- dx_hat of reader t, entries a of this group: 2 (G x_hat)_a + sum_i z_ti y_hat_ia ----
    for (int jj = 0; jj < na; ++jj) {
      const int a = grp * na + jj;
      float dxa = 0.f;
      for (int b = 0; b < d; ++b) {
        const int f = a <= b ? pair_index(a, b, d) : pair_index(b, a, d);
        const float4 s0 = *reinterpret_cast<const float4*>(A9 + (size_t)f * AS);
        const float4 s1 = *reinterpret_cast<const float4*>(A9 + (size_t)f * AS + 4);
        float gab = A9[(size_t)f * AS + 8] * cf[8];
        gab = fmaf(s0.x, cf[0], gab); gab = fmaf(s0.y, cf[1], gab); gab = fmaf(s0.z, cf[2], gab); gab = fmaf(s0.w, cf[3], gab);
        gab = fmaf(s1.x, cf[4], gab); gab = fmaf(s1.y, cf[5], gab); gab = fmaf(s1.z, cf[6], gab); gab = fmaf(s1.w, cf[7], gab);
        dxa = fmaf(gab, xT[b * (C + 1) + t], dxa);
      }
      dxa *= 2.f;
      for (int yi = 0; yi < C; ++yi) dxa = fmaf(sT[yi * C + t], ys[yi * d + a], dxa);
      if (t0 + t < Tlen) part[((bh * nsl + slice) * (size_t)Tlen + t0 + t) * d + a] = dxa;
    }
    __syncthreads();
    // ---- the writers of the chunk join the state ----
    for (int f = tid; f < nf; f += NT) {
      const unsigned ab = pab[f];
      const int a = ab & 255, b = ab >> 8;
      float up[9];
#pragma unroll
      for (int c = 0; c < 9; ++c) up[c] = 0.f;
      for (int i = 0; i < C; ++i) {
        const float p = ys[i * d + a] * ys[i * d + b];
#pragma unroll
        for (int c = 0; c < 9; ++c) up[c] = fmaf(p, W9s[i * AS + c], up[c]);
      }
#pragma unroll
      for (int c = 0; c < 9; ++c) A9[(size_t)f * AS + c] += up[c];
    }
    __syncthreads();
  }
}

// dx = (dx_hat - x_hat (x_hat . dx_hat)) / ||x|| with dx_hat = the slices' parts added in order; one warp per row.
template <typename T>
__global__ void __launch_bounds__(256) bwdc_finish_kernel(const float* __restrict__ part, const float* __restrict__ xn,
                                                          const float* __restrict__ rnorm, T* __restrict__ dx, int BH,
                                                          int Tlen, int d, int nsl) {
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= (size_t)BH * Tlen) return;
  const size_t bh = row / Tlen, tok = row - bh * Tlen;
  float h0 = 0.f, h1 = 0.f;
  for (int s = 0; s < nsl; ++s) {
    const float* src = part + ((bh * nsl + s) * (size_t)Tlen + tok) * d;
    if (lane < d) h0 += src[lane];
    if (lane + 32 < d) h1 += src[lane + 32];
  }
  const float x0 = lane < d ? xn[row * d + lane] : 0.f, x1 = lane + 32 < d ? xn[row * d + lane + 32] : 0.f;
  float dot = x0 * h0 + x1 * h1;
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
  const float r = rnorm[row];
  if (lane < d) stf(dx + row * d + lane, (h0 - x0 * dot) * r);
  if (lane + 32 < d) stf(dx + row * d + lane + 32, (h1 - x1 * dot) * r);
}

template <typename T>
void launch_bwd_chunked(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* ws, LaunchCtx& ctx) {
  const size_t BH = (size_t)p.B * p.H, rows = BH * p.T;
  const int d = p.d_k, nsl = p.d_v / VS;
  float* qn = ws;
  float* kn = qn + rows * d;
  float* rq = kn + rows * d;
  float* rk = rq + rows;
  float* u32 = rk + rows;
  float* cpart = u32 + rows * p.d_v;
  float* part = cpart + rows * nsl;
  const unsigned nb = (unsigned)((rows + 7) / 8);
  bwdc_normalise_kernel<T><<<nb, 256, 0, ctx.stream>>>(static_cast<const T*>(p.q), qn, rq, rows, d);
  note_launch(ctx);
  bwdc_normalise_kernel<T><<<nb, 256, 0, ctx.stream>>>(static_cast<const T*>(p.k), kn, rk, rows, d);
  note_launch(ctx);
  const size_t smem = sweep_smem_floats(d) * sizeof(float) + (size_t)d * (d + 1) / 2 * sizeof(unsigned short);
  auto fwd = bwdc_sweep_kernel<T, false>;
  auto rev = bwdc_sweep_kernel<T, true>;
  if (cudaFuncSetAttribute(fwd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
      cudaFuncSetAttribute(rev, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  const unsigned grid = (unsigned)(BH * nsl);
  fwd<<<grid, NT, smem, ctx.stream>>>(qn, kn, static_cast<const T*>(p.v), static_cast<const T*>(dout), u32, cpart, part,
                                      static_cast<T*>(nullptr), p.T, d, p.d_v, nsl);
  note_launch(ctx);
  bwdc_finish_kernel<T><<<nb, 256, 0, ctx.stream>>>(part, qn, rq, static_cast<T*>(dq), (int)BH, p.T, d, nsl);
  note_launch(ctx);
  rev<<<grid, NT, smem, ctx.stream>>>(kn, qn, static_cast<const T*>(p.v), static_cast<const T*>(nullptr), u32, cpart, part,
                                      static_cast<T*>(dv), p.T, d, p.d_v, nsl);
  note_launch(ctx);
  bwdc_finish_kernel<T><<<nb, 256, 0, ctx.stream>>>(part, kn, rk, static_cast<T*>(dk), (int)BH, p.T, d, nsl);
  note_launch(ctx);
}

}  // namespace

bool simt_bwd_chunked_supported(const Problem& p) {
  return p.feature_order == 2 && p.groups == 1 && (p.d_k == 16 || p.d_k == 32 || p.d_k == 64) && p.d_v % VS == 0 && p.d_v >= VS &&
         p.d_v <= 64;
}

// q_hat, k_hat | 1/||q||, 1/||k|| | u | the slices' parts of c | the slices' parts of dq_hat, then of dk_hat
size_t simt_bwd_chunked_workspace_elems(const Problem& p) {
  const size_t rows = (size_t)p.B * p.H * p.T, nsl = p.d_v / VS;
  return rows * (2 * (size_t)p.d_k + 2 + p.d_v + nsl + nsl * (size_t)p.d_k);
}

void simt_bwd_chunked(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* ws, LaunchCtx& ctx) {
  if (p.dtype == KATA_BF16)
    launch_bwd_chunked<__nv_bfloat16>(p, dout, dq, dk, dv, ws, ctx);
  else
    launch_bwd_chunked<float>(p, dout, dq, dk, dv, ws, ctx);
}

}  // namespace kata
