// Single-token decode step of the recurrent form (section "Linear attention as a recurrence"):
//   S <- S + psi(k) v^T,  Z <- Z + psi(k),  out = psi(q)^T S / psi(q)^T Z   (0 where the denominator is 0)
// (the readout is taken as psi(q)^T S_old + <psi(q),psi(k)> v over psi(q)^T Z_old + <psi(q),psi(k)>)
// for every (b,h), with the state in the layout of the exported prefix states (fp32; DIRECT or PACKED for the
// rank-one PSD feature, n_psi = d_k for already-mapped features).
//
// HBM-bound: the state (n_psi x (d_v + 1) floats per head) is read and written once per token.  One CTA streams
// 256 feature rows of one head: 16 threads x float4 cover the d_v = 64 floats of a row (8 threads at d_v = 32,
// 4 at d_v = 16), so a warp reads and writes whole 128-byte lines; the feature values psi(k)_r, psi(q)_r are
// formed on the fly from the two d_k-vectors kept in shared memory.  Each CTA leaves a partial numerator and
// denominator; a second small kernel adds the partials of a head in a fixed order (bit-reproducible) and writes
// the output row.
#include "kata_common.cuh"

namespace kata {
namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_ROWS = 256;     // feature rows per CTA

// feature pair (a,b) and scale of row r.  With g feature blocks (blockwise PSD map) the rows of the blocks follow
// one another and (a,b) stay inside one block of m = d / g features.
__device__ __forceinline__ void feature_pair(int r, int d, int layout, int order, int groups, int& a, int& b, float& scale) {
  if (order == 1) {
    a = r; b = -1; scale = 1.f;
    return;
  }
  const int m = d / groups;
  const int per = (layout == KATA_LAYOUT_PACKED) ? m * (m + 1) / 2 : m * m;
  const int gb = r / per;
  r -= gb * per;
  if (layout == KATA_LAYOUT_DIRECT) {
    a = r / m; b = r - a * m; scale = 1.f;
  } else {
    // upper triangle a <= b in row-major order: row a starts at a m - a (a - 1) / 2
    int aa = (int)((2.f * m + 1.f - sqrtf((2.f * m + 1.f) * (2.f * m + 1.f) - 8.f * (float)r)) * 0.5f);
    if (aa < 0) aa = 0;
    if (aa > m - 1) aa = m - 1;
    while (aa > 0 && aa * m - aa * (aa - 1) / 2 > r) --aa;
    while (aa + 1 < m && (aa + 1) * m - (aa + 1) * aa / 2 <= r) ++aa;
    a = aa; b = aa + (r - (aa * m - aa * (aa - 1) / 2));
    scale = (a == b) ? 1.f : 1.41421356237309504880f;
  }
  a += gb * m;
  b += gb * m;
}

template <typename T, int DV>
__global__ void __launch_bounds__(DEC_THREADS) decode_update_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                                    const T* __restrict__ v, float* __restrict__ S,
                                                                    float* __restrict__ Z, float* __restrict__ part,
                                                                    int d_k, int n_psi, int layout, int order, int groups) {
  constexpr int TPR = DV / 4;                  // threads per state row
  constexpr int RPI = DEC_THREADS / TPR;       // rows per iteration
  __shared__ float kh[64], qs[64], red[DEC_THREADS / 32][DV + 1];
  const int bh = blockIdx.y, slab = blockIdx.x, n_slabs = gridDim.x;
  const int tid = threadIdx.x;
  // Launched with programmatic stream serialisation: the CTAs may be resident before the kernel ahead in the stream
  // (the producer of q, k, v, or the previous step's finish kernel, which still reads `part`) has ended.
  cudaGridDependencySynchronize();
  // k_hat = k / ||k|| (zero row -> zero feature); the query norm cancels in the readout and is not applied
  if (tid < 64) {
    float kv = tid < d_k ? to_f32<T>(k[(size_t)bh * d_k + tid]) : 0.f;
    float ss = kv * kv;
    if (order == 1) {
      kh[tid] = kv;
    } else {
      ss += __shfl_xor_sync(0xffffffffu, ss, 16);
      ss += __shfl_xor_sync(0xffffffffu, ss, 8);
      ss += __shfl_xor_sync(0xffffffffu, ss, 4);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      red[tid >> 5][0] = ss;
    }
    qs[tid] = tid < d_k ? to_f32<T>(q[(size_t)bh * d_k + tid]) : 0.f;
  }
  __syncthreads();
  if (order != 1 && tid < 64) kh[tid] = (tid < d_k ? to_f32<T>(k[(size_t)bh * d_k + tid]) : 0.f) * rsqrt_or_zero(red[0][0] + red[1][0]);
  __syncthreads();

  const int col = (tid % TPR) * 4;
  const float4 vv = make_float4(to_f32<T>(v[(size_t)bh * DV + col]), to_f32<T>(v[(size_t)bh * DV + col + 1]),
                                to_f32<T>(v[(size_t)bh * DV + col + 2]), to_f32<T>(v[(size_t)bh * DV + col + 3]));
  float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
  float den = 0.f;
  float* Sh = S + (size_t)bh * n_psi * DV;
  float* Zh = Z + (size_t)bh * n_psi;
  const int r_end = min(n_psi, (slab + 1) * DEC_ROWS);
  // four rows per thread in flight: all loads of a group are issued before the first store
  constexpr int UNR = 4;
  for (int r0 = slab * DEC_ROWS + tid / TPR; r0 < r_end; r0 += UNR * RPI) {
    float4 s[UNR];
    float z[UNR], fk[UNR], fq[UNR];
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int r = r0 + u * RPI;
      if (r < r_end) {
        s[u] = *reinterpret_cast<const float4*>(Sh + (size_t)r * DV + col);
        z[u] = (tid % TPR == 0) ? Zh[r] : 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int r = r0 + u * RPI;
      int a, b;
      float scale;
      feature_pair(r < r_end ? r : 0, d_k, layout, order, groups, a, b, scale);
      fk[u] = (b < 0) ? kh[a] : kh[a] * kh[b] * scale;
      fq[u] = (b < 0) ? qs[a] : qs[a] * qs[b] * scale;
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int r = r0 + u * RPI;
      if (r < r_end) {
        // read the state of the earlier tokens, then add this token (its own weight is added exactly at the end)
        num.x = fmaf(fq[u], s[u].x, num.x);
        num.y = fmaf(fq[u], s[u].y, num.y);
        num.z = fmaf(fq[u], s[u].z, num.z);
        num.w = fmaf(fq[u], s[u].w, num.w);
        s[u].x = fmaf(fk[u], vv.x, s[u].x);
        s[u].y = fmaf(fk[u], vv.y, s[u].y);
        s[u].z = fmaf(fk[u], vv.z, s[u].z);
        s[u].w = fmaf(fk[u], vv.w, s[u].w);
        *reinterpret_cast<float4*>(Sh + (size_t)r * DV + col) = s[u];
        if (tid % TPR == 0) {
          den = fmaf(fq[u], z[u], den);
          Zh[r] = z[u] + fk[u];
        }
      }
    }
  }
  // rows of one warp: sum over the lanes that share a column group, then over the warps (fixed order)
#pragma unroll
  for (int off = TPR; off < 32; off <<= 1) {
    num.x += __shfl_xor_sync(0xffffffffu, num.x, off);
    num.y += __shfl_xor_sync(0xffffffffu, num.y, off);
    num.z += __shfl_xor_sync(0xffffffffu, num.z, off);
    num.w += __shfl_xor_sync(0xffffffffu, num.w, off);
    den += __shfl_xor_sync(0xffffffffu, den, off);
  }
  __syncthreads();
  const int lane = tid & 31, warp = tid >> 5;
  if (lane < TPR) {
    red[warp][lane * 4] = num.x; red[warp][lane * 4 + 1] = num.y; red[warp][lane * 4 + 2] = num.z; red[warp][lane * 4 + 3] = num.w;
    if (lane == 0) red[warp][DV] = den;
  }
  __syncthreads();
  if (tid <= DV) {
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_THREADS / 32; ++w) acc += red[w][tid];
    part[((size_t)bh * n_slabs + slab) * (DV + 1) + tid] = acc;
  }
}

// Adds the partials of the earlier tokens' state in a fixed order, then this token's own term with its weight
// <psi(q), psi(k)> formed directly from the dot product (exact where the feature-space sum would cancel).
template <typename T, int DV>
__global__ void decode_finish_kernel(const float* __restrict__ part, const T* __restrict__ q, const T* __restrict__ k,
                                     const T* __restrict__ v, T* __restrict__ out, int n_slabs, int d_k, int order,
                                     int groups) {
  const int bh = blockIdx.x, c = threadIdx.x;
  float kk = 0.f, w = 0.f;
  const int m = d_k / groups;
  for (int gb = 0; gb < groups; ++gb) {
    float qk = 0.f;
    for (int a = gb * m; a < (gb + 1) * m; ++a) {
      const float qa = to_f32<T>(q[(size_t)bh * d_k + a]), ka = to_f32<T>(k[(size_t)bh * d_k + a]);
      qk = fmaf(qa, ka, qk);
      kk = fmaf(ka, ka, kk);
    }
    w += (order == 1) ? qk : qk * qk;
  }
  if (order != 1) w *= inv_or_zero(kk);     // raw q: the query norm cancels in the ratio
  // Launched with programmatic stream serialisation: everything above ran while the update kernel was still
  // streaming the state; its partial sums are visible from here on.
  cudaGridDependencySynchronize();
  if (c >= DV) return;
  float num = 0.f, den = 0.f;
  for (int s = 0; s < n_slabs; ++s) {
    num += part[((size_t)bh * n_slabs + s) * (DV + 1) + c];
    den += part[((size_t)bh * n_slabs + s) * (DV + 1) + DV];
  }
  num = fmaf(w, to_f32<T>(v[(size_t)bh * DV + c]), num);
  den += w;
  out[(size_t)bh * DV + c] = from_f32<T>(den != 0.f ? num / den : 0.f);
}

template <typename T, int DV>
void launch(const void* q, const void* k, const void* v, void* out, float* S, float* Z, float* part, int BH, int d_k,
            int n_psi, int layout, int order, int groups, LaunchCtx& ctx) {
  const int n_slabs = decode_slabs(n_psi);
  // both kernels may become resident before the kernel ahead of them has ended (each waits inside: the update kernel
  // at its top, the finish kernel after its own prologue)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_slabs, BH);
  cfg.blockDim = dim3(DEC_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = ctx.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const float* part_c = part;
  const T *qc = static_cast<const T*>(q), *kc = static_cast<const T*>(k), *vc = static_cast<const T*>(v);
  T* oc = static_cast<T*>(out);
  if (cudaLaunchKernelEx(&cfg, decode_update_kernel<T, DV>, qc, kc, vc, S, Z, part, d_k, n_psi, layout, order, groups) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  ++ctx.launches;
  cfg.gridDim = dim3(BH);
  cfg.blockDim = dim3(64);
  if (cudaLaunchKernelEx(&cfg, decode_finish_kernel<T, DV>, part_c, qc, kc, vc, oc, n_slabs, d_k, order, groups) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  ++ctx.launches;
}

}  // namespace

int decode_n_psi(int d_k, int layout, int order, int groups) {
  if (order == 1) return d_k;
  const int m = d_k / groups;
  return groups * (layout == KATA_LAYOUT_PACKED ? m * (m + 1) / 2 : m * m);
}

int decode_slabs(int n_psi) { return (n_psi + DEC_ROWS - 1) / DEC_ROWS; }

size_t decode_workspace_elems(int BH, int n_psi, int d_v) { return (size_t)BH * decode_slabs(n_psi) * (d_v + 1); }

void decode_step(const void* q, const void* k, const void* v, void* out, float* S, float* Z, float* part, int BH,
                 int d_k, int d_v, int dtype, int layout, int order, int groups, LaunchCtx& ctx) {
  const int n_psi = decode_n_psi(d_k, layout, order, groups);
#define KATA_DEC(T, DV) launch<T, DV>(q, k, v, out, S, Z, part, BH, d_k, n_psi, layout, order, groups, ctx)
  if (dtype == KATA_F32) {
    if (d_v == 64) KATA_DEC(float, 64); else if (d_v == 32) KATA_DEC(float, 32); else KATA_DEC(float, 16);
  } else {
    if (d_v == 64) KATA_DEC(__nv_bfloat16, 64); else if (d_v == 32) KATA_DEC(__nv_bfloat16, 32); else KATA_DEC(__nv_bfloat16, 16);
  }
#undef KATA_DEC
}

}  // namespace kata
