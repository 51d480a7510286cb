// Chunked-state KATA forward (Algorithm 1) and its scan form on plain fp32 FMAs.
//
// One CTA owns one head and one slice of the value columns; output columns are independent, so
// CTAs never exchange data.  The running state S[a,b,v] = sum_i k_hat_a k_hat_b v_v is symmetric in
// (a,b): only the upper block triangle is kept, spread over threads as BLK x BLK register blocks
// (thread <-> block pair (A,B), A <= B), with the normaliser state Z[a,b] = sum_i k_hat_a k_hat_b as
// one extra "value column".  Per chunk:
//   P = (Q_hat K_hat^T)^2 o M          from the d-dimensional dot product, squared
//   N = Psi(Q) S + P V,  D = Psi(Q) Z + P 1,  O = N / D      (chunk-output equations)
//   S += Psi(K)^T V,  Z += Psi(K)^T 1                         (chunk state update)
// The feature products q_a q_b, k_a k_b are formed in registers; Psi is never written anywhere.
//
// Scan form: the chunk axis is cut into groups.  Pass 1 reduces every group to its local state,
// the group states go through a log-depth (Hillis-Steele) inclusive scan in global memory, pass 3
// restarts every group from the prefix before it.  With one chunk per group this is the paper's
// chunk-state / cumulative / chunk-output pipeline and the prefix states can be exported.
#include "kata_common.cuh"

namespace kata {
namespace {

constexpr int NB = 16;                       // blocks per feature axis (d_k / BLK)
constexpr int NPAIR = NB * (NB + 1) / 2;     // 136 block pairs A <= B
constexpr int NTHR = 160;                    // 5 warps; threads >= NPAIR idle in the state phases
constexpr int NWARP = NTHR / 32;
constexpr int TS = 68;                       // row stride of the transposed q/k tiles
constexpr int C = kChunk;

template <int D, int DV> struct Cfg {
  static constexpr int BLK = D / NB;                        // 4, 2, 1 for d_k = 64, 32, 16
  static constexpr int VCAP = 128 / (BLK * BLK) > 32 ? 32 : 128 / (BLK * BLK);
  static constexpr int VS = DV < VCAP ? DV : VCAP;          // value columns per CTA
  static constexpr int NSLICE = DV / VS;
  static constexpr int NREG = BLK * BLK * (VS + 1);         // state floats per thread
  static constexpr int RS = D + 4;                          // row stride of the row-major q/k tiles
  static constexpr size_t STATE_ELEMS = (size_t)NSLICE * NREG * NTHR;   // per (b,h,group)
  static constexpr int SMEM_FLOATS = 2 * C * RS + 2 * D * TS + C * VS + C * (C + 1) +
                                     NWARP * C * (VS + 1) + C * (VS + 1);
};

// Sum NV per-lane values over the 32 lanes of a warp; every lane ends with the total of ONE of the
// NV values (index idx), lanes that share idx hold the same total.
template <int NV>
__device__ __forceinline__ float warp_reduce_scatter(float (&x)[NV], int lane, int& idx) {
  static_assert(NV == 8 || NV == 16 || NV == 32, "NV");
  idx = 0;
  int s = 16;
#pragma unroll
  for (int half = NV / 2; half >= 1; half >>= 1) {
    const bool upper = (lane & s) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float keep = upper ? x[i + half] : x[i];
      const float send = upper ? x[i] : x[i + half];
      x[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
    }
    if (upper) idx += half;
    s >>= 1;
  }
  float r = x[0];
#pragma unroll
  for (; s >= 1; s >>= 1) r += __shfl_xor_sync(0xffffffffu, r, s);
  return r;
}

template <typename T, int D, int DV>
__global__ void __launch_bounds__(NTHR) chunk_simt_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                           const T* __restrict__ v, T* __restrict__ out,
                                                           int Tlen, int n_chunks, int chunks_per_group,
                                                           int n_groups,
                                                           const float* __restrict__ init_state,
                                                           float* __restrict__ final_state, int write_out,
                                                           int groups, int init_first) {
  using G = Cfg<D, DV>;
  constexpr int BLK = G::BLK, VS = G::VS, RS = G::RS;
  extern __shared__ __align__(16) float smem[];
  float (*qs)[RS] = reinterpret_cast<float (*)[RS]>(smem);
  float (*ks)[RS] = reinterpret_cast<float (*)[RS]>(smem + C * RS);
  float (*qT)[TS] = reinterpret_cast<float (*)[TS]>(smem + 2 * C * RS);
  float (*kT)[TS] = reinterpret_cast<float (*)[TS]>(smem + 2 * C * RS + D * TS);
  float (*vs)[VS] = reinterpret_cast<float (*)[VS]>(smem + 2 * C * RS + 2 * D * TS);
  float (*P)[C + 1] = reinterpret_cast<float (*)[C + 1]>(smem + 2 * C * RS + 2 * D * TS + C * VS);
  float* Nw = smem + 2 * C * RS + 2 * D * TS + C * VS + C * (C + 1);        // [NWARP][C][VS+1]
  float (*Nin)[VS + 1] = reinterpret_cast<float (*)[VS + 1]>(Nw + NWARP * C * (VS + 1));

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int slice = blockIdx.x, grp = blockIdx.z;
  const size_t bh = blockIdx.y;

  // block pair owned by this thread
  int A = 0, Bq = 0;
  const bool active = tid < NPAIR;
  if (active) {
    int t = tid;
    while (t >= NB - A) { t -= NB - A; ++A; }
    Bq = A + t;
  }
  // blockwise PSD map: only pairs (a,b) of the same feature group carry state (NB / groups blocks per group)
  const bool same_group = (A / (NB / groups)) == (Bq / (NB / groups));
  float wgt[BLK][BLK];   // 2 above the diagonal, 1 on it, 0 below (and for idle threads and other groups)
#pragma unroll
  for (int i = 0; i < BLK; ++i)
#pragma unroll
    for (int j = 0; j < BLK; ++j) {
      const int a = A * BLK + i, b = Bq * BLK + j;
      wgt[i][j] = (!active || !same_group) ? 0.f : (a < b ? 2.f : (a == b ? 1.f : 0.f));
    }

  float S[BLK][BLK][VS];
  float Z[BLK][BLK];
  const size_t slot = (size_t)G::NREG * NTHR;
  // group grp starts from the state in slot grp - 1 (the prefix before it); with init_first the slots hold the
  // states the groups start from, slot 0 being the state before the first token
  const int src_grp = grp - 1 + init_first;
  if (init_state != nullptr && src_grp >= 0) {
    const float* src = init_state + ((bh * n_groups + src_grp) * G::NSLICE + slice) * slot + tid;
#pragma unroll
    for (int i = 0; i < BLK; ++i)
#pragma unroll
      for (int j = 0; j < BLK; ++j) {
#pragma unroll
        for (int c = 0; c < VS; ++c) S[i][j][c] = src[(size_t)((i * BLK + j) * (VS + 1) + c) * NTHR];
        Z[i][j] = src[(size_t)((i * BLK + j) * (VS + 1) + VS) * NTHR];
      }
  } else {
#pragma unroll
    for (int i = 0; i < BLK; ++i)
#pragma unroll
      for (int j = 0; j < BLK; ++j) {
#pragma unroll
        for (int c = 0; c < VS; ++c) S[i][j][c] = 0.f;
        Z[i][j] = 0.f;
      }
  }

  for (int idx = tid; idx < C * (C + 1); idx += NTHR) (&P[0][0])[idx] = 0.f;

  const T* qh = q + bh * (size_t)Tlen * D;
  const T* kh = k + bh * (size_t)Tlen * D;
  const T* vh = v + bh * (size_t)Tlen * DV + slice * VS;
  T* oh = out + bh * (size_t)Tlen * DV + slice * VS;

  const int c_begin = grp * chunks_per_group;
  const int c_end = min(n_chunks, c_begin + chunks_per_group);

  for (int c = c_begin; c < c_end; ++c) {
    const int t0 = c * C;
    __syncthreads();
    // ---- load the chunk (zero rows beyond T: padded keys carry a zero feature) ----
    for (int idx = tid; idx < C * D; idx += NTHR) {
      const int r = idx / D, a = idx % D;
      const bool ok = t0 + r < Tlen;
      qs[r][a] = (ok && write_out) ? to_f32(qh[(size_t)(t0 + r) * D + a]) : 0.f;
      ks[r][a] = ok ? to_f32(kh[(size_t)(t0 + r) * D + a]) : 0.f;
    }
    for (int idx = tid; idx < C * VS; idx += NTHR) {
      const int r = idx / VS, cc = idx % VS;
      vs[r][cc] = (t0 + r < Tlen) ? to_f32(vh[(size_t)(t0 + r) * DV + cc]) : 0.f;
    }
    __syncthreads();
    // ---- l2-normalise rows in place, keep transposed copies for the score tiles ----
    if (tid < 2 * C) {
      const int r = tid & (C - 1);
      float* row = (tid < C) ? qs[r] : ks[r];
      float (*tr)[TS] = (tid < C) ? qT : kT;
      float ss = 0.f;
#pragma unroll 8
      for (int a = 0; a < D; ++a) ss = fmaf(row[a], row[a], ss);
      const float sc = rsqrt_or_zero(ss);
#pragma unroll 8
      for (int a = 0; a < D; ++a) {
        const float x = row[a] * sc;
        row[a] = x;
        tr[a][r] = x;
      }
    }
    __syncthreads();

    if (write_out) {
      // ---- intra-chunk scores, one 4x4 tile per thread on or below the block diagonal ----
      if (active) {
        const int tb = Bq, ib = A;
        float s[4][4], w2[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) w2[i][j] = 0.f;
        const int mblk = D / groups;
        for (int gb = 0; gb < groups; ++gb) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
          for (int a = gb * mblk; a < (gb + 1) * mblk; ++a) {
            const float4 qa = *reinterpret_cast<const float4*>(&qT[a][tb * 4]);
            const float4 ka = *reinterpret_cast<const float4*>(&kT[a][ib * 4]);
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
            for (int j = 0; j < 4; ++j) w2[i][j] = fmaf(s[i][j], s[i][j], w2[i][j]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = tb * 4 + i, i2 = ib * 4 + j;
            P[t][i2] = (i2 <= t) ? w2[i][j] : 0.f;
          }
      }
      __syncthreads();
      // ---- N_intra = P V, D_intra = P 1 ----
      for (int item = tid; item < C * VS; item += NTHR) {
        const int t = item / VS, cc = item % VS;
        float acc = 0.f;
        for (int i2 = 0; i2 <= t; ++i2) acc = fmaf(P[t][i2], vs[i2][cc], acc);
        Nin[t][cc] = acc;
      }
      if (tid < C) {
        float acc = 0.f;
        for (int i2 = 0; i2 <= tid; ++i2) acc += P[tid][i2];
        Nin[tid][VS] = acc;
      }
      // ---- inter-chunk read: N += Psi(Q) S, D += Psi(Q) Z ----
      for (int t = 0; t < C; ++t) {
        float qa[BLK], qb[BLK];
#pragma unroll
        for (int i = 0; i < BLK; ++i) {
          qa[i] = qs[t][A * BLK + i];
          qb[i] = qs[t][Bq * BLK + i];
        }
        float x[VS];
#pragma unroll
        for (int cc = 0; cc < VS; ++cc) x[cc] = 0.f;
        float xz = 0.f;
#pragma unroll
        for (int i = 0; i < BLK; ++i)
#pragma unroll
          for (int j = 0; j < BLK; ++j) {
            const float g = wgt[i][j] * qa[i] * qb[j];
#pragma unroll
            for (int cc = 0; cc < VS; ++cc) x[cc] = fmaf(g, S[i][j][cc], x[cc]);
            xz = fmaf(g, Z[i][j], xz);
          }
        int idx;
        const float r = warp_reduce_scatter<VS>(x, lane, idx);
#pragma unroll
        for (int s2 = 16; s2 >= 1; s2 >>= 1) xz += __shfl_xor_sync(0xffffffffu, xz, s2);
        float* dst = Nw + ((size_t)warp * C + t) * (VS + 1);
        if ((lane & (32 / VS - 1)) == 0) dst[idx] = r;
        if (lane == 0) dst[VS] = xz;
      }
      __syncthreads();
      // ---- gate/normalise epilogue: o = N / D (0 where D = 0) ----
      for (int item = tid; item < C * VS; item += NTHR) {
        const int t = item / VS, cc = item % VS;
        if (t0 + t >= Tlen) continue;
        float n = Nin[t][cc], dsum = Nin[t][VS];
#pragma unroll
        for (int w = 0; w < NWARP; ++w) {
          n += Nw[((size_t)w * C + t) * (VS + 1) + cc];
          dsum += Nw[((size_t)w * C + t) * (VS + 1) + VS];
        }
        oh[(size_t)(t0 + t) * DV + cc] = from_f32<T>(dsum > 0.f ? n / dsum : 0.f);
      }
    }

    // ---- state update with this chunk's keys and values ----
    const bool need_update = (c + 1 < c_end) || (final_state != nullptr);
    if (need_update) {
      for (int t = 0; t < C; ++t) {
        float ka[BLK], kb[BLK];
#pragma unroll
        for (int i = 0; i < BLK; ++i) {
          ka[i] = ks[t][A * BLK + i];
          kb[i] = ks[t][Bq * BLK + i];
        }
        float vv[VS];
#pragma unroll
        for (int cc = 0; cc < VS; ++cc) vv[cc] = vs[t][cc];
#pragma unroll
        for (int i = 0; i < BLK; ++i)
#pragma unroll
          for (int j = 0; j < BLK; ++j) {
            const float f = ka[i] * kb[j];
#pragma unroll
            for (int cc = 0; cc < VS; ++cc) S[i][j][cc] = fmaf(f, vv[cc], S[i][j][cc]);
            Z[i][j] += f;
          }
      }
    }
  }

  if (final_state != nullptr) {
    float* dst = final_state + ((bh * n_groups + grp) * G::NSLICE + slice) * slot + tid;
#pragma unroll
    for (int i = 0; i < BLK; ++i)
#pragma unroll
      for (int j = 0; j < BLK; ++j) {
#pragma unroll
        for (int c = 0; c < VS; ++c) dst[(size_t)((i * BLK + j) * (VS + 1) + c) * NTHR] = S[i][j][c];
        dst[(size_t)((i * BLK + j) * (VS + 1) + VS) * NTHR] = Z[i][j];
      }
  }
}

// One round of the Hillis-Steele inclusive scan over the group axis of x[BH][G][E]:
// dst[g] = src[g] + (g >= stride ? src[g - stride] : 0), for the first g_used groups.
__global__ void scan_round_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t e4,
                                  int n_groups, int g_used, int stride) {
  const int bh = blockIdx.y;
  cudaGridDependencySynchronize();      // a programmatic dependent launch: resident while the kernel ahead drains
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < (size_t)g_used * e4;
       i += (size_t)gridDim.x * blockDim.x) {
    const int g = (int)(i / e4);
    const size_t e = i % e4;
    const size_t base = ((size_t)bh * n_groups + g) * e4 + e;
    float4 a = src[base];
    if (g >= stride) {
      const float4 b = src[base - (size_t)stride * e4];
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    dst[base] = a;
  }
}

// Exclusive-prefix chunk states in the public layouts, from the inclusive scan of per-chunk states.
template <int D, int DV>
__global__ void export_states_kernel(const float* __restrict__ incl, float* __restrict__ s_pre,
                                     float* __restrict__ z_pre, int n_chunks, int layout, int groups) {
  using G = Cfg<D, DV>;
  constexpr int BLK = G::BLK, VS = G::VS;
  const int c = blockIdx.x;
  const size_t bh = blockIdx.y;
  const int n_psi = groups * ((layout == KATA_LAYOUT_PACKED) ? (D / groups) * (D / groups + 1) / 2 : (D / groups) * (D / groups));
  const size_t slot = (size_t)G::NREG * NTHR;
  float* sp = s_pre + (bh * n_chunks + c) * (size_t)n_psi * DV;
  float* zp = z_pre + (bh * n_chunks + c) * (size_t)n_psi;
  for (int item = threadIdx.x; item < n_psi * (DV + 1); item += blockDim.x) {
    const int row = item / (DV + 1), col = item % (DV + 1);
    int a, b;
    float scale = 1.f;
    {
      // rows of the g feature blocks follow one another; inside a block of m = D / g features the layout is
      // the direct m x m or the packed upper triangle
      const int m = D / groups;
      const int per = (layout == KATA_LAYOUT_PACKED) ? m * (m + 1) / 2 : m * m;
      const int gb = row / per;
      int r = row - gb * per;
      if (layout == KATA_LAYOUT_PACKED) {
        a = 0;
        while (r >= m - a) { r -= m - a; ++a; }
        b = a + r;
        if (a != b) scale = 1.41421356237309504880f;
      } else {
        a = r / m;
        b = r % m;
      }
      a += gb * m;
      b += gb * m;
    }
    float val = 0.f;
    if (c > 0) {
      const int lo = min(a, b), hi = max(a, b);
      const int Ab = lo / BLK, Bb = hi / BLK, i = lo % BLK, j = hi % BLK;
      const int tid = Ab * NB - Ab * (Ab - 1) / 2 + (Bb - Ab);
      const int slice = (col < DV) ? col / VS : 0;
      const int cc = (col < DV) ? col % VS : VS;
      const float* src = incl + ((bh * n_chunks + (c - 1)) * G::NSLICE + slice) * slot;
      val = scale * src[(size_t)((i * BLK + j) * (VS + 1) + cc) * NTHR + tid];
    }
    if (col < DV) sp[(size_t)row * DV + col] = val;
    else zp[row] = val;
  }
}

// State after the last token in the public layouts, from the internal state [BH][NSLICE][slot] of a
// whole-sequence pass.
template <int D, int DV>
__global__ void export_final_kernel(const float* __restrict__ fin, float* __restrict__ s_out, float* __restrict__ z_out,
                                    int layout, int groups) {
  using G = Cfg<D, DV>;
  constexpr int BLK = G::BLK, VS = G::VS;
  const size_t bh = blockIdx.y;
  const int n_psi = groups * ((layout == KATA_LAYOUT_PACKED) ? (D / groups) * (D / groups + 1) / 2 : (D / groups) * (D / groups));
  const size_t slot = (size_t)G::NREG * NTHR;
  float* sp = s_out + bh * (size_t)n_psi * DV;
  float* zp = z_out + bh * (size_t)n_psi;
  for (int item = blockIdx.x * blockDim.x + threadIdx.x; item < n_psi * (DV + 1); item += gridDim.x * blockDim.x) {
    const int row = item / (DV + 1), col = item % (DV + 1);
    int a, b;
    float scale = 1.f;
    {
      // rows of the g feature blocks follow one another; inside a block of m = D / g features the layout is
      // the direct m x m or the packed upper triangle
      const int m = D / groups;
      const int per = (layout == KATA_LAYOUT_PACKED) ? m * (m + 1) / 2 : m * m;
      const int gb = row / per;
      int r = row - gb * per;
      if (layout == KATA_LAYOUT_PACKED) {
        a = 0;
        while (r >= m - a) { r -= m - a; ++a; }
        b = a + r;
        if (a != b) scale = 1.41421356237309504880f;
      } else {
        a = r / m;
        b = r % m;
      }
      a += gb * m;
      b += gb * m;
    }
    const int lo = min(a, b), hi = max(a, b);
    const int Ab = lo / BLK, Bb = hi / BLK, i = lo % BLK, j = hi % BLK;
    const int tid = Ab * NB - Ab * (Ab - 1) / 2 + (Bb - Ab);
    const int slice = (col < DV) ? col / VS : 0;
    const int cc = (col < DV) ? col % VS : VS;
    const float* src = fin + (bh * G::NSLICE + slice) * slot;
    const float val = scale * src[(size_t)((i * BLK + j) * (VS + 1) + cc) * NTHR + tid];
    if (col < DV) sp[(size_t)row * DV + col] = val;
    else zp[row] = val;
  }
}

// The state before the first token, from the public layouts to the internal state [BH][NSLICE][slot] of a
// whole-sequence pass (the inverse of export_final_kernel).
template <int D, int DV>
__global__ void import_initial_kernel(const float* __restrict__ s_in, const float* __restrict__ z_in,
                                      float* __restrict__ dst, int layout, int groups) {
  using G = Cfg<D, DV>;
  constexpr int BLK = G::BLK, VS = G::VS;
  const size_t bh = blockIdx.y;
  const int m = D / groups;
  const bool packed = layout == KATA_LAYOUT_PACKED;
  const int per = packed ? m * (m + 1) / 2 : m * m;
  const int n_psi = groups * per;
  const size_t slot = (size_t)G::NREG * NTHR;
  const float* sp = s_in + bh * (size_t)n_psi * DV;
  const float* zp = z_in + bh * (size_t)n_psi;
  const int total = G::NSLICE * G::NREG * NTHR;
  for (int item = blockIdx.x * blockDim.x + threadIdx.x; item < total; item += gridDim.x * blockDim.x) {
    const int tid = item % NTHR;
    const int reg = (item / NTHR) % G::NREG;
    const int slice = item / (NTHR * G::NREG);
    const int cc = reg % (VS + 1), ij = reg / (VS + 1), i = ij / BLK, j = ij % BLK;
    float val = 0.f;
    if (tid < NPAIR) {
      int A = 0, t = tid;
      while (t >= NB - A) { t -= NB - A; ++A; }
      const int Bq = A + t;
      const int a = A * BLK + i, b = Bq * BLK + j;
      const int lo = min(a, b), hi = max(a, b);
      const int gb = lo / m;
      if (hi / m == gb) {
        const int la = lo - gb * m, lb = hi - gb * m;
        const int row = gb * per + (packed ? la * m - la * (la - 1) / 2 + (lb - la) : la * m + lb);
        const float scale = (packed && la != lb) ? 0.70710678118654752440f : 1.f;
        val = scale * (cc < VS ? sp[(size_t)row * DV + slice * VS + cc] : zp[row]);
      }
    }
    dst[(bh * G::NSLICE + slice) * slot + (size_t)reg * NTHR + tid] = val;
  }
}

template <typename T, int D, int DV>
void run(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, const float* s_init, const float* z_init,
         float* s_pre, float* z_pre,
         int state_layout, LaunchCtx& ctx) {
  using G = Cfg<D, DV>;
  auto kern = chunk_simt_kernel<T, D, DV>;
  constexpr size_t smem = sizeof(float) * G::SMEM_FLOATS;
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
    // whole sequence in one pass; with s_init/z_init it starts from that state, with s_pre/z_pre the state after
    // the last token is exported (both through the one internal state per head in the workspace)
    float* fin = (s_pre != nullptr) ? ws : nullptr;
    const float* ini = (s_init != nullptr) ? ws : nullptr;
    if (ini != nullptr) {
      import_initial_kernel<D, DV><<<dim3(16, BH), 256, 0, ctx.stream>>>(s_init, z_init, ws, state_layout, p.groups);
      note_launch(ctx);
    }
    kern<<<dim3(G::NSLICE, BH, 1), NTHR, smem, ctx.stream>>>(q, k, v, o, p.T, plan.n_chunks, plan.n_chunks,
                                                            1, ini, fin, 1, p.groups, 1);
    note_launch(ctx);
    if (fin != nullptr) {
      export_final_kernel<D, DV><<<dim3(16, BH), 256, 0, ctx.stream>>>(fin, s_pre, z_pre, state_layout, p.groups);
      note_launch(ctx);
    }
    return;
  }
  const int NG = plan.n_groups;
  const size_t E = G::STATE_ELEMS;
  float* bufA = ws;
  float* bufB = ws + (size_t)BH * NG * E;
  const float* incl = bufA;
  if (NG > 1) {
    // pass 1: local states of all groups but the last (its state is never read)
    kern<<<dim3(G::NSLICE, BH, NG - 1), NTHR, smem, ctx.stream>>>(q, k, v, o, p.T, plan.n_chunks,
                                                                 plan.chunks_per_group, NG, nullptr, bufA, 0, p.groups, 0);
    note_launch(ctx);
    // pass 2: inclusive scan over the first NG-1 group states, ceil(log2(NG-1)) rounds
    incl = scan_group_states(bufA, bufB, BH, NG, NG - 1, E, ctx);
  }
  // pass 3: every group restarts from the prefix before it
  kern<<<dim3(G::NSLICE, BH, NG), NTHR, smem, ctx.stream>>>(q, k, v, o, p.T, plan.n_chunks,
                                                           plan.chunks_per_group, NG, incl, nullptr, 1, p.groups, 0);
  note_launch(ctx);
  if (s_pre != nullptr && z_pre != nullptr) {
    export_states_kernel<D, DV><<<dim3(plan.n_chunks, BH), 256, 0, ctx.stream>>>(incl, s_pre, z_pre,
                                                                               plan.n_chunks, state_layout, p.groups);
    note_launch(ctx);
  }
}

template <typename T, int D>
void run_dv(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, const float* s_init, const float* z_init,
            float* s_pre, float* z_pre,
            int layout, LaunchCtx& ctx) {
  switch (p.d_v) {
    case 16: run<T, D, 16>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, layout, ctx); break;
    case 32: run<T, D, 32>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, layout, ctx); break;
    default: run<T, D, 64>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, layout, ctx); break;
  }
}

template <typename T>
void run_d(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, const float* s_init, const float* z_init,
           float* s_pre, float* z_pre,
           int layout, LaunchCtx& ctx) {
  switch (p.d_k) {
    case 16: run_dv<T, 16>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, layout, ctx); break;
    case 32: run_dv<T, 32>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, layout, ctx); break;
    default: run_dv<T, 64>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, layout, ctx); break;
  }
}

template <int D> size_t elems_dv(int d_v) {
  switch (d_v) {
    case 16: return Cfg<D, 16>::STATE_ELEMS;
    case 32: return Cfg<D, 32>::STATE_ELEMS;
    default: return Cfg<D, 64>::STATE_ELEMS;
  }
}

}  // namespace

const float* scan_group_states(float* bufA, float* bufB, int BH, int n_groups, int g_used, size_t E,
                               LaunchCtx& ctx) {
  float* src = bufA;
  float* dst = bufB;
  const size_t e4 = E / 4;
  for (int stride = 1; stride < g_used; stride <<= 1) {
    const size_t work = (size_t)g_used * e4;
    const int blocks = (int)((work + 255) / 256 > 4096 ? 4096 : (work + 255) / 256);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks, BH);
    cfg.blockDim = dim3(256);
    cfg.stream = ctx.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, scan_round_kernel, reinterpret_cast<const float4*>(src), reinterpret_cast<float4*>(dst),
                           e4, n_groups, g_used, stride) != cudaSuccess) {
      cudaGetLastError();
      ctx.status = KATA_ERR_CUDA;
      return src;
    }
    ++ctx.launches;
    float* t = src; src = dst; dst = t;
  }
  return src;
}

int simt_chunked_slices(int d_k, int d_v) {
  const int blk = d_k / NB;
  int vcap = 128 / (blk * blk);
  if (vcap > 32) vcap = 32;
  const int vs = d_v < vcap ? d_v : vcap;
  return d_v / vs;
}

size_t simt_chunked_state_elems(int d_k, int d_v) {
  switch (d_k) {
    case 16: return elems_dv<16>(d_v);
    case 32: return elems_dv<32>(d_v);
    default: return elems_dv<64>(d_v);
  }
}

void simt_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, const float* s_init,
                  const float* z_init, float* s_pre, float* z_pre, int state_layout, LaunchCtx& ctx) {
  if (p.dtype == KATA_F32) run_d<float>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, state_layout, ctx);
  else run_d<__nv_bfloat16>(p, plan, use_scan, ws, s_init, z_init, s_pre, z_pre, state_layout, ctx);
}

}  // namespace kata
