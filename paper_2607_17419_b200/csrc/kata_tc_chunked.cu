// Chunked-state KATA forward on the Blackwell tensor cores (tcgen05 + TMEM), bf16, d_k = d_v = 64, C = 64.
//
// Formulation.  With k' = k / ||k|| the state is S[a,b,v] = sum_i k'_a k'_b v_v (symmetric in a,b) and the
// normaliser state Z[a,b] = sum_i k'_a k'_b.  One CTA owns one head and 8 value columns; output columns
// are independent, so CTAs never exchange data.  The d_k^2-wide feature GEMMs of the chunk equations are
// re-associated so that no feature matrix Psi is ever built:
//
//   state update   S[(b,v), a] += sum_t W[(b,v), t] * k[t, a],   W[(b,v), t] = k[t,b] v[t,v] / ||k_t||^2
//                  (tcgen05 kind::f16: A = W from shared memory, built on the fly; B = the TMA-loaded
//                   key tile used MN-major; D = fp32 accumulators resident in TMEM for the whole head)
//   inter-chunk    Y[(b,v), t] = sum_a S[(b,v), a] * q[t, a]     (tcgen05 kind::tf32: A = the fp32
//   read           accumulators of the update, read straight from TMEM; B = the query tile as tf32)
//                  N_inter[t, v] = sum_b q[t,b] * Y[(b,v), t]    (fp32 FMAs on the TMEM read-back)
//   normaliser     the same two steps with the "ones" value column: rows (b) of a fifth tile hold Z
//   intra-chunk    P = (Q K^T)^2 / ||k||^2 o M from one d-dimensional bf16 MMA, squared in fp32;
//                  N_intra = P V, D_intra = P 1 on fp32 FMAs
//   epilogue       O = (N_inter + N_intra) / (D_inter + D_intra)   (gate + normalise), bf16 store
//
// The query norm is a common factor of numerator and denominator and is never applied.  Rows (b,v) of a
// 128-row MMA tile are b = 16*tile + row/8, v = row%8; four tiles cover b = 0..63, the fifth holds Z.
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 operand builders
// (norms, tf32 query tile, transposes, W tiles), warps 6-9 TMEM readers (Y reduction, scores, epilogue).
// All hand-offs go through mbarriers with bounded waits; on a timeout the CTA records
// KATA_ERR_DEVICE_TIMEOUT in *device_status, drains and returns.
#include <cuda.h>

#include "kata_common.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int C = kChunk;        // 64 tokens per chunk
constexpr int D = 64;            // d_k = d_v
constexpr int VS = 8;            // value columns per CTA
constexpr int NSLICE = D / VS;   // CTAs per head
constexpr int NT = 5;            // MMA tiles per chunk: 4 state tiles + the normaliser tile
constexpr int NTHREADS = 320;

// TMEM columns (fp32 accumulators, 128 lanes each)
constexpr uint32_t COL_S = 0;      // 5 tiles x 64 columns: S tiles 0..3, Z tile 4
constexpr uint32_t COL_Y = 320;    // 2 x 64: ring of read results
constexpr uint32_t COL_P = 448;    // 64: intra-chunk scores (rows 0..63 valid)
constexpr uint32_t TMEM_COLS = 512;

// shared memory map (bytes from a 1024-aligned base)
constexpr uint32_t OFF_QK = 0;                    // 2 stages x (Q tile 8 KB, K tile 8 KB), TMA, 128B swizzle
constexpr uint32_t OFF_V = 32768;                 // 2 stages x 64 x 8 bf16
constexpr uint32_t OFF_QF = 34816;                // 2 x 16 KB: query tile as tf32, K-major, 128B swizzle, 2 atoms
constexpr uint32_t OFF_W = 67584;                 // 2 x 16 KB: W tile, bf16, K-major, 128B swizzle
constexpr uint32_t OFF_KT = 100352;               // kT[b][t] fp32 (builders only)
constexpr uint32_t OFF_VT = 116736;               // vT[v][t] = v / ||k||^2, fp32 (builders only)
constexpr uint32_t OFF_QT = 118784;               // 2 x qT[b][t] fp32 (readers)
constexpr uint32_t OFF_VS = 151552;               // 2 x vS[t][v] fp32 raw values (readers)
constexpr uint32_t OFF_R2 = 155648;               // 2 x r2[t] = 1/||k_t||^2
constexpr uint32_t OFF_RED = 156160;              // red[128][68] fp32 cross-lane reduction scratch
constexpr uint32_t RED_STRIDE = 68;
constexpr uint32_t OFF_NINTRA = 190976;           // [64][9]
constexpr uint32_t OFF_NINTER = 193280;           // [64][9]
constexpr uint32_t OFF_BAR = 195584;              // mbarriers
constexpr uint32_t SMEM_BYTES = 195584 + 256;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;  // slack for the 1024-byte alignment

enum {
  BAR_FULL = 0,     // [2] TMA landed
  BAR_EMPTY = 2,    // [2] stage free (128 builders + MMA commit)
  BAR_PREP = 4,     // [2] operands of the chunk built (128 builders)
  BAR_WFULL = 6,    // [2] W tile built
  BAR_WEMPTY = 8,   // [2] W tile consumed by the MMA
  BAR_YFULL = 10,   // [2] read result in TMEM
  BAR_YEMPTY = 12,  // [2] read result drained (128 readers)
  BAR_PFULL = 14,
  BAR_PEMPTY = 15,
  BAR_U = 16,       // [5] update of state tile i complete
  BAR_COUNT = 21
};

struct Shared {
  unsigned char* base;
  __device__ unsigned char* qtile(int s) const { return base + OFF_QK + s * 16384; }
  __device__ unsigned char* ktile(int s) const { return base + OFF_QK + s * 16384 + 8192; }
  __device__ unsigned char* vtile(int s) const { return base + OFF_V + s * 1024; }
  __device__ unsigned char* qf(int s) const { return base + OFF_QF + s * 16384; }
  __device__ unsigned char* w(int s) const { return base + OFF_W + s * 16384; }
  __device__ float* kT() const { return reinterpret_cast<float*>(base + OFF_KT); }
  __device__ float* vT() const { return reinterpret_cast<float*>(base + OFF_VT); }
  __device__ float* qT(int s) const { return reinterpret_cast<float*>(base + OFF_QT + s * 16384); }
  __device__ float* vS(int s) const { return reinterpret_cast<float*>(base + OFF_VS + s * 2048); }
  __device__ float* r2(int s) const { return reinterpret_cast<float*>(base + OFF_R2 + s * 256); }
  __device__ float* red() const { return reinterpret_cast<float*>(base + OFF_RED); }
  __device__ float* nintra() const { return reinterpret_cast<float*>(base + OFF_NINTRA); }
  __device__ float* ninter() const { return reinterpret_cast<float*>(base + OFF_NINTER); }
  __device__ uint64_t* bar(int i) const { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; }
};

__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

// Bounded wait that also gives up as soon as another role has flagged an abort.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(NTHREADS, 1)
tc_chunk_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ out, int Tlen, int n_chunks,
                int* __restrict__ device_status) {
  extern __shared__ unsigned char smem_raw[];
  Shared sm;
  sm.base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slice = blockIdx.x;
  const int bh = blockIdx.y;

  if (tid == 0) {
    abort_s = 0;
    mbar_init(sm.bar(BAR_FULL + 0), 1);
    mbar_init(sm.bar(BAR_FULL + 1), 1);
    mbar_init(sm.bar(BAR_EMPTY + 0), 129);
    mbar_init(sm.bar(BAR_EMPTY + 1), 129);
    for (int i = 0; i < 2; ++i) {
      mbar_init(sm.bar(BAR_PREP + i), 128);
      mbar_init(sm.bar(BAR_WFULL + i), 128);
      mbar_init(sm.bar(BAR_WEMPTY + i), 1);
      mbar_init(sm.bar(BAR_YFULL + i), 1);
      mbar_init(sm.bar(BAR_YEMPTY + i), 128);
    }
    mbar_init(sm.bar(BAR_PFULL), 1);
    mbar_init(sm.bar(BAR_PEMPTY), 128);
    for (int i = 0; i < NT; ++i) mbar_init(sm.bar(BAR_U + i), 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  // zero the state accumulators (readers own the TMEM lanes)
  if (warp >= 6) {
    const uint32_t q4 = warp & 3;
    uint32_t z[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) z[j] = 0u;
    for (int cblk = 0; cblk < (NT * 64) / 32; ++cblk) tmem_st32(tmem_addr(tb, q4 * 32, COL_S + cblk * 32), z);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  bool ok = true;

  if (warp == 0) {
    // =========================== TMA producer ===========================
    if (lane == 0) {
      for (int c = 0; c < n_chunks && ok; ++c) {
        const int s = c & 1;
        ok = wait_or_abort(sm.bar(BAR_EMPTY + s), ((c >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(sm.bar(BAR_FULL + s), 8192 + 8192 + 1024);
        tma_load_3d(sm.qtile(s), &tmQ, sm.bar(BAR_FULL + s), 0, c * C, bh);
        tma_load_3d(sm.ktile(s), &tmK, sm.bar(BAR_FULL + s), 0, c * C, bh);
        tma_load_3d(sm.vtile(s), &tmV, sm.bar(BAR_FULL + s), slice * VS, c * C, bh);
      }
    }
  } else if (warp == 1) {
    // =========================== MMA issuer ===========================
    if (lane == 0) {
      const uint32_t id_read = instr_desc(kFmtTF32, kFmtTF32, 0, 0, 128, 64);    // A tmem, B K-major
      const uint32_t id_qk = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 64);      // both K-major
      const uint32_t id_upd = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 64);     // B MN-major
      for (int c = 0; c < n_chunks && ok; ++c) {
        const int s = c & 1;
        const uint32_t ph = (c >> 1) & 1;
        ok = wait_or_abort(sm.bar(BAR_FULL + s), ph, abort_flag) &&
             wait_or_abort(sm.bar(BAR_PREP + s), ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // ---- inter-chunk reads Y_i = S_i * Q^T (tf32, A from TMEM) ----
        for (int i = 0; i < NT && ok; ++i) {
          const int g = c * NT + i;
          ok = wait_or_abort(sm.bar(BAR_YEMPTY + (g & 1)), ((g >> 1) & 1) ^ 1, abort_flag);
          if (ok && c > 0) ok = wait_or_abort(sm.bar(BAR_U + i), (c - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t qf = smem_u32(sm.qf(s));
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_tf32_ts(tb + COL_Y + (g & 1) * 64, tb + COL_S + i * 64 + ks * 8,
                        smem_desc(qf + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024, kSwizzle128B), id_read, ks > 0);
          mma_commit(sm.bar(BAR_YFULL + (g & 1)));
        }
        if (!ok) break;
        // ---- intra-chunk scores [Q;K] K^T (rows 0..63 used) ----
        ok = wait_or_abort(sm.bar(BAR_PEMPTY), (c & 1) ^ 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        {
          const uint32_t qa = smem_u32(sm.qtile(s)), ka = smem_u32(sm.ktile(s));
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            mma_f16_ss(tb + COL_P, smem_desc(qa + ks * 32, 16, 1024, kSwizzle128B),
                       smem_desc(ka + ks * 32, 16, 1024, kSwizzle128B), id_qk, ks > 0);
          mma_commit(sm.bar(BAR_PFULL));
        }
        // ---- state updates S_i += W_i * K ----
        for (int i = 0; i < NT && ok; ++i) {
          const int g = c * NT + i;
          ok = wait_or_abort(sm.bar(BAR_WFULL + (g & 1)), (g >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t wa = smem_u32(sm.w(g & 1)), ka = smem_u32(sm.ktile(s));
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            mma_f16_ss(tb + COL_S + i * 64, smem_desc(wa + ks * 32, 16, 1024, kSwizzle128B),
                       smem_desc(ka + ks * 2048, 8192, 1024, kSwizzle128B), id_upd, 1u);
          mma_commit(sm.bar(BAR_WEMPTY + (g & 1)));
          mma_commit(sm.bar(BAR_U + i));
        }
        if (!ok) break;
        mma_commit(sm.bar(BAR_EMPTY + s));
      }
    }
  } else if (warp < 6) {
    // =========================== operand builders (128 threads) ===========================
    const int ta = tid - 64;
    const int row = ta >> 1, hf = ta & 1;          // prep mapping: two threads per token row
    float* kT = sm.kT();
    float* vT = sm.vT();
    for (int c = 0; c < n_chunks && ok; ++c) {
      const int s = c & 1;
      ok = wait_or_abort(sm.bar(BAR_FULL + s), (c >> 1) & 1, abort_flag);
      if (!ok) break;
      group_sync(2);   // every builder is done with kT / vT of the previous chunk
      float* qT = sm.qT(s);
      float* r2 = sm.r2(s);
      // ---- phase 1: key norms, kT, tf32 query tile, qT ----
      {
        const unsigned char* kt = sm.ktile(s);
        const unsigned char* qt = sm.qtile(s);
        unsigned char* qf = sm.qf(s) + hf * 8192;
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int chunk = hf * 4 + j;
          const uint4 kraw = *reinterpret_cast<const uint4*>(kt + sw128_offset(row, chunk));
          const uint4 qraw = *reinterpret_cast<const uint4*>(qt + sw128_offset(row, chunk));
          const uint32_t kw[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
          const uint32_t qw[4] = {qraw.x, qraw.y, qraw.z, qraw.w};
          float kf[8], qv[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            kf[2 * e] = __uint_as_float(kw[e] << 16);
            kf[2 * e + 1] = __uint_as_float(kw[e] & 0xFFFF0000u);
            qv[2 * e] = __uint_as_float(qw[e] << 16);
            qv[2 * e + 1] = __uint_as_float(qw[e] & 0xFFFF0000u);
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            ss = fmaf(kf[e], kf[e], ss);
            kT[(chunk * 8 + e) * C + row] = kf[e];
            qT[(chunk * 8 + e) * C + row] = qv[e];
          }
          // tf32 query tile: 32 fp32 per 128-byte row, this thread's half-row is atom `hf`
          *reinterpret_cast<float4*>(qf + sw128_offset(row, 2 * j)) = make_float4(qv[0], qv[1], qv[2], qv[3]);
          *reinterpret_cast<float4*>(qf + sw128_offset(row, 2 * j + 1)) = make_float4(qv[4], qv[5], qv[6], qv[7]);
        }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        if (hf == 0) r2[row] = inv_or_zero(ss);
      }
      group_sync(2);
      // ---- phase 2: values: raw copy for the readers, scaled transposed copy for the W tiles ----
      if (ta < C) {
        const uint4 vraw = *reinterpret_cast<const uint4*>(sm.vtile(s) + ta * 16);
        const uint32_t vw[4] = {vraw.x, vraw.y, vraw.z, vraw.w};
        const float rr = r2[ta];
        float* vS = sm.vS(s);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = __uint_as_float(vw[e] << 16), hi = __uint_as_float(vw[e] & 0xFFFF0000u);
          vS[ta * VS + 2 * e] = lo;
          vS[ta * VS + 2 * e + 1] = hi;
          vT[(2 * e) * C + ta] = lo * rr;
          vT[(2 * e + 1) * C + ta] = hi * rr;
        }
      }
      fence_async_smem();
      group_sync(2);
      mbar_arrive(sm.bar(BAR_PREP + s));
      mbar_arrive(sm.bar(BAR_EMPTY + s));     // done with the raw tiles (the MMA adds its own arrival)
      // ---- W tiles: row ta <-> (b = 16 i + ta/8, v = ta%8); fifth tile: rows < 64 hold k[t,b]/||k||^2 ----
      for (int i = 0; i < NT && ok; ++i) {
        const int g = c * NT + i;
        ok = wait_or_abort(sm.bar(BAR_WEMPTY + (g & 1)), ((g >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        unsigned char* wt = sm.w(g & 1);
        const float* krow = kT + ((i < 4) ? (16 * i + (ta >> 3)) : (ta & 63)) * C;
        const float* vrow = (i < 4) ? (vT + (ta & 7) * C) : r2;
        const bool zero = (i == 4) && (ta >= 64);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float4 k0 = *reinterpret_cast<const float4*>(krow + 8 * j);
          const float4 k1 = *reinterpret_cast<const float4*>(krow + 8 * j + 4);
          const float4 v0 = *reinterpret_cast<const float4*>(vrow + 8 * j);
          const float4 v1 = *reinterpret_cast<const float4*>(vrow + 8 * j + 4);
          uint4 pk;
          pk.x = pack_bf16(k0.x * v0.x, k0.y * v0.y);
          pk.y = pack_bf16(k0.z * v0.z, k0.w * v0.w);
          pk.z = pack_bf16(k1.x * v1.x, k1.y * v1.y);
          pk.w = pack_bf16(k1.z * v1.z, k1.w * v1.w);
          if (zero) pk = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(wt + sw128_offset(ta, j)) = pk;
        }
        fence_async_smem();
        mbar_arrive(sm.bar(BAR_WFULL + (g & 1)));
      }
    }
  } else {
    // =========================== TMEM readers (128 threads) ===========================
    const int tr = tid - 192;                  // 0..127
    const uint32_t q4 = warp & 3;              // TMEM lane quadrant this warp may access
    const int rowl = q4 * 32 + lane;           // tile row (= TMEM lane) of this thread
    float* red = sm.red();
    float* nintra = sm.nintra();
    float* ninter = sm.ninter();
    __nv_bfloat16* oh = out + (size_t)bh * Tlen * D + slice * VS;
    for (int c = 0; c < n_chunks && ok; ++c) {
      const int s = c & 1;
      ok = wait_or_abort(sm.bar(BAR_PREP + s), (c >> 1) & 1, abort_flag);
      if (!ok) break;
      const float* qT = sm.qT(s);
      const float* vS = sm.vS(s);
      const float* r2 = sm.r2(s);
      float acc[C];
#pragma unroll
      for (int t = 0; t < C; ++t) acc[t] = 0.f;
      for (int i = 0; i < NT && ok; ++i) {
        const int g = c * NT + i;
        ok = wait_or_abort(sm.bar(BAR_YFULL + (g & 1)), (g >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (i == 4) {
          // the four state tiles are in acc: reduce over b within the CTA -> ninter[t][v]
#pragma unroll
          for (int t4 = 0; t4 < C; t4 += 4)
            *reinterpret_cast<float4*>(red + rowl * RED_STRIDE + t4) =
                make_float4(acc[t4], acc[t4 + 1], acc[t4 + 2], acc[t4 + 3]);
          group_sync(3);
          {
            const int t = tr & 63, vh = tr >> 6;
#pragma unroll
            for (int vv = 0; vv < 4; ++vv) {
              const int v = vh * 4 + vv;
              float sum = 0.f;
#pragma unroll
              for (int bl = 0; bl < 16; ++bl) sum += red[(bl * 8 + v) * RED_STRIDE + t];
              ninter[t * 9 + v] = sum;
            }
          }
          group_sync(3);
#pragma unroll
          for (int t = 0; t < C; ++t) acc[t] = 0.f;
        }
        const int b = (i < 4) ? (16 * i + (rowl >> 3)) : (rowl & 63);
        const float* qrow = qT + b * C;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t y[32];
          tmem_ld32(tmem_addr(tb, q4 * 32, COL_Y + (g & 1) * 64 + half * 32), y);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 qq = *reinterpret_cast<const float4*>(qrow + half * 32 + j);
            acc[half * 32 + j] = fmaf(qq.x, __uint_as_float(y[j]), acc[half * 32 + j]);
            acc[half * 32 + j + 1] = fmaf(qq.y, __uint_as_float(y[j + 1]), acc[half * 32 + j + 1]);
            acc[half * 32 + j + 2] = fmaf(qq.z, __uint_as_float(y[j + 2]), acc[half * 32 + j + 2]);
            acc[half * 32 + j + 3] = fmaf(qq.w, __uint_as_float(y[j + 3]), acc[half * 32 + j + 3]);
          }
        }
        tc_fence_before();
        mbar_arrive(sm.bar(BAR_YEMPTY + (g & 1)));
      }
      if (!ok) break;
      // normaliser tile: rows 0..63 hold b, reduce over them -> ninter[t][8]
      if (rowl < 64) {
#pragma unroll
        for (int t4 = 0; t4 < C; t4 += 4)
          *reinterpret_cast<float4*>(red + rowl * RED_STRIDE + t4) =
              make_float4(acc[t4], acc[t4 + 1], acc[t4 + 2], acc[t4 + 3]);
      }
      group_sync(3);
      if (tr < C) {
        float sum = 0.f;
#pragma unroll 16
        for (int r = 0; r < 64; ++r) sum += red[r * RED_STRIDE + tr];
        ninter[tr * 9 + 8] = sum;
      }
      // ---- intra-chunk: P = s^2 / ||k||^2 (causal), N_intra = P V, D_intra = P 1 ----
      ok = wait_or_abort(sm.bar(BAR_PFULL), c & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if (rowl < 64) {
        float nacc[VS];
#pragma unroll
        for (int v = 0; v < VS; ++v) nacc[v] = 0.f;
        float dacc = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t sc[32];
          tmem_ld32(tmem_addr(tb, q4 * 32, COL_P + half * 32), sc);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int i2 = half * 32 + j;
            const float sv = __uint_as_float(sc[j]);
            const float w = (i2 <= rowl) ? sv * sv * r2[i2] : 0.f;
            dacc += w;
            const float4 va = *reinterpret_cast<const float4*>(vS + i2 * VS);
            const float4 vb = *reinterpret_cast<const float4*>(vS + i2 * VS + 4);
            nacc[0] = fmaf(w, va.x, nacc[0]);
            nacc[1] = fmaf(w, va.y, nacc[1]);
            nacc[2] = fmaf(w, va.z, nacc[2]);
            nacc[3] = fmaf(w, va.w, nacc[3]);
            nacc[4] = fmaf(w, vb.x, nacc[4]);
            nacc[5] = fmaf(w, vb.y, nacc[5]);
            nacc[6] = fmaf(w, vb.z, nacc[6]);
            nacc[7] = fmaf(w, vb.w, nacc[7]);
          }
        }
#pragma unroll
        for (int v = 0; v < VS; ++v) nintra[rowl * 9 + v] = nacc[v];
        nintra[rowl * 9 + 8] = dacc;
      } else {
        // lanes 64..127 of the score tile are not used; still order the TMEM access for the arrive below
      }
      tc_fence_before();
      mbar_arrive(sm.bar(BAR_PEMPTY));
      group_sync(3);
      // ---- gate + normalise epilogue ----
      {
        const int t = tr >> 1, vq = (tr & 1) * 4;
        const int tg = c * C + t;
        if (tg < Tlen) {
          const float den = ninter[t * 9 + 8] + nintra[t * 9 + 8];
          const float inv = den > 0.f ? 1.f / den : 0.f;
          float o[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) o[e] = (ninter[t * 9 + vq + e] + nintra[t * 9 + vq + e]) * inv;
          uint2 pk;
          pk.x = pack_bf16(o[0], o[1]);
          pk.y = pack_bf16(o[2], o[3]);
          *reinterpret_cast<uint2*>(oh + (size_t)tg * D + vq) = pk;
        }
      }
      group_sync(3);   // ninter / nintra / red are rewritten in the next chunk
    }
  }

  // ---------------- teardown ----------------
  if (!ok && device_status != nullptr) atomicExch(device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1 && lane == 0) {
    // make sure no MMA is still in flight before TMEM is released
    mbar_init(sm.bar(BAR_COUNT), 1);
    fence_mbar_init();
    mma_commit(sm.bar(BAR_COUNT));
    mbar_wait(sm.bar(BAR_COUNT), 0);
  }
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// [BH][T][64] bf16 tensor, box = `box_cols` x 64 rows x 1 head; rows beyond T read as zero.
bool make_map(CUtensorMap* tm, const void* ptr, int BH, int T, int box_cols, bool swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
  cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)C, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t tc_chunked_state_elems() { return (size_t)NSLICE * NT * 128 * 64; }
int tc_chunked_slices() { return NSLICE; }

void tc_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, int* device_status,
                LaunchCtx& ctx) {
  (void)use_scan;
  (void)ws;
  const int BH = p.B * p.H;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_map(&tmQ, p.q, BH, p.T, 64, true) || !make_map(&tmK, p.k, BH, p.T, 64, true) ||
      !make_map(&tmV, p.v, BH, p.T, VS, false)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  if (cudaFuncSetAttribute(tc_chunk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) !=
      cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  tc_chunk_kernel<<<dim3(NSLICE, BH), NTHREADS, SMEM_ALLOC, ctx.stream>>>(
      tmQ, tmK, tmV, static_cast<__nv_bfloat16*>(p.out), p.T, plan.n_chunks, device_status);
  note_launch(ctx);
}

}  // namespace kata
