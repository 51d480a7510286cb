// Chunked-state KATA forward on the Blackwell tensor cores (tcgen05 + TMEM), bf16, d_k = d_v = 64, C = 64.
//
// Formulation.  With k' = k / ||k|| the state is S[a,b,v] = sum_i k'_a k'_b v_v (symmetric in a,b) and the
// normaliser state Z[a,b] = sum_i k'_a k'_b.  One CTA owns one head and 8 value columns; output columns
// are independent, so CTAs never exchange data.  The d_k^2-wide feature GEMMs of the chunk equations are
// re-associated so that no feature matrix Psi is ever built:
//
//   state update   S[(b,v), a] += sum_t W[(b,v), t] * k[t, a],   W[(b,v), t] = k[t,b] v[t,v] / ||k_t||^2
//                  (tcgen05 kind::f16: A = W, built in registers and stored to TMEM; B = the TMA-loaded
//                   key tile used MN-major; D = fp32 accumulators resident in TMEM for the whole head)
//   inter-chunk    Y[(b,v), t] = sum_a S[(b,v), a] * q[t, a]     (tcgen05 kind::tf32: A = the fp32
//   read           accumulators of the update, read straight from TMEM; B = the query tile as tf32)
//                  N_inter[t, v] = sum_b q[t,b] * Y[(b,v), t]    (fp32 FMAs on the TMEM read-back)
//   normaliser     the same two steps with the "ones" value column: rows (b) of a fifth tile hold Z
//   intra-chunk    scores s = Q K^T from one d-dimensional bf16 MMA; P = s^2 / ||k||^2 o M in fp32,
//                  rounded to bf16 into TMEM; [N_intra | D_intra] = P [V | 1] as one more MMA, so the
//                  normaliser is the row sum of exactly the P that multiplies V
//   epilogue       O = (N_inter + N_intra) / (D_inter + D_intra)   (gate + normalise), bf16 store
//
// The query norm is a common factor of numerator and denominator and is never applied.  Rows (b,v) of a
// 128-row MMA tile are b = 16*tile + row/8, v = row%8; four tiles cover b = 0..63, the fifth holds Z.
//
// Scan form: grid.z cuts the chunk axis into groups.  A first launch (write_out = 0) only accumulates
// the group-local states and stores them; after the log-depth scan over groups a second launch restarts
// every group from the prefix before it.
//
// Warp roles (512 threads): warp 0 TMA producer; warps 1-3 MMA issuers (one elected lane each; issuer j
// owns state tiles j and j+3: the read of a tile and then its update, so the write-after-read on the tile
// is ordered by issue order; issuer 2 also issues the score MMA and the P[V|1] MMA); warps 4-7 operand
// builders (norms, tf32 query tile, transposes, W tiles); warps 8-15 TMEM readers in two groups (Y
// reduction, scores, epilogue).  Several issuing warps are needed because a thread that has MMAs in flight stalls on its next
// barrier wait until they drain; with three issuers the tensor pipe stays fed.
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
constexpr int NT = 5;            // state tiles: 4 x S + the normaliser tile
constexpr int NI = 6;            // ring items per chunk: 5 reads + the score/intra item
constexpr int NTHREADS = 512;   // 16 warps = 4 per scheduler: 128 registers per thread
constexpr int WARP_ISS0 = 1, WARP_BLD0 = 4, WARP_RD0 = 8;   // first warp of each role
constexpr int NISSUER = 3;
constexpr size_t STATE_PER_SLICE = (size_t)NT * 128 * 64;   // floats

// TMEM columns (128 lanes each)
constexpr uint32_t COL_S = 0;      // 5 x 64 fp32: S tiles 0..3, Z tile 4
constexpr uint32_t COL_R = 320;    // 2 x 64: ring (read results; scores -> P bf16 [0,32) -> P[V|1] at [32,48))
constexpr uint32_t COL_W = 448;    // 2 x 32: W tiles (bf16 pairs), A operand of the update
constexpr uint32_t TMEM_COLS = 512;

// shared memory map (bytes from a 1024-aligned base)
constexpr uint32_t KT_STRIDE = 144;               // bytes per kT / vT row: 64 bf16 + 16 pad (conflict-free LDS.128)
constexpr uint32_t OFF_QK = 0;                    // 2 stages x (Q tile 8 KB, K tile 8 KB), TMA, 128B swizzle
constexpr uint32_t OFF_V = 32768;                 // 2 stages x 64 x 8 bf16 (TMA, dense 16-byte rows)
constexpr uint32_t OFF_ONES = 34816;              // 64 x 8 bf16 rows (1,0,..,0): the "ones" column group
constexpr uint32_t OFF_QF = 35840;                // 2 x 16 KB: query tile as tf32, K-major, 128B swizzle, 2 atoms
constexpr uint32_t OFF_KT = 68608;                // kT[b][t] bf16, 64 rows (builders only)
constexpr uint32_t OFF_VT = 86016;                // vT[v][t] = bf16(v / ||k||^2), row 8 = bf16(1 / ||k||^2) (builders only)
constexpr uint32_t OFF_QT = 88192;                // 2 x qT[b][t] bf16, 144-byte rows (readers)
constexpr uint32_t OFF_R2 = 120960;               // 2 x r2[t] = 1/||k_t||^2
constexpr uint32_t OFF_RED = 121472;              // red[128+64][68] fp32: state partials, normaliser partials
constexpr uint32_t RED_STRIDE = 68;
constexpr uint32_t OFF_NINTRA = 173696;           // [64][9]
constexpr uint32_t OFF_BAR = 176000;              // mbarriers
constexpr uint32_t SMEM_BYTES = OFF_BAR + 512;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;  // slack for the 1024-byte alignment
static_assert(OFF_QF % 1024 == 0 && OFF_QK % 1024 == 0, "swizzled tiles need 1024-byte alignment");
static_assert(SMEM_ALLOC > 116 * 1024, "one CTA per SM is assumed (the CTA allocates all of TMEM)");

// Barriers are indexed per tile / per ring item, never per buffer: roles run at different speeds, and a
// buffer-indexed barrier shared by several waiters lets a waiter observe the parity of a phase that is
// two completions away from the one it means (phase aliasing).  Every barrier below completes exactly
// once per chunk (stage barriers: once per two chunks) and each waiter waits for every phase in order.
enum {
  BAR_FULL = 0,     // [2] TMA landed
  BAR_EMPTY = 2,    // [2] stage free (128 builders + one commit per issuer)
  BAR_PREP = 4,     // [2] operands of the chunk built (128 builders)
  BAR_WFULL = 6,    // [5] W tile i stored to TMEM (128 builders)
  BAR_RFULL = 11,   // [6] ring item i produced by the MMA
  BAR_REMPTY = 17,  // [6] ring item i drained (256 readers)
  BAR_PREADY = 23,  // P (bf16) stored to TMEM (256 readers)
  BAR_PVFULL = 24,  // P [V|1] complete
  BAR_U = 25,       // [5] update of state tile i complete (frees the W buffer, allows the next read)
  BAR_DRAIN = 30,
  BAR_DONE = 31,    // every update of this CTA has completed
  BAR_COUNT = 32
};

struct Shared {
  unsigned char* base;
  __device__ unsigned char* qtile(int s) const { return base + OFF_QK + s * 16384; }
  __device__ unsigned char* ktile(int s) const { return base + OFF_QK + s * 16384 + 8192; }
  __device__ unsigned char* vtile(int s) const { return base + OFF_V + s * 1024; }
  __device__ unsigned char* ones() const { return base + OFF_ONES; }
  __device__ unsigned char* qf(int s) const { return base + OFF_QF + s * 16384; }
  __device__ unsigned char* kT() const { return base + OFF_KT; }
  __device__ unsigned char* vT() const { return base + OFF_VT; }
  __device__ unsigned char* qT(int s) const { return base + OFF_QT + s * 16384; }
  __device__ float* r2(int s) const { return reinterpret_cast<float*>(base + OFF_R2 + s * 256); }
  __device__ float* red() const { return reinterpret_cast<float*>(base + OFF_RED); }
  __device__ float* nintra() const { return reinterpret_cast<float*>(base + OFF_NINTRA); }
  __device__ uint64_t* bar(int i) const { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; }
};

__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
__device__ __forceinline__ void reader_sync() { asm volatile("bar.sync 3, 256;" ::: "memory"); }
// the two reader warps (one per group) that share TMEM lane quadrant q
__device__ __forceinline__ void group_pair_sync(uint32_t q) { asm volatile("bar.sync %0, 64;" ::"r"(4 + q) : "memory"); }

// Bounded wait that also gives up as soon as another role has flagged an abort.
// Bounded wait, as few instructions per poll as possible (the polling warps share the issue slots with the warps
// that work): try_wait, exit branch, counter, loop branch.  A wait that gives up raises the abort flag; the other
// waiters give up on their own limits.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  uint32_t ok;
  asm volatile(
      "{\n\t"
      ".reg .pred p, q;\n\t"
      ".reg .u32 i;\n\t"
      "mov.u32 i, 0;\n\t"
      "KATA_WAIT_%=:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "@p bra KATA_DONE_%=;\n\t"
      "add.u32 i, i, 1;\n\t"
      "setp.lt.u32 q, i, %3;\n\t"
      "@q bra KATA_WAIT_%=;\n\t"
      "KATA_DONE_%=:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kSpinLimit)
      : "memory");
  if (ok == 0) *abort_flag = 1;
  return ok != 0;
}

// element-wise product of two packed bf16 pairs (one HMUL2.BF16)
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

struct KernelArgs {
  __nv_bfloat16* out;
  const float* init_state;   // inclusive group scan [BH][n_groups][NSLICE][5][128][64]; group g starts from entry g-1
  float* final_state;        // same layout; group g stores entry g
  int* device_status;
  int Tlen, n_chunks, chunks_per_group, n_groups, write_out;
};

__global__ void __launch_bounds__(NTHREADS, 1)
tc_chunk_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const KernelArgs args) {
  extern __shared__ unsigned char smem_raw[];
  Shared sm;
  sm.base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slice = blockIdx.x, bh = blockIdx.y, grp = blockIdx.z;
  const int c_begin = grp * args.chunks_per_group;
  const int c_end = min(args.n_chunks, c_begin + args.chunks_per_group);
  const int nloc = c_end - c_begin;                  // chunks handled by this CTA
  const bool write_out = args.write_out != 0;
  const bool have_init = args.init_state != nullptr && grp > 0;
  const size_t state_off = (((size_t)bh * args.n_groups + grp) * NSLICE + slice) * STATE_PER_SLICE;

  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(sm.bar(BAR_FULL + i), 1);
      mbar_init(sm.bar(BAR_EMPTY + i), 128 + NISSUER);
      mbar_init(sm.bar(BAR_PREP + i), 128);
    }
    for (int i = 0; i < NT; ++i) {
      mbar_init(sm.bar(BAR_WFULL + i), 128);
      mbar_init(sm.bar(BAR_U + i), 1);
    }
    for (int i = 0; i < NI; ++i) {
      mbar_init(sm.bar(BAR_RFULL + i), 1);
      mbar_init(sm.bar(BAR_REMPTY + i), 256);
    }
    mbar_init(sm.bar(BAR_PREADY), 256);
    mbar_init(sm.bar(BAR_PVFULL), 1);
    mbar_init(sm.bar(BAR_DRAIN), NISSUER);
    mbar_init(sm.bar(BAR_DONE), NISSUER);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  // constant "ones" column group for the intra-chunk MMA: row t = (1, 0, 0, 0, 0, 0, 0, 0) in bf16
  if (tid < 64) {
    *reinterpret_cast<uint4*>(sm.ones() + tid * 16) = make_uint4(0x00003F80u, 0u, 0u, 0u);
    fence_async_smem();
  }
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;

  // initial state: zero, or the prefix of the groups before this one (readers own the TMEM lanes)
  if (warp >= WARP_RD0 && warp < WARP_RD0 + 4) {
    const uint32_t q4 = warp & 3;
    const int rowl = q4 * 32 + lane;
    uint32_t z[32];
    for (int cblk = 0; cblk < (NT * 64) / 32; ++cblk) {
      if (have_init) {
        const float* src = args.init_state + (state_off - (size_t)NSLICE * STATE_PER_SLICE) +
                           ((size_t)(cblk >> 1) * 128 + rowl) * 64 + (cblk & 1) * 32;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 f = *reinterpret_cast<const float4*>(src + j);
          z[j] = __float_as_uint(f.x);
          z[j + 1] = __float_as_uint(f.y);
          z[j + 2] = __float_as_uint(f.z);
          z[j + 3] = __float_as_uint(f.w);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) z[j] = 0u;
      }
      tmem_st32(tmem_addr(tb, q4 * 32, COL_S + cblk * 32), z);
    }
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  bool ok = true;

  if (warp == 0) {
    // =========================== TMA producer ===========================
    if (lane == 0) {
      for (int c = 0; c < nloc && ok; ++c) {
        const int s = c & 1;
        ok = wait_or_abort(sm.bar(BAR_EMPTY + s), ((c >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        const int t0 = (c_begin + c) * C;
        mbar_arrive_expect_tx(sm.bar(BAR_FULL + s), 8192 + 8192 + 1024);
        tma_load_3d(sm.qtile(s), &tmQ, sm.bar(BAR_FULL + s), 0, t0, bh);
        tma_load_3d(sm.ktile(s), &tmK, sm.bar(BAR_FULL + s), 0, t0, bh);
        tma_load_3d(sm.vtile(s), &tmV, sm.bar(BAR_FULL + s), slice * VS, t0, bh);
      }
    }
  } else if (warp < WARP_BLD0) {
    // =========================== MMA issuers ===========================
    if (lane == 0) {
      const int j = warp - WARP_ISS0;            // issuer index = state tile it owns
      const uint32_t id_read = instr_desc(kFmtTF32, kFmtTF32, 0, 0, 128, 64);    // A tmem (fp32 as tf32), B K-major
      const uint32_t id_qk = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 64);      // both K-major from smem
      const uint32_t id_upd = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 64);     // A tmem, B MN-major
      const uint32_t id_pv = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 16);      // A tmem, B MN-major, N = 16
      const uint64_t d_k128 = smem_desc(0, 16, 1024, kSwizzle128B);              // K-major, 128B swizzle
      const uint64_t d_mn128 = smem_desc(0, 8192, 1024, kSwizzle128B);           // MN-major, 128B swizzle
      auto at = [](uint64_t d, uint32_t addr) { return d + (uint64_t)((addr >> 4) & 0x3FFF); };

      // Y_i = S_i * Q^T (tf32, A = accumulators in TMEM) into ring item (c, i)
      auto issue_read = [&](int c, int i) {
        const int g = c * NI + i;
        // the ring slot (g & 1) is free once its previous occupant, item g - 2, has been drained
        if (g >= 2) ok = wait_or_abort(sm.bar(BAR_REMPTY + (g - 2) % NI), ((g - 2) / NI) & 1, abort_flag);
        if (ok && c > 0) ok = wait_or_abort(sm.bar(BAR_U + i), (c - 1) & 1, abort_flag);
        if (!ok) return;
        tc_fence_after();
        const uint32_t qf = smem_u32(sm.qf(c & 1));
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          mma_tf32_ts(tb + COL_R + (g & 1) * 64, tb + COL_S + i * 64 + ks * 8,
                      at(d_k128, qf + (ks >> 2) * 8192 + (ks & 3) * 32), id_read, ks > 0);
        mma_commit(sm.bar(BAR_RFULL + i));
      };
      // S_i += W_i * K (A = W in TMEM, B = key tile MN-major)
      auto issue_update = [&](int c, int i) {
        const int g = c * NT + i;
        ok = wait_or_abort(sm.bar(BAR_WFULL + i), c & 1, abort_flag);
        if (!ok) return;
        tc_fence_after();
        const uint32_t ka = smem_u32(sm.ktile(c & 1));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_f16_ts(tb + COL_S + i * 64, tb + COL_W + (g & 1) * 32 + ks * 8, at(d_mn128, ka + ks * 2048), id_upd, 1u);
        mma_commit(sm.bar(BAR_U + i));
      };
      // intra-chunk scores [Q;K] K^T into ring item (c, 5) (rows 0..63 used)
      auto issue_qk = [&](int c) {
        const int g = c * NI + 5;
        ok = wait_or_abort(sm.bar(BAR_REMPTY + 3), c & 1, abort_flag);     // item (c, 3) shared the slot
        if (!ok) return;
        tc_fence_after();
        const uint32_t qa = smem_u32(sm.qtile(c & 1)), ka = smem_u32(sm.ktile(c & 1));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_f16_ss(tb + COL_R + (g & 1) * 64, at(d_k128, qa + ks * 32), at(d_k128, ka + ks * 32), id_qk, ks > 0);
        mma_commit(sm.bar(BAR_RFULL + 5));
      };
      // [N_intra | D_intra] = P [V | 1] (A = P bf16 in the ring slot; B = the value tile and the ones group)
      auto issue_pv = [&](int c) {
        const int g = c * NI + 5;
        ok = wait_or_abort(sm.bar(BAR_PREADY), c & 1, abort_flag);
        if (!ok) return;
        tc_fence_after();
        const uint32_t va = smem_u32(sm.vtile(c & 1));
        const uint32_t ones_off = smem_u32(sm.ones()) - va;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          // MN-major, no swizzle: 8 k-rows x 16 bytes per core matrix, next 8 k at +128 (LBO), the second
          // group of 8 columns (the ones group) at +ones_off (SBO)
          mma_f16_ts(tb + COL_R + (g & 1) * 64 + 32, tb + COL_R + (g & 1) * 64 + ks * 8,
                     smem_desc(va + ks * 256, 128, ones_off, kSwizzleNone), id_pv, ks > 0);
        mma_commit(sm.bar(BAR_PVFULL));
      };

      for (int c = 0; c < nloc && ok; ++c) {
        const int s = c & 1;
        const uint32_t ph = (c >> 1) & 1;
        ok = wait_or_abort(sm.bar(BAR_FULL + s), ph, abort_flag) &&
             wait_or_abort(sm.bar(BAR_PREP + s), ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (write_out) issue_read(c, j);
        if (ok) issue_update(c, j);
        if (j < 2) {
          if (ok && write_out) issue_read(c, j + 3);
          if (ok) issue_update(c, j + 3);
        } else if (write_out) {
          if (ok) issue_qk(c);
          if (ok) issue_pv(c);
        }
        if (!ok) break;
        mma_commit(sm.bar(BAR_EMPTY + s));
      }
      if (ok) mma_commit(sm.bar(BAR_DONE));
    }
  } else if (warp < WARP_RD0) {
    // =========================== operand builders (128 threads) ===========================
    const int ta = tid - WARP_BLD0 * 32;
    const int row = ta >> 1, hf = ta & 1;          // prep mapping: two threads per token row
    const uint32_t q4 = warp & 3;                  // TMEM lane quadrant of this warp
    const int rowl = q4 * 32 + lane;               // W-tile row owned by this thread
    unsigned char* kT = sm.kT();
    unsigned char* vT = sm.vT();
    for (int c = 0; c < nloc && ok; ++c) {
      const int s = c & 1;
      ok = wait_or_abort(sm.bar(BAR_FULL + s), (c >> 1) & 1, abort_flag);
      if (!ok) break;
      group_sync(2);   // every builder is done with kT / vT of the previous chunk
      unsigned char* qT = sm.qT(s);
      float* r2 = sm.r2(s);
      // ---- phase 1: key norms, tf32 query tile; kT and qT (bf16 transposes) via ldmatrix / stmatrix.trans ----
      {
        const unsigned char* kt = sm.ktile(s);
        const unsigned char* qt = sm.qtile(s);
        unsigned char* qf = sm.qf(s) + hf * 8192;
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int chunk = hf * 4 + j;
          const uint4 kraw = *reinterpret_cast<const uint4*>(kt + sw128_offset(row, chunk));
          const uint32_t kw[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float lo = __uint_as_float(kw[e] << 16), hi = __uint_as_float(kw[e] & 0xFFFF0000u);
            ss = fmaf(lo, lo, ss);
            ss = fmaf(hi, hi, ss);
          }
          if (write_out) {
            const uint4 qraw = *reinterpret_cast<const uint4*>(qt + sw128_offset(row, chunk));
            const uint32_t qw[4] = {qraw.x, qraw.y, qraw.z, qraw.w};
            // tf32 query tile: 32 fp32 per 128-byte row, this thread's half-row is atom `hf`
            *reinterpret_cast<float4*>(qf + sw128_offset(row, 2 * j)) =
                make_float4(__uint_as_float(qw[0] << 16), __uint_as_float(qw[0] & 0xFFFF0000u),
                            __uint_as_float(qw[1] << 16), __uint_as_float(qw[1] & 0xFFFF0000u));
            *reinterpret_cast<float4*>(qf + sw128_offset(row, 2 * j + 1)) =
                make_float4(__uint_as_float(qw[2] << 16), __uint_as_float(qw[2] & 0xFFFF0000u),
                            __uint_as_float(qw[3] << 16), __uint_as_float(qw[3] & 0xFFFF0000u));
          }
        }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        if (hf == 0) r2[row] = inv_or_zero(ss);
        // transposes: this warp owns feature blocks 2*wb and 2*wb+1 (8 features each) for all 64 tokens.
        // One ldmatrix.x4 reads four 8-token x 8-feature blocks, stmatrix.x4.trans writes their transposes.
        const int wb = warp - WARP_BLD0;
        const int mj = lane >> 3, mr = lane & 7;      // matrix index and row this lane addresses
#pragma unroll
        for (int ab = 0; ab < 2; ++ab) {
          const int A = 2 * wb + ab;                  // feature block = 16-byte chunk index of a tile row
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int tblk = 4 * h + mj;              // token block of the matrix this lane addresses
            uint32_t frag[4];
            ldmatrix_x4(frag, smem_u32(kt + sw128_offset(tblk * 8 + mr, A)));
            stmatrix_x4_trans(smem_u32(kT + (A * 8 + mr) * KT_STRIDE + tblk * 16), frag);
            if (write_out) {
              ldmatrix_x4(frag, smem_u32(qt + sw128_offset(tblk * 8 + mr, A)));
              stmatrix_x4_trans(smem_u32(qT + (A * 8 + mr) * KT_STRIDE + tblk * 16), frag);
            }
          }
        }
      }
      group_sync(2);
      // ---- phase 2: transposed values scaled by 1/||k||^2 (bf16); row 8 is the scale itself ----
      if (ta < C) {
        const uint4 vraw = *reinterpret_cast<const uint4*>(sm.vtile(s) + ta * 16);
        const uint32_t vw[4] = {vraw.x, vraw.y, vraw.z, vraw.w};
        const float rr = r2[ta];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t p2 = pack_bf16(__uint_as_float(vw[e] << 16) * rr, __uint_as_float(vw[e] & 0xFFFF0000u) * rr);
          *reinterpret_cast<uint16_t*>(vT + (2 * e) * KT_STRIDE + ta * 2) = (uint16_t)(p2 & 0xFFFFu);
          *reinterpret_cast<uint16_t*>(vT + (2 * e + 1) * KT_STRIDE + ta * 2) = (uint16_t)(p2 >> 16);
        }
        *reinterpret_cast<uint16_t*>(vT + 8 * KT_STRIDE + ta * 2) = (uint16_t)(pack_bf16(rr, 0.f) & 0xFFFFu);
      }
      fence_async_smem();
      group_sync(2);
      mbar_arrive(sm.bar(BAR_PREP + s));
      // the scaled value row of this thread (v = rowl % 8) as 32 bf16 pairs
      uint32_t vr[32];
      {
        const unsigned char* vrow = vT + (rowl & 7) * KT_STRIDE;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 f = *reinterpret_cast<const uint4*>(vrow + j * 16);
          vr[4 * j] = f.x; vr[4 * j + 1] = f.y; vr[4 * j + 2] = f.z; vr[4 * j + 3] = f.w;
        }
      }
      // ---- W tiles: row rowl <-> (b = 16 i + rowl/8, v = rowl%8); fifth tile: rows < 64 hold k[t,b]/||k||^2.
      //      One packed bf16 multiply per token pair; the products go straight to TMEM.  The key row of
      //      the next tile is fetched while the TMEM store of the current one is in flight. ----
      uint32_t kk[32];
      auto load_krow = [&](int i) {
        const unsigned char* krow = kT + ((i < 4) ? (16 * i + (rowl >> 3)) : (rowl & 63)) * KT_STRIDE;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint4 f = *reinterpret_cast<const uint4*>(krow + j * 16);
          kk[4 * j] = f.x; kk[4 * j + 1] = f.y; kk[4 * j + 2] = f.z; kk[4 * j + 3] = f.w;
        }
      };
      load_krow(0);
      for (int i = 0; i < NT && ok; ++i) {
        const int g = c * NT + i;
        uint32_t pk[32];
        if (i == 4) {
          // normaliser tile: the value row is the scale 1/||k||^2 itself; rows 64..127 are not used
          const unsigned char* srow = vT + 8 * KT_STRIDE;
          const bool live = rowl < 64;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint4 rr = *reinterpret_cast<const uint4*>(srow + j * 16);
            pk[4 * j] = live ? mul_bf16x2(kk[4 * j], rr.x) : 0u;
            pk[4 * j + 1] = live ? mul_bf16x2(kk[4 * j + 1], rr.y) : 0u;
            pk[4 * j + 2] = live ? mul_bf16x2(kk[4 * j + 2], rr.z) : 0u;
            pk[4 * j + 3] = live ? mul_bf16x2(kk[4 * j + 3], rr.w) : 0u;
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) pk[j] = mul_bf16x2(kk[j], vr[j]);
        }
        if (g >= 2) {   // the W buffer is free once the update two tiles back has completed
          const int gp = g - 2;
          ok = wait_or_abort(sm.bar(BAR_U + gp % NT), (gp / NT) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
        }
        tmem_st32(tmem_addr(tb, q4 * 32, COL_W + (g & 1) * 32), pk);
        if (i + 1 < NT) load_krow(i + 1);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(sm.bar(BAR_WFULL + i));
      }
      if (!ok) break;
      mbar_arrive(sm.bar(BAR_EMPTY + s));     // done with the stage (each issuer adds its own arrival)
    }
  } else {
    // =========================== TMEM readers (2 groups x 128 threads) ===========================
    // Both groups drain every ring item; group g owns the token columns [32 g, 32 g + 32) of it, so a
    // thread keeps 32 accumulators and one TMEM load of 32 columns covers its share of an item.  The
    // load of an item is in flight while the previous item is multiplied in.
    const int rgrp = (warp - WARP_RD0) >> 2;   // column half
    const int tr = tid - WARP_RD0 * 32;        // 0..255
    const uint32_t q4 = warp & 3;              // TMEM lane quadrant this warp may access
    const int rowl = q4 * 32 + lane;           // tile row (= TMEM lane) of this thread
    const int t0h = rgrp * 32;                 // first token column of this group
    float* redS = sm.red();                               // [128][68]: partial sums over the four state tiles
    float* redZ = sm.red() + 128 * RED_STRIDE;            // [64][68]: normaliser partials
    float* nintra = sm.nintra();
    __nv_bfloat16* oh = args.out + (size_t)bh * args.Tlen * D + slice * VS;
    for (int c = 0; c < nloc && ok && write_out; ++c) {
      const int s = c & 1;
      ok = wait_or_abort(sm.bar(BAR_PREP + s), (c >> 1) & 1, abort_flag);
      if (!ok) break;
      const unsigned char* qT = sm.qT(s);
      const float* r2 = sm.r2(s);
      float acc[32];
#pragma unroll
      for (int t = 0; t < 32; ++t) acc[t] = 0.f;
      // acc[t] += q[t,b] * Y[row, t] over this group's 32 token columns (b = feature index of the row)
      auto fma32 = [&](const uint32_t (&y)[32], int i) {
        const int b = (i < 4) ? (16 * i + (rowl >> 3)) : (rowl & 63);
        const unsigned char* qrow = qT + b * KT_STRIDE + t0h * 2;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint4 qa = *reinterpret_cast<const uint4*>(qrow + j * 16);
          const uint32_t qw[4] = {qa.x, qa.y, qa.z, qa.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int t = j * 8 + 2 * e;
            const float2 r = __ffma2_rn(make_float2(__uint_as_float(qw[e] << 16), __uint_as_float(qw[e] & 0xFFFF0000u)),
                                        make_float2(__uint_as_float(y[t]), __uint_as_float(y[t + 1])),
                                        make_float2(acc[t], acc[t + 1]));
            acc[t] = r.x;
            acc[t + 1] = r.y;
          }
        }
      };
      auto start_item = [&](uint32_t (&y)[32], int i) {
        ok = wait_or_abort(sm.bar(BAR_RFULL + i), c & 1, abort_flag);
        if (!ok) return;
        tc_fence_after();
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_R + (i & 1) * 64 + t0h), y);
      };
      auto finish_item = [&](uint32_t (&y)[32], int i) {
        tmem_wait_ld(y);
        tc_fence_before();
        mbar_arrive(sm.bar(BAR_REMPTY + i));      // this group's share of the item is in registers now
      };
      auto store_acc = [&](float* dst) {
#pragma unroll
        for (int t4 = 0; t4 < 32; t4 += 4)
          *reinterpret_cast<float4*>(dst + rowl * RED_STRIDE + t0h + t4) =
              make_float4(acc[t4], acc[t4 + 1], acc[t4 + 2], acc[t4 + 3]);
      };
      uint32_t ya[32], yb[32];
      start_item(ya, 0);
      if (!ok) break;
      finish_item(ya, 0);
      start_item(yb, 1);
      if (!ok) break;
      fma32(ya, 0);
      finish_item(yb, 1);
      start_item(ya, 2);
      if (!ok) break;
      fma32(yb, 1);
      finish_item(ya, 2);
      start_item(yb, 3);
      if (!ok) break;
      fma32(ya, 2);
      finish_item(yb, 3);
      start_item(ya, 4);
      if (!ok) break;
      fma32(yb, 3);
      store_acc(redS);            // the four state tiles
#pragma unroll
      for (int t = 0; t < 32; ++t) acc[t] = 0.f;
      finish_item(ya, 4);
      // ---- intra-chunk scores (item 5): start the load, finish the normaliser tile meanwhile ----
      ok = wait_or_abort(sm.bar(BAR_RFULL + 5), c & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if (rowl < 64) tmem_ld32(tmem_addr(tb, q4 * 32, COL_R + 64 + t0h), yb);
      fma32(ya, 4);
      if (rowl < 64) {
        store_acc(redZ);          // normaliser tile: rows 0..63 hold b
        // P = s^2 / ||k||^2 (causal) -> bf16 into columns [16 g, 16 g + 16) of the slot.  Every lane's
        // scores are read (by both groups) before PREADY completes, and the MMA that overwrites the
        // slot waits for PREADY.
        tmem_wait_ld(yb);
        uint32_t pk[16];
#pragma unroll
        for (int jj = 0; jj < 32; jj += 4) {
          const int j = t0h + jj;
          const float4 rr = *reinterpret_cast<const float4*>(r2 + j);
          const float s0 = __uint_as_float(yb[jj]), s1 = __uint_as_float(yb[jj + 1]);
          const float s2 = __uint_as_float(yb[jj + 2]), s3 = __uint_as_float(yb[jj + 3]);
          const float w0 = (j <= rowl) ? s0 * s0 * rr.x : 0.f;
          const float w1 = (j + 1 <= rowl) ? s1 * s1 * rr.y : 0.f;
          const float w2 = (j + 2 <= rowl) ? s2 * s2 * rr.z : 0.f;
          const float w3 = (j + 3 <= rowl) ? s3 * s3 * rr.w : 0.f;
          pk[jj / 2] = pack_bf16(w0, w1);
          pk[jj / 2 + 1] = pack_bf16(w2, w3);
        }
        tc_fence_before();
        group_pair_sync(q4);      // both groups have read their scores of these 32 lanes
        tc_fence_after();
        tmem_st16(tmem_addr(tb, q4 * 32, COL_R + 64 + rgrp * 16), pk);
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(sm.bar(BAR_PREADY));
      // ---- [N_intra | D_intra] from the MMA ----
      ok = wait_or_abort(sm.bar(BAR_PVFULL), c & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if (rowl < 64 && rgrp == 0) {
        uint32_t pv[16];
        tmem_ld16(tmem_addr(tb, q4 * 32, COL_R + 64 + 32), pv);
        tmem_wait_ld(pv);
#pragma unroll
        for (int v = 0; v < 9; ++v) nintra[rowl * 9 + v] = __uint_as_float(pv[v]);
      }
      tc_fence_before();
      mbar_arrive(sm.bar(BAR_REMPTY + 5));
      reader_sync();      // partial sums are in shared memory
      // ---- reduce over b, gate + normalise epilogue: thread <-> (t, two value columns) ----
      {
        const int t = tr >> 2, sub = tr & 3;
        float zv[16], nv[32];
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) zv[kk] = redZ[(4 * kk + sub) * RED_STRIDE + t];
#pragma unroll
        for (int bl = 0; bl < 16; ++bl) {
          nv[2 * bl] = redS[(bl * 8 + 2 * sub) * RED_STRIDE + t];
          nv[2 * bl + 1] = redS[(bl * 8 + 2 * sub + 1) * RED_STRIDE + t];
        }
        float zp = 0.f, n0 = 0.f, n1 = 0.f;
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) zp += zv[kk];
#pragma unroll
        for (int bl = 0; bl < 16; ++bl) {
          n0 += nv[2 * bl];
          n1 += nv[2 * bl + 1];
        }
        zp += __shfl_xor_sync(0xffffffffu, zp, 1);
        zp += __shfl_xor_sync(0xffffffffu, zp, 2);
        const int tg = (c_begin + c) * C + t;
        if (tg < args.Tlen) {
          const float den = zp + nintra[t * 9 + 8];
          const float inv = den > 0.f ? 1.f / den : 0.f;
          const uint32_t pk = pack_bf16((n0 + nintra[t * 9 + 2 * sub]) * inv, (n1 + nintra[t * 9 + 2 * sub + 1]) * inv);
          *reinterpret_cast<uint32_t*>(oh + (size_t)tg * D + 2 * sub) = pk;
        }
      }
      reader_sync();      // the scratch is rewritten in the next chunk
    }
    // ---- final state of this group (scan pass 1) ----
    if (ok && args.final_state != nullptr && rgrp == 0) {
      ok = wait_or_abort(sm.bar(BAR_DONE), 0, abort_flag);
      tc_fence_after();
      if (ok) {
        float* dst = args.final_state + state_off;
        for (int cblk = 0; cblk < (NT * 64) / 32; ++cblk) {
          uint32_t z[32];
          tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + cblk * 32), z);
          tmem_wait_ld(z);
          float* d = dst + ((size_t)(cblk >> 1) * 128 + rowl) * 64 + (cblk & 1) * 32;
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            *reinterpret_cast<float4*>(d + j) = make_float4(__uint_as_float(z[j]), __uint_as_float(z[j + 1]),
                                                            __uint_as_float(z[j + 2]), __uint_as_float(z[j + 3]));
        }
      }
    }
  }

  // ---------------- teardown ----------------
  if (!ok && args.device_status != nullptr) atomicExch(args.device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp >= WARP_ISS0 && warp < WARP_BLD0 && lane == 0) {
    // make sure no MMA is still in flight before TMEM is released
    mma_commit(sm.bar(BAR_DRAIN));
    mbar_wait(sm.bar(BAR_DRAIN), 0);
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

size_t tc_chunked_state_elems() { return (size_t)NSLICE * STATE_PER_SLICE; }
int tc_chunked_slices() { return NSLICE; }

void tc_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, int* device_status,
                const float* s_init, const float* z_init, float* s_final, float* z_final, int state_layout,
                LaunchCtx& ctx) {
  if (!use_scan) {   // whole sequence in one pass: the token-major streaming kernel
    if (s_final != nullptr || s_init != nullptr)
      tc_chunked_stream_export(p, device_status, s_init, z_init, s_final, z_final, state_layout, ctx);
    else tc_chunked_stream(p, device_status, ctx);
    return;
  }
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
  KernelArgs a;
  a.out = static_cast<__nv_bfloat16*>(p.out);
  a.device_status = device_status;
  a.Tlen = p.T;
  a.n_chunks = plan.n_chunks;
  const int NG = plan.n_groups;
  const size_t E = tc_chunked_state_elems();
  float* bufA = ws;
  float* bufB = ws + (size_t)BH * NG * E;
  const float* incl = bufA;
  a.chunks_per_group = plan.chunks_per_group;
  a.n_groups = NG;
  if (NG > 1) {
    a.init_state = nullptr;
    a.final_state = bufA;
    a.write_out = 0;
    tc_chunk_kernel<<<dim3(NSLICE, BH, NG - 1), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, tmV, a);
    note_launch(ctx);
    incl = scan_group_states(bufA, bufB, BH, NG, NG - 1, E, ctx);
  }
  a.init_state = incl;
  a.final_state = nullptr;
  a.write_out = 1;
  tc_chunk_kernel<<<dim3(NSLICE, BH, NG), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, tmV, a);
  note_launch(ctx);
}

}  // namespace kata
