// Quadratic ("flash-style") KATA forward on the Blackwell tensor cores (tcgen05 + TMEM), bf16, d_k = d_v = 64.
//
// Pre-pass (one light kernel per call): V'[i] = v_i / ||k_i||^2 (bf16) and r[i] = 1 / ||k_i||^2 (bf16) into
// the workspace, so that the key scale never touches the 128 x 128 weight tiles.
//
// Main kernel: persistent, one CTA per SM.  A work item = one head x one tile of 128 queries; the items are ordered
// heaviest first (latest query tiles first) and dealt round-robin to the CTAs, which walk the key tiles j <= i of
// 128 keys of each of their items:
//   scores   S = Q K_j^T            tcgen05 kind::f16; A = the query tile and B = the key tile, both TMA-loaded
//                                   128B-swizzled tiles in shared memory; fp32 result in one of three TMEM buffers
//   weights  P = S^2 (causal mask   packed fp32x2 multiplies on the TMEM read-back, rounded to bf16 and stored
//            on the diagonal tile)  back over the first 64 columns of the same buffer
//   apply    [O | D] += P [V' | r]  tcgen05 kind::f16, A = P from TMEM, B = the V' tile plus one extra column
//                                   group holding r, MN-major, N = 80: the normaliser is column 64 of the
//                                   same accumulator
//   epilogue out = O / D (0 where D = 0)      the gate/normalise step of the readout
// There is no running maximum and no rescaling: the weights are polynomial.  The query norm cancels between
// numerator and denominator and is never applied.  The d^2-wide feature state is never formed.
// Nothing is set up per item: TMEM and the barriers are the CTA's, the stage and buffer rings run on across items
// (every role counts tiles cumulatively), the query tile is double-buffered, and the producer and the score MMAs
// run ahead into the next item while the builders finish the current one; only [O | D] is handed over (the apply
// MMAs of the next item wait until the epilogue has read it).
//
// Warps (384 threads): 0 TMA producer (its lanes also place r into the extra column group), 1 score-MMA
// issuer, 2 apply-MMA issuer, 3 idle, 4-11 weight builders (TMEM lane quadrant = warp % 4, column half =
// (warp - 4) / 4).  All waits are bounded.
#include <cuda.h>
#include <type_traits>

#include "kata_common.cuh"
#include "kata_tmap.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int QT = 128;          // queries per CTA
constexpr int KTILE = 128;       // keys per tile
constexpr int NSTAGE = 4;        // shared-memory stages of (K, V', r) tiles
constexpr int NBUF = 3;          // TMEM score / weight buffers
constexpr int NTHREADS = 384;
constexpr int WARP_BLD0 = 4;

constexpr uint32_t COL_S = 0;    // 3 x 128 fp32 score buffers; the bf16 weights overwrite columns [0,64) of a buffer
constexpr uint32_t COL_O = 384;  // 80 fp32 accumulators: 64 outputs, column 64 = normaliser
constexpr uint32_t TMEM_COLS = 512;

constexpr uint32_t OFF_Q = 0;                       // 2 x (128 x 64 bf16, 128B swizzle): the query tiles of this and the next work item
constexpr uint32_t STAGE_BYTES = 49152;             // K tile 16 KB, V' tile 16 KB, scale-column tile 16 KB
constexpr uint32_t OFF_KV = 32768;                  // NSTAGE stages
constexpr uint32_t OFF_BAR = OFF_KV + NSTAGE * STAGE_BYTES;
constexpr uint32_t OFF_RV = OFF_BAR + 256;          // NSTAGE x 128 bf16: 1 / ||k||^2 of the keys of a tile
constexpr uint32_t SMEM_BYTES = OFF_RV + NSTAGE * 256;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(SMEM_ALLOC > 116 * 1024, "one CTA per SM is assumed (the CTA allocates all of TMEM)");

// Every barrier has waiters that consume each of its phases in order (no waiter skips a phase).
enum {
  BAR_QFULL = 0,     // [2] query tile of a work item landed in shared memory
  BAR_FULL = 2,      // [4] K and V tiles landed (TMA bytes)
  BAR_EMPTY = 6,     // [4] stage free: both issuers' commits
  BAR_SFULL = 10,    // [3] scores in TMEM
  BAR_PFULL = 13,    // [3] weights stored (256 builders)
  BAR_PEMPTY = 16,   // [3] weights consumed by the apply MMA: the buffer may take new scores
  BAR_ODONE = 19,    // the apply MMAs of a work item are complete: [O | D] is final
  BAR_DRAIN = 20,
  BAR_QEMPTY = 21,   // [2] the score MMAs of a work item are complete: its query tile may be replaced
  BAR_OFREE = 23,    // [O | D] of a work item has been read (256 builders): the next item may overwrite it
  BAR_RFULL = 24,    // [4] the key scales of a tile are in shared memory (the scale warp)
  BAR_COUNT = 28
};

// Pre-pass: r = 1 / ||k||^2 per key row (0 for a zero row), one warp per 4 rows (8 lanes x 16 bytes per row).
__global__ void __launch_bounds__(256) quad_rscale_kernel(const __nv_bfloat16* __restrict__ k, __nv_bfloat16* __restrict__ rscale,
                                                          size_t n_rows) {
  const size_t row = (size_t)blockIdx.x * 32 + (threadIdx.x >> 3);
  const int part = threadIdx.x & 7;
  if (row >= n_rows) return;
  const uint4 kraw = *reinterpret_cast<const uint4*>(k + row * D + part * 8);
  const uint32_t kw[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
  float ss = 0.f;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float lo = __uint_as_float(kw[e] << 16), hi = __uint_as_float(kw[e] & 0xFFFF0000u);
    ss = fmaf(lo, lo, ss);
    ss = fmaf(hi, hi, ss);
  }
  ss += __shfl_xor_sync(0xffffffffu, ss, 1);
  ss += __shfl_xor_sync(0xffffffffu, ss, 2);
  ss += __shfl_xor_sync(0xffffffffu, ss, 4);
  if (part == 0) rscale[row] = __float2bfloat16_rn(inv_or_zero(ss));
}

// a pair of bf16 weights times the pair of key scales 1 / ||k||^2
__device__ __forceinline__ uint32_t scale_pair(uint32_t w2, uint32_t r2) {
  const __nv_bfloat162 p = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&w2), *reinterpret_cast<const __nv_bfloat162*>(&r2));
  return *reinterpret_cast<const uint32_t*>(&p);
}

struct QArgs {
  __nv_bfloat16* out;
  const __nv_bfloat16* rscale;   // [BH][T] bf16: 1 / ||k||^2 (pre-pass)
  int* device_status;
  int Tlen;
  int BH, n_qtiles;              // work items: (head, tile of 128 queries), heaviest tiles first
};

// G = feature groups of the blockwise map (Section 3.3): a key tile holds KT = 128 / G keys, and the 128 score
// columns of a buffer hold the G per-group score blocks Q_a K_a^T side by side (group a in columns [a KT, a KT + KT));
// the weight of a key is the sum over the groups of the squared scores.
template <int G>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_quad_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const QArgs args) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  auto bar = [&](int i) { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; };
  auto ktile = [&](int s) { return base + OFF_KV + s * STAGE_BYTES; };
  auto vtile = [&](int s) { return base + OFF_KV + s * STAGE_BYTES + 16384; };
  auto rtile = [&](int s) { return base + OFF_KV + s * STAGE_BYTES + 32768; };   // column group 64..127 of the B operand
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int KT = KTILE / G;                   // keys per tile
  constexpr int KPL = KT / 32;                    // keys per producer lane
  const int n_items = args.BH * args.n_qtiles;
  // work item id -> (head, query tile): the latest query tiles (the most key tiles) come first
  auto item_qtile = [&](int id) { return args.n_qtiles - 1 - id / args.BH; };
  auto item_bh = [&](int id) { return id % args.BH; };
  // the n-th item of this CTA: rounds of gridDim.x items, dealt forwards and backwards in turn, so that the CTA that got
  // the heaviest item of one round gets the lightest of the next
  auto item_id = [&](int n) { return n * (int)gridDim.x + ((n & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x); };

  if (tid == 0) {
    abort_s = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_QFULL + i), 1);
      mbar_init(bar(BAR_QEMPTY + i), 1);
    }
    mbar_init(bar(BAR_OFREE), 256);
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(bar(BAR_FULL + i), 1);
      mbar_init(bar(BAR_RFULL + i), 1);
      mbar_init(bar(BAR_EMPTY + i), 2);
    }
    for (int i = 0; i < NBUF; ++i) {
      mbar_init(bar(BAR_SFULL + i), 1);
      mbar_init(bar(BAR_PFULL + i), G == 1 ? 128 : 256);
      mbar_init(bar(BAR_PEMPTY + i), 1);
    }
    mbar_init(bar(BAR_ODONE), 1);
    mbar_init(bar(BAR_DRAIN), 2);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  // column 64 of the B operand of the apply MMA is a column of ones (the normaliser is the row sum of the weights):
  // the extra column-group tiles are zero except for one bf16 1.0 per key row, written once
  for (int i = tid; i < NSTAGE * 1024; i += NTHREADS)
    *reinterpret_cast<uint4*>(rtile(i >> 10) + (i & 1023) * 16) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  for (int i = tid; i < NSTAGE * 128; i += NTHREADS)
    *reinterpret_cast<uint16_t*>(rtile(i >> 7) + sw128_offset(i & 127, 0)) = (uint16_t)0x3F80;
  fence_async_smem();
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;
  bool ok = true;

  if (warp == 0) {
    // =========================== TMA producer ===========================
    uint32_t it = 0;                                   // key tiles loaded so far, over all items
    int n = 0;
    for (int id = item_id(n); id < n_items && ok; id = item_id(++n)) {
      const int qtile = item_qtile(id), bh = item_bh(id), ntiles = (qtile + 1) * G, qb = n & 1;
      ok = wait_or_abort(bar(BAR_QEMPTY + qb), ((n >> 1) & 1) ^ 1, abort_flag);
      if (!ok) break;
      if (lane == 0) {
        mbar_arrive_expect_tx(bar(BAR_QFULL + qb), 16384);
        tma_load_3d(base + OFF_Q + qb * 16384, &tmQ, bar(BAR_QFULL + qb), 0, qtile * QT, bh);
      }
      for (int j = 0; j < ntiles && ok; ++j, ++it) {
        const int s = it % NSTAGE;
        ok = wait_or_abort(bar(BAR_EMPTY + s), ((it / NSTAGE) & 1) ^ 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          mbar_arrive_expect_tx(bar(BAR_FULL + s), 2 * KT * 128);   // K and V tiles
          tma_load_3d(ktile(s), &tmK, bar(BAR_FULL + s), 0, j * KT, bh);
          tma_load_3d(vtile(s), &tmV, bar(BAR_FULL + s), 0, j * KT, bh);
        }
      }
    }
  } else if (warp == 1) {
    // =========================== score MMA issuer: S = Q K^T ===========================
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, KT);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      uint32_t it = 0;
      int n = 0;
      for (int id = item_id(n); id < n_items && ok; id = item_id(++n)) {
        const int ntiles = (item_qtile(id) + 1) * G, qb = n & 1;
        ok = wait_or_abort(bar(BAR_QFULL + qb), (n >> 1) & 1, abort_flag);
        const uint32_t qa = smem_u32(base + OFF_Q + qb * 16384);
        for (int j = 0; j < ntiles && ok; ++j, ++it) {
          const int s = it % NSTAGE, b = it % NBUF;
          ok = wait_or_abort(bar(BAR_FULL + s), (it / NSTAGE) & 1, abort_flag) &&
               wait_or_abort(bar(BAR_PEMPTY + b), ((it / NBUF) & 1) ^ 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t ka = smem_u32(ktile(s));
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)   // 16 features per step; group ks / (4 / G) accumulates over its own steps
            mma_f16_ss(tb + COL_S + b * 128 + (ks / (4 / G)) * KT, dk + (uint64_t)(((qa + ks * 32) >> 4) & 0x3FFF),
                       dk + (uint64_t)(((ka + ks * 32) >> 4) & 0x3FFF), idesc, (ks % (4 / G)) > 0);
          mma_commit(bar(BAR_SFULL + b));
          mma_commit(bar(BAR_EMPTY + s));
        }
        mma_commit(bar(BAR_QEMPTY + qb));   // (also after a failed wait: the producer is not left waiting)
      }
    }
  } else if (warp == 2) {
    // =========================== apply MMA issuer: [O | D] += P [V' | r] ===========================
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 80);     // A tmem, B MN-major, N = 64 + 16
      // MN-major, 128B swizzle: 8 key rows per 1024-byte atom (SBO), second group of 64 columns 16 KB on (LBO)
      const uint64_t dmn = smem_desc(0, 16384, 1024, kSwizzle128B);
      uint32_t it = 0;
      int n = 0;
      for (int id = item_id(n); id < n_items && ok; id = item_id(++n)) {
        const int ntiles = (item_qtile(id) + 1) * G;
        if (n > 0) ok = wait_or_abort(bar(BAR_OFREE), (n - 1) & 1, abort_flag);   // the epilogue of the item before has read [O | D]
        for (int j = 0; j < ntiles && ok; ++j, ++it) {
          const int s = it % NSTAGE, b = it % NBUF;
          ok = wait_or_abort(bar(BAR_FULL + s), (it / NSTAGE) & 1, abort_flag) &&
               wait_or_abort(bar(BAR_PFULL + b), (it / NBUF) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t va = smem_u32(vtile(s));
#pragma unroll
          for (int ks = 0; ks < KT / 16; ++ks)
            mma_f16_ts(tb + COL_O, tb + COL_S + b * 128 + ks * 8, dmn + (uint64_t)(((va + ks * 2048) >> 4) & 0x3FFF),
                       idesc, (j > 0 || ks > 0) ? 1u : 0u);
          mma_commit(bar(BAR_PEMPTY + b));
          mma_commit(bar(BAR_EMPTY + s));
        }
        mma_commit(bar(BAR_ODONE));
      }
    }
  } else if (warp == 3) {
    // =========================== scale warp: r = 1 / ||k||^2 of the keys of every tile, from the pre-pass to shared memory ===========================
    // (the key scale multiplies the weights, so the values are used as they are; a zero key row has r = 0: zero
    // feature).  The kernel is a programmatic dependent launch behind the pre-pass that computes r: this warp is the
    // only one that reads it, everything else starts at once.
    cudaGridDependencySynchronize();
    uint32_t it = 0;
    int n = 0;
    for (int id = item_id(n); id < n_items && ok; id = item_id(++n)) {
      const int ntiles = (item_qtile(id) + 1) * G;
      const unsigned short* rs = reinterpret_cast<const unsigned short*>(args.rscale) + (size_t)item_bh(id) * args.Tlen;
      auto load_r = [&](int j, unsigned short (&rv)[KPL]) {       // r of this lane's keys of tile j
#pragma unroll
        for (int e = 0; e < KPL; ++e) {
          const int key = j * KT + lane * KPL + e;
          rv[e] = (j < ntiles && key < args.Tlen) ? rs[key] : (unsigned short)0;
        }
      };
      unsigned short rv[KPL];
      load_r(0, rv);
      for (int j = 0; j < ntiles && ok; ++j, ++it) {
        const int s = it % NSTAGE;
        unsigned short rn[KPL];
        load_r(j + 1, rn);              // one tile ahead: the global-load latency stays off the ring
        ok = wait_or_abort(bar(BAR_FULL + s), (it / NSTAGE) & 1, abort_flag);   // (the stage, and with it its r, has been let go of)
        if (!ok) break;
#pragma unroll
        for (int e = 0; e < KPL; ++e) {
          reinterpret_cast<unsigned short*>(base + OFF_RV + s * 256)[lane * KPL + e] = rv[e];
          rv[e] = rn[e];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_RFULL + s));
      }
    }
  } else if (warp >= WARP_BLD0) {
    // =========================== weight builders (256 threads) ===========================
    const uint32_t q4 = warp & 3;
    const int ch = (warp - WARP_BLD0) >> 2;      // column half: keys [64 ch, 64 ch + 64) of the tile
    const int rowl = q4 * 32 + lane;             // query row inside the tile (= TMEM lane)
    uint32_t it = 0;                             // key tiles weighed so far, over all items
    int n = 0;
    for (int id = item_id(n); id < n_items && ok; id = item_id(++n)) {
    const int qtile = item_qtile(id), bh = item_bh(id), ntiles = (qtile + 1) * G;
    const int qrow = qtile * QT + rowl;
    for (int j = 0; j < ntiles && ok; ++j, ++it) {
      const int b = it % NBUF;
      ok = wait_or_abort(bar(BAR_SFULL + b), (it / NBUF) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const bool diag = (j >= ntiles - G);
      if constexpr (G > 1) {
        // this warp weighs keys [ch KT/2, ch KT/2 + KT/2) of the tile: one column run per group
        constexpr int KH = KT / 2;
        const int key0 = j * KT + ch * KH;
        uint32_t y[G][KH], pk[KH / 2];
        ok = wait_or_abort(bar(BAR_RFULL + (it % NSTAGE)), (it / NSTAGE) & 1, abort_flag);
        if (!ok) break;
        const uint32_t* rw = reinterpret_cast<const uint32_t*>(base + OFF_RV + (it % NSTAGE) * 256) + ch * (KH / 2);   // r of this warp's keys, in pairs
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const uint32_t col = tmem_addr(tb, q4 * 32, COL_S + b * 128 + g * KT + ch * KH);
          if constexpr (KH == 32) tmem_ld32(col, y[g]); else tmem_ld16(col, y[g]);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) tmem_wait_ld(y[g]);
        // two copies of the loop, chosen once per tile: the causal test exists on the diagonal tiles only
        auto weigh_g = [&](auto masked) {
#pragma unroll
          for (int c = 0; c < KH; c += 2) {
            float2 w = make_float2(0.f, 0.f);
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const float2 sv = make_float2(__uint_as_float(y[g][c]), __uint_as_float(y[g][c + 1]));
              w = __ffma2_rn(sv, sv, w);
            }
            if constexpr (decltype(masked)::value) {
              if (key0 + c > qrow) w.x = 0.f;
              if (key0 + c + 1 > qrow) w.y = 0.f;
            }
            pk[c / 2] = scale_pair(pack_bf16(w.x, w.y), rw[c / 2]);
          }
        };
        if (diag) weigh_g(std::true_type{}); else weigh_g(std::false_type{});
        // the weights overwrite score columns [0, KT/2) of the buffer (group 0, read by the ch = 0 warp)
        tc_fence_before();
        asm volatile("bar.sync %0, 64;" ::"r"(1 + (int)q4) : "memory");
        tc_fence_after();
        const uint32_t pcol = tmem_addr(tb, q4 * 32, COL_S + b * 128 + ch * (KH / 2));
        if constexpr (KH == 32) tmem_st16(pcol, pk); else tmem_st8(pcol, pk);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_PFULL + b));
        continue;
      }
      // Full lift: the two groups of four warps take alternate tiles (both wait for every tile's scores, so that
      // neither skips a phase of a barrier), and a warp weighs all 128 keys of its 32 query rows: while one group
      // turns the scores of a tile into weights, the MMAs work for the other group's tile.
      if ((it & 1u) != (uint32_t)ch) continue;
      ok = wait_or_abort(bar(BAR_RFULL + (it % NSTAGE)), (it / NSTAGE) & 1, abort_flag);   // (a stage belongs to one group: NSTAGE is even)
      if (!ok) break;
      const uint4* rv4 = reinterpret_cast<const uint4*>(base + OFF_RV + (it % NSTAGE) * 256);   // r of the tile's 128 keys, 8 per load
      const uint32_t scol = tmem_addr(tb, q4 * 32, COL_S + b * 128);
      const int key0 = j * KTILE;
      uint32_t ya[32], yb[32], pk0[32];
      // two copies of the loop, chosen once per tile: the causal test exists on the diagonal tile only
      auto weigh = [&](const uint32_t (&y)[32], uint32_t (&pk)[32], int col0, auto masked) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint4 t4 = rv4[col0 / 8 + i];          // r of 8 keys
          const uint32_t rr[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            const int jj = 8 * i + e, c = col0 + jj;
            const float2 sv = make_float2(__uint_as_float(y[jj]), __uint_as_float(y[jj + 1]));
            float2 w = __fmul2_rn(sv, sv);
            if constexpr (decltype(masked)::value) {
              if (key0 + c > qrow) w.x = 0.f;
              if (key0 + c + 1 > qrow) w.y = 0.f;
            }
            pk[(c & 63) / 2] = scale_pair(pack_bf16(w.x, w.y), rr[e / 2]);
          }
        }
      };
      // The weights overwrite score columns [0,64) of the buffer (this warp's lanes only): those of keys 0..63 once
      // the scores of keys 0..63 are in registers, those of keys 64..127 after.
      auto weigh_tile = [&](auto masked) {
        tmem_ld32(scol, ya);
        tmem_ld32(scol + 32, yb);
        tmem_wait_ld(ya);
        weigh(ya, pk0, 0, masked);
        tmem_wait_ld(yb);
        weigh(yb, pk0, 32, masked);
        tmem_ld32(scol + 64, ya);
        tmem_ld32(scol + 96, yb);
        tmem_st32(scol, pk0);
        tmem_wait_ld(ya);
        tmem_wait_st();                 // pk0 is reused
        weigh(ya, pk0, 64, masked);
        tmem_wait_ld(yb);
        weigh(yb, pk0, 96, masked);
        tmem_st32(scol + 32, pk0);
      };
      if (diag) weigh_tile(std::true_type{}); else weigh_tile(std::false_type{});
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_PFULL + b));
    }
    // ---- epilogue: out = O / D ----
    if (ok) ok = wait_or_abort(bar(BAR_ODONE), n & 1, abort_flag);
    if (ok) {
      tc_fence_after();
      uint32_t o[32], dn[16];
      tmem_ld32(tmem_addr(tb, q4 * 32, COL_O + ch * 32), o);
      tmem_ld16(tmem_addr(tb, q4 * 32, COL_O + 64), dn);
      tmem_wait_ld(o);
      tmem_wait_ld(dn);
      tc_fence_before();
      mbar_arrive(bar(BAR_OFREE));               // the apply MMAs of the next item may overwrite [O | D]
      const float den = __uint_as_float(dn[0]);
      const float inv = den > 0.f ? 1.f / den : 0.f;
      if (qrow < args.Tlen) {
        __nv_bfloat16* dst = args.out + ((size_t)bh * args.Tlen + qrow) * D + ch * 32;
#pragma unroll
        for (int jj = 0; jj < 32; jj += 8) {
          uint4 pkt;
          pkt.x = pack_bf16(__uint_as_float(o[jj]) * inv, __uint_as_float(o[jj + 1]) * inv);
          pkt.y = pack_bf16(__uint_as_float(o[jj + 2]) * inv, __uint_as_float(o[jj + 3]) * inv);
          pkt.z = pack_bf16(__uint_as_float(o[jj + 4]) * inv, __uint_as_float(o[jj + 5]) * inv);
          pkt.w = pack_bf16(__uint_as_float(o[jj + 6]) * inv, __uint_as_float(o[jj + 7]) * inv);
          *reinterpret_cast<uint4*>(dst + jj) = pkt;
        }
      }
    }
    }   // work items
  }

  // ---------------- teardown ----------------
  if (!ok && args.device_status != nullptr) atomicExch(args.device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if ((warp == 1 || warp == 2) && lane == 0) {
    mma_commit(bar(BAR_DRAIN));
    mbar_wait(bar(BAR_DRAIN), 0);
  }
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, TMEM_COLS);
}

}  // namespace

// workspace: r [BH][T] bf16
size_t tc_quadratic_workspace_bytes(const Problem& p) { return ((size_t)p.B * p.H * p.T * 2 + 255) / 256 * 256; }

void tc_quadratic(const Problem& p, void* workspace, int* device_status, LaunchCtx& ctx) {
  const int BH = p.B * p.H;
  __nv_bfloat16* rscale = static_cast<__nv_bfloat16*>(workspace);
  const size_t n_rows = (size_t)BH * p.T;
  quad_rscale_kernel<<<(unsigned)((n_rows + 31) / 32), 256, 0, ctx.stream>>>(static_cast<const __nv_bfloat16*>(p.k), rscale, n_rows);
  note_launch(ctx);
  CUtensorMap tmQ, tmK, tmV;
  const int kt = KTILE / p.groups;
  if (!make_tile_map(&tmQ, p.q, BH, p.T, QT) || !make_tile_map(&tmK, p.k, BH, p.T, kt) || !make_tile_map(&tmV, p.v, BH, p.T, kt)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  auto kern = p.groups == 1 ? tc_quad_kernel<1> : p.groups == 2 ? tc_quad_kernel<2> : tc_quad_kernel<4>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  const int n_qtiles = (p.T + QT - 1) / QT;
  QArgs a{static_cast<__nv_bfloat16*>(p.out), rscale, device_status, p.T, BH, n_qtiles};
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    sms = 148;
  }
  const long long n_items = (long long)BH * n_qtiles;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_items < sms ? n_items : sms));   // persistent: one CTA per SM, items dealt round-robin
  cfg.blockDim = dim3(NTHREADS);
  cfg.dynamicSmemBytes = SMEM_ALLOC;
  cfg.stream = ctx.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, tmV, a) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  ++ctx.launches;
}

}  // namespace kata
