// Chunked (linear-state) KATA forward on the Blackwell tensor cores with the FEATURE axis of the state split over
// the CTAs of a head (bf16, d_k = d_v = 64, sequential inter-chunk recurrence, whole sequence in one pass).
//
// Algorithm 1 / section "Chunkwise forward", with the rank-one lift psi(u) = u u^T written as 8 x 8 blocks: the 64
// features of a row are cut into 8 runs of 8, and a "block pair" (g, h), g <= h, is the 64 products
// u[8g+i] u[8h+j].  <psi(q), psi(k)> = (q.k)^2 = sum over the 36 block pairs of w_gh <Q_gh, K_gh> with w = 1 on
// the diagonal pairs (which hold both (i,j) and (j,i)) and w = 2 off it.  One CTA owns 4 block pairs = 256 state
// rows (two M = 128 accumulator tiles S[m], 80 fp32 TMEM columns each: 64 value columns, the normaliser column,
// padding); nine CTAs make a head; they meet only through the shares they publish.  With the key scale r = 1/||k||^2
// folded into the values (V' = r V, written once per head by a light pre-pass) and the normaliser carried as column
// 64 of every B operand, per tile of 128 tokens a CTA does
//   update   S[m] += Psi(K)_m^T [V' | r]      A = the products, built by token threads in shared memory (MN-major),
//                                             B = the TMA-loaded tile of scaled values, N = 80
//   snapshot B_m = bf16(S[m])                 TMEM -> shared memory, the B operand of the next tile's read
//   read     ACC  = Psi(Q)_m [S | Z]_m        A = the weighted query products in TMEM, N = 80
//   intra    ACC += P_c [V' | r]_c            P_c = (Q K_c^T)^2 masked causally for the 16 keys c of the tile this
//                                             CTA owns (the eight 16-key runs of a tile go to eight of the CTAs)
// ACC is this CTA's share of [N | D] of the tile's 128 queries.  The share is staged in shared memory (numerators as
// fp16 with a power-of-two scale per row, normaliser in fp32) and goes to global memory as one bulk copy per tile; a
// counter per head and tile, released at GPU scope once the copy is complete, tells the other CTAs of the head that it
// is there.  Each CTA finishes 15 of the 128 query rows of a tile (the ninth: 8): it adds the nine shares of those
// rows, which it finds in L2, applies the gate/normalise step out = N / D (0 where D = 0) and writes the output.  The
// query norm cancels between N and D and is never applied.  Heads are dealt to CTAs by a ticket taken when a CTA
// starts, so that the CTAs a CTA waits for are running or next in line whatever order blocks are dispatched in.
//
// The tiles are walked in lockstep.  Tile j is two phases:
//   A  everything the MMAs of the tile read is put in place: key products (key teams), weighted query products and
//      the intra-tile weights (query team, after the score MMA), the snapshot of the state after tile j - 1 (state
//      team); one named barrier ends the phase;
//   B  the update, read and apply MMAs of the tile are issued back to back by two threads (two independent
//      accumulation chains in the pipe at a time) and commit to one mbarrier, which every team waits for before it
//      touches its buffers again.  Under phase B the share team stages the share of tile j - 1 and the TMA producer
//      refills the key/query stage that phase A emptied.
// Two synchronisations per tile instead of a web of point-to-point hand-offs: a hand-off between warps costs several
// hundred cycles from arrival to the waiter's next instruction, and a pipeline whose buffers are all single (shared
// memory and TMEM are full) turns each of them into a round trip; a version of this kernel built that way spent
// 5 k cycles per tile on synchronisation alone.
//
// Blockwise map (section "KATA-Mg", g = 2 or 4 feature groups): only the block pairs inside a group carry state (20
// or 12 of the 36), the intra-tile weights are the sum over the groups of the squared per-group scores, and a head is
// cut differently: the kernel is a template over (accumulator tiles per CTA, groups, CTAs per head) = (2, 1, 9) for
// the full lift, (1, 2, 10) or (2, 2, 5) for two groups, (1, 4, 6) for four.  With fewer than eight CTAs per head a
// CTA weighs two of the eight key runs of a tile.  Each CTA finishes ceil(128 / CTAs per head) query rows of a tile.
//
// Warps (896 threads): 0 TMA producer, 1 update issuer, 2 read issuer, 3 score issuer; 4-11 key teams (team m builds
// the products of accumulator tile m; team 0 also places r); 12-15 query team; 16-19 state team; 20-23 share team;
// 24-27 combine team (its last thread issues the bulk copies and publishes the tiles).  Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kata_common.cuh"
#include "kata_tmap.cuh"
#include "kata_umma.cuh"

#ifndef KATA_SPLIT_PROF
#define KATA_SPLIT_PROF 0
#endif

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int CT = 128;            // tokens per tile
// CTAs of a head (template parameter NCTA): 36 block pairs / 4 (full lift), 20 / 4 or 20 / 2 (two feature groups), 12 / 2 (four)
constexpr int BP_MAX = 40;
constexpr int NTHREADS = 896;
constexpr int kPrefetchTiles = 4;    // tiles between a tile's L2 prefetch and its load
constexpr int kRowSlots = 15;        // query rows of a tile the combine team finishes per pass (8 threads each)
constexpr int W_TMA = 0, W_U = 1, W_R = 2, W_I = 3, W_K0 = 4, W_Q0 = 12, W_S0 = 16, W_E0 = 20, W_O0 = 24;

// ---- TMEM columns; NM = accumulator tiles (of 128 state rows = 2 block pairs) per CTA ----
constexpr uint32_t COL_S = 0;      // NM x 80: state tiles (lanes = state rows)
constexpr uint32_t COL_ACC = 288;  // 2 x 80: this CTA's share of [N | D] (lanes = tokens), double-buffered
// weighted query products as bf16 pairs (lanes = tokens), 32 columns per block pair
template <int NM> struct Cols { static constexpr uint32_t PSIQ = NM == 2 ? 160u : 208u, SC = NM == 2 ? 448u : 80u; };
// fp32 scores, 16 columns per (key run, feature group); the bf16 weights of a run overwrite the start of its scores
// (at most 4 (run, group) tiles = 64 columns with two accumulator tiles, 8 = 128 columns with one)
constexpr uint32_t TMEM_COLS = 512;

// ---- shared memory (1024-byte aligned tiles of 128-byte rows, 128B swizzle) ----
constexpr uint32_t OFF_PSIK = 0;        // 4 block pairs x [128 tokens][64 products]
constexpr uint32_t OFF_KRAW = 65536;    // 2 x key tile
constexpr uint32_t OFF_QRAW = 98304;    // 2 x query tile
constexpr uint32_t OFF_VP = 131072;     // 2 x tile of scaled values
constexpr uint32_t OFF_SNAP = 163840;   // 2 x [128 state rows][64 values] bf16
constexpr uint32_t OFF_COL64 = 196608;  // column 64 of the four B operands above: 32 bytes of every row each
constexpr uint32_t OFF_BAR = 212992;
constexpr uint32_t OFF_MISC = OFF_BAR + 256;
constexpr uint32_t OFF_STG = OFF_MISC + 128;      // this CTA's share of a tile as it goes to global memory
constexpr uint32_t kShareBytes = CT * 128 + CT * 8;
constexpr uint32_t SMEM_BYTES = OFF_STG + kShareBytes;
static_assert(OFF_STG % 128 == 0, "staging tile");
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(SMEM_ALLOC <= 232448, "shared memory");

// Every barrier has waiters that consume each of its phases in order.
enum {
  B_K_FULL = 0,      // [2] key tile landed
  B_Q_FULL = 2,      // [2] query tile landed
  B_V_FULL = 4,      // [2] tile of scaled values landed
  B_SC_FULL = 6,     // [2] intra-tile scores in TMEM
  B_MMA_DONE = 8,    // update, read and apply MMAs of a tile complete (two commits)
  B_ACC_FULL = 9,    // [2] read and apply MMAs of a tile complete: its share is in TMEM buffer tile & 1
  B_ACC_FREE = 11,   // [2] ... and has been copied out of it (128 threads of the share team)
  B_STG_FULL = 13,   // [2] the share of a tile is staged (128 threads of the share team); one barrier per store thread
  B_STG_FREE = 15,   // the bulk store has read the staging tile
  B_A_DONE = 16,     // phase A of a tile is complete (16 warps)
  B_DRAIN = 17,
  B_COUNT = 18
};
static_assert(B_COUNT * 8 <= 256, "barrier block");
constexpr int kBarA = 2;                    // named barrier that ends phase A (full lift)
constexpr int kBarAThreads = 32 * 19;       // TMA producer, update and read issuers, key, query and state teams

struct BlockPairs {
  unsigned char g[BP_MAX], h[BP_MAX], w[BP_MAX];
};

struct SplitArgs {
  __nv_bfloat16* out;
  const __nv_bfloat16* rscale;   // [BH][T] bf16: 1 / ||k||^2 (pre-pass)
  unsigned char* share;          // [BH][ncta][ntiles] blocks: [128 rows][64 fp16 numerators / scale, 16-byte pieces swizzled by row] | [128][normaliser, scale] fp32
  unsigned* counter;             // [BH][ntiles]: CTAs of the head that have written their share of the tile
  int* device_status;
  int T, ntiles;
  int ncta;                      // CTAs per head
  int groups;                    // feature groups of the blockwise map (1 = the full lift)
  long long* prof;               // profiling build only: [CTA][5 teams][8] cycle counts
  BlockPairs bp;
};

// Shared-memory accesses of buffers that other agents refill (TMA, MMA operands): by address in the shared window.
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(saddr) : "memory");
  return r;
}
__device__ __forceinline__ void sts128(uint32_t saddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t saddr, unsigned short v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(saddr), "h"(v) : "memory");
}

// Bounded waits on plain counters (the phases of an mbarrier cannot be used where the waiter may fall several tiles
// behind).  The wait on a counter of the head lasts as long as the slowest CTA of the head needs, which may be one
// that has not started yet: its limit is 2 s of wall time.
__device__ __forceinline__ bool wait_count_global(const unsigned* p, unsigned want, volatile int* abort_flag) {
  unsigned t0 = 0;
  for (uint32_t i = 0;; ++i) {
    unsigned v, t1;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    if (v >= want) return true;
    if (*abort_flag) return false;
    asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t1));
    if (i == 0) t0 = t1;
    if (t1 - t0 > 2000000000u) break;
    __nanosleep(128);
  }
  *abort_flag = 1;
  return false;
}

// Register budget per warp group (the kernel is launched with 72 registers per thread for 896 threads): the four
// issuer warps and the key teams give registers up, the teams that hold tiles of TMEM in registers take them.
template <int N> __device__ __forceinline__ void regs_release() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_take() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
static_assert(128 * 48 + 256 * 56 + 384 * 88 + 128 * 80 <= 896 * 72, "register budget");

// 64 products a[i] b[j] (i, j < 8) of two runs of 8 bf16 (4 words each), scaled by the bf16 pair `wgt` if SCALED, as
// 8 chunks of 8 bf16 (chunk i = a[i] * b[0..7]).  One rounding per product (the scale is 1 or 2).
template <bool SCALED>
__device__ __forceinline__ void products8x8(const uint32_t (&a)[4], const uint32_t (&b)[4], uint32_t wgt, uint32_t (&out)[32]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t ai = __byte_perm(a[i >> 1], 0u, (i & 1) ? 0x3232 : 0x1010);   // a[i] in both halves
    __nv_bfloat162 s = *reinterpret_cast<const __nv_bfloat162*>(&ai);
    if (SCALED) s = __hmul2(s, *reinterpret_cast<const __nv_bfloat162*>(&wgt));
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      __nv_bfloat162 pr = __hmul2(s, *reinterpret_cast<const __nv_bfloat162*>(&b[c]));
      out[i * 4 + c] = *reinterpret_cast<uint32_t*>(&pr);
    }
  }
}

// Pre-pass: V' = v / ||k||^2 (bf16) and r = 1 / ||k||^2 (bf16), so that the key scale is applied once per head and not
// once in each of the nine CTAs of a head.  One warp per 4 key rows (8 lanes x 16 bytes per row).
__global__ void __launch_bounds__(256) split_prescale_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                                                             __nv_bfloat16* __restrict__ vs, __nv_bfloat16* __restrict__ rscale,
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
  const float r2 = inv_or_zero(ss);
  const uint4 vraw = *reinterpret_cast<const uint4*>(v + row * D + part * 8);
  uint4 sc;
  sc.x = pack_bf16(__uint_as_float(vraw.x << 16) * r2, __uint_as_float(vraw.x & 0xFFFF0000u) * r2);
  sc.y = pack_bf16(__uint_as_float(vraw.y << 16) * r2, __uint_as_float(vraw.y & 0xFFFF0000u) * r2);
  sc.z = pack_bf16(__uint_as_float(vraw.z << 16) * r2, __uint_as_float(vraw.z & 0xFFFF0000u) * r2);
  sc.w = pack_bf16(__uint_as_float(vraw.w << 16) * r2, __uint_as_float(vraw.w & 0xFFFF0000u) * r2);
  *reinterpret_cast<uint4*>(vs + row * D + part * 8) = sc;
  if (part == 0) rscale[row] = __float2bfloat16_rn(r2);
}

template <int NM, int G, int NCTA>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_split_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ SplitArgs args) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  auto bar = [&](int i) { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; };
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(base + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base + OFF_MISC + 4);
  volatile unsigned* ticket_s = reinterpret_cast<volatile unsigned*>(base + OFF_MISC + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ntiles = args.ntiles;

  if (tid == 0) {
    *abort_flag = 0;
    *ticket_s = atomicAdd(args.counter + (size_t)gridDim.x / NCTA * args.ntiles, 1u);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_K_FULL + i), 1);
      mbar_init(bar(B_Q_FULL + i), 1);
      mbar_init(bar(B_V_FULL + i), 1);
      mbar_init(bar(B_SC_FULL + i), 1);
      mbar_init(bar(B_ACC_FULL + i), 1);
      mbar_init(bar(B_ACC_FREE + i), 128);
      mbar_init(bar(B_STG_FULL + i), 128);
    }
    mbar_init(bar(B_MMA_DONE), 2);
    mbar_init(bar(B_STG_FREE), 1);
    mbar_init(bar(B_A_DONE), 16);
    mbar_init(bar(B_DRAIN), 2);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  // column 64 of the B operands: zero except one bf16 per row and operand
  const uint32_t sbase = smem_u32(base);
  for (int i = tid; i < 1024; i += NTHREADS) sts128(sbase + OFF_COL64 + i * 16, 0u, 0u, 0u, 0u);
  fence_async_smem();
  if (warp == 0) {
    tmem_alloc(tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = *tmem_base_s;
  // Heads are dealt out in the order the CTAs start, not by block index: a CTA waits (combine team) for the shares of
  // the other eight CTAs of its head, and with tickets those are running or next in line whatever order the blocks
  // are dispatched in.
  const unsigned ticket = *ticket_s;
  constexpr int NBP = 2 * NM;                                 // block pairs of this CTA
  constexpr uint32_t COL_PSIQ = Cols<NM>::PSIQ, COL_SC = Cols<NM>::SC;
  constexpr int ncta = NCTA;
  constexpr int MAXRUN = NCTA < 8 ? 2 : 1;                     // key runs a CTA can have
  // With one run and one group the scores are double-buffered and the weights have columns of their own, so that the
  // scores of a tile can be issued as soon as its keys and queries have landed; otherwise one buffer, the weights
  // over the start of the scores, and the score MMAs wait for the apply MMA of the tile before.
  constexpr bool SC2 = MAXRUN == 1 && G == 1;
  constexpr int kRowsPerCta = (CT + NCTA - 1) / NCTA;          // query rows of a tile this CTA finishes
  constexpr uint32_t COL_P = 480;
  const int bh = (int)(ticket / ncta);
  const int cta_head = (int)(ticket % ncta);                  // CTA of the head
  // The eight 16-key runs of a tile are dealt round-robin to the CTAs of the head: run cta_head, and run
  // cta_head + ncta where that is still below 8 (heads of fewer than eight CTAs).
  const int nrun = (cta_head < 8 ? 1 : 0) + (cta_head + ncta < 8 ? 1 : 0);
  const bool has_intra = nrun > 0;
  bool ok = true;
#if KATA_SPLIT_PROF
  long long pacc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, plast = clock64();
#define TICK(slot) do { long long c_ = clock64(); pacc[slot] += c_ - plast; plast = c_; } while (0)
#define TOCK(team) do { if (lane == 0) for (int i_ = 0; i_ < 8; ++i_) args.prof[((size_t)ticket * 5 + team) * 8 + i_] = pacc[i_]; } while (0)
#else
#define TICK(slot)
#define TOCK(team)
#endif
  // Every lane of a warp waits for itself: one lane waiting for the others (and a shuffle to tell them) wakes the warp
  // later than 32 waiters do.
  auto wwait = [&](int b, uint32_t parity) { return wait_or_abort_counted(bar(b), parity, abort_flag); };
  // the wait that opens tile j + 1 for every team: the MMAs of tile j are complete
  auto mma_done = [&](int j) { return j < 0 ? true : wwait(B_MMA_DONE, j & 1); };
  // End of phase A.  Two forms, chosen by measurement (c4, ms: full lift 3.34 / 3.73, two groups 3.63 / 2.99, four
  // groups 3.05 / 3.03): a named barrier that the issuers, the TMA producer and the sixteen warps of the key, query
  // and state teams all wait at, or an mbarrier on which the teams only arrive (and go on to wait for the MMAs) and
  // for which only the issuers and the producer wait.  A team that gave up keeps arriving in both.
  constexpr bool kArriveOnly = G != 1;
  constexpr bool kRollIssue = G != 1;
  auto phase_a_arrive = [&]() {
    if (kArriveOnly) {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_A_DONE));
    } else {
      asm volatile("bar.sync %0, %1;" ::"n"(kBarA), "n"(kBarAThreads) : "memory");
    }
  };
  auto phase_a_wait = [&](int j) {
    if (kArriveOnly) return wwait(B_A_DONE, j & 1);
    asm volatile("bar.sync %0, %1;" ::"n"(kBarA), "n"(kBarAThreads) : "memory");
    return true;
  };
  // A staged share goes to global memory as one bulk copy, issued by one thread; once the copy of the tile before is
  // complete that tile is published (a counter per head and tile, released at GPU scope).  The release waits for
  // memory operations of the whole SM that are in flight, the loads of the combine team among them; the share team
  // only ever waits for a copy to have read the staging tile.
  auto store_thread = [&]() {
    unsigned char* mine = args.share + ((size_t)bh * ncta + cta_head) * ntiles * kShareBytes;
    unsigned* cnt = args.counter + (size_t)bh * ntiles;
    int prev = -1;
    for (int j = 0; j < ntiles; ++j) {
      ok = wait_or_abort_counted(bar(B_STG_FULL + (j & 1)), (j >> 1) & 1, abort_flag);
      if (!ok) break;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n\tcp.async.bulk.commit_group;\n\t"
                   "cp.async.bulk.wait_group.read 0;" ::"l"(mine + (size_t)j * kShareBytes), "r"(sbase + OFF_STG), "n"(kShareBytes)
                   : "memory");
      mbar_arrive(bar(B_STG_FREE));
      if (prev >= 0) {
        asm volatile("cp.async.bulk.wait_group 1;" ::: "memory");
        asm volatile("fence.acq_rel.gpu;\n\tred.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(cnt + prev) : "memory");
      }
      prev = j;
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (prev >= 0) asm volatile("fence.acq_rel.gpu;\n\tred.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(cnt + prev) : "memory");
  };

  if (warp < W_K0) {
    regs_release<48>();
    if (warp == W_TMA) {
      // =========================== TMA producer ===========================
      auto load = [&](int what, uint32_t off, const CUtensorMap* tm, int j) {
        const int s = j & 1;
        mbar_arrive_expect_tx(bar(what + s), 16384);
        tma_load_3d(base + off + s * 16384, tm, bar(what + s), 0, j * CT, bh);
      };
      // One CTA of the head asks L2 for each tensor's tile a few tiles ahead: the nine CTAs of a head read the same
      // tiles, and a tile that comes from DRAM arrives later than the two stages of shared memory can hide.
      auto prefetch = [&](int j) {
        if (cta_head < 3 && j < ntiles)
          asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(cta_head == 0 ? &tmK : cta_head == 1 ? &tmQ : &tmV),
                       "r"(0), "r"(j * CT), "r"(bh)
                       : "memory");
      };
      if (lane == 0) {
        for (int j = 0; j < 2 && j < ntiles; ++j) {
          load(B_K_FULL, OFF_KRAW, &tmK, j);
          load(B_Q_FULL, OFF_QRAW, &tmQ, j);
          load(B_V_FULL, OFF_VP, &tmV, j);
        }
        for (int j = 2; j < 2 + kPrefetchTiles; ++j) prefetch(j);
      }
      for (int j = 0; j < ntiles; ++j) {
        ok = ok && phase_a_wait(j);                 // keys and queries of tile j have been read (teams) and multiplied (score MMA)
        if (j + 2 < ntiles) {
          if (lane == 0 && ok) {
            load(B_K_FULL, OFF_KRAW, &tmK, j + 2);
            load(B_Q_FULL, OFF_QRAW, &tmQ, j + 2);
            prefetch(j + 2 + kPrefetchTiles);
          }
          ok = ok && mma_done(j);       // the MMAs of tile j are done with the value tile
          if (lane == 0 && ok) load(B_V_FULL, OFF_VP, &tmV, j + 2);
        }
      }
    } else if (warp == W_U) {
      // =========================== update issuer ===========================
      // After phase A of tile j: the update S[m] += Psi(K)_m^T [V' | r].
      const uint32_t idesc_u = instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 80);
      const uint64_t da = smem_desc(0, 16384, 1024, kSwizzle128B);      // second run of 64 state rows: next block pair
      for (int j = 0; j < ntiles; ++j) {
        const int b = j & 1;
        ok = ok && wwait(B_V_FULL + b, (j >> 1) & 1);
        TICK(0);
        ok = ok && phase_a_wait(j);
        TICK(1);
        if (lane == 0) {
          if (ok) {
            tc_fence_after();
            const uint32_t vp = sbase + OFF_VP + b * 16384;
            const uint64_t dbv = smem_desc(0, sbase + OFF_COL64 + 32 * b - vp, 1024, kSwizzle128B);
#pragma unroll
            for (int m = 0; m < NM; ++m) {
              const uint32_t pa = sbase + OFF_PSIK + m * 32768;
              // (whether these loops are unrolled changes how the update and the read chains interleave in the pipe:
              // c4, ms, unrolled / rolled: full lift 3.35 / 3.70, two groups 3.90 / 2.99, four groups 3.08 / 3.03)
              if (kRollIssue) {
#pragma unroll 1
                for (int ks = 0; ks < 8; ++ks)
                  mma_f16_ss(tb + COL_S + m * 80, at(da, pa + ks * 2048), at(dbv, vp + ks * 2048), idesc_u, (j > 0 || ks > 0) ? 1u : 0u);
              } else {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                  mma_f16_ss(tb + COL_S + m * 80, at(da, pa + ks * 2048), at(dbv, vp + ks * 2048), idesc_u, (j > 0 || ks > 0) ? 1u : 0u);
              }
            }
          }
          mma_commit(bar(B_MMA_DONE));
        }
        __syncwarp();
        TICK(2);
      }
      TOCK(0);
    } else if (warp == W_R) {
      // =========================== read issuer: ACC = Psi(Q) [S | Z] + sum over this CTA's key runs c of P_c [V' | r]_c ===========================
      const uint32_t idesc_r = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 80);
      for (int j = 0; j < ntiles; ++j) {
        const int b = j & 1;
        if (has_intra) ok = ok && wwait(B_V_FULL + b, (j >> 1) & 1);
        if (j >= 2) ok = ok && wwait(B_ACC_FREE + b, ((j >> 1) - 1) & 1);          // share of tile j - 2 copied out
        ok = ok && phase_a_wait(j);
        if (lane == 0) {
          if (ok) {
            tc_fence_after();
            if (j >= 1) {
#pragma unroll
              for (int m = 0; m < NM; ++m) {
                const uint32_t sn = sbase + OFF_SNAP + m * 16384;
                const uint64_t db = smem_desc(0, sbase + OFF_COL64 + 32 * (2 + m) - sn, 1024, kSwizzle128B);
                if (kRollIssue) {
#pragma unroll 1
                  for (int ks = 0; ks < 8; ++ks)
                    mma_f16_ts(tb + COL_ACC + b * 80, tb + COL_PSIQ + m * 64 + ks * 8, at(db, sn + ks * 2048), idesc_r, (m > 0 || ks > 0) ? 1u : 0u);
                } else {
#pragma unroll
                  for (int ks = 0; ks < 8; ++ks)
                    mma_f16_ts(tb + COL_ACC + b * 80, tb + COL_PSIQ + m * 64 + ks * 8, at(db, sn + ks * 2048), idesc_r, (m > 0 || ks > 0) ? 1u : 0u);
                }
              }
            }
            if (has_intra) {
              const uint32_t vp = sbase + OFF_VP + b * 16384;
              const uint64_t dbv = smem_desc(0, sbase + OFF_COL64 + 32 * b - vp, 1024, kSwizzle128B);
#pragma unroll
              for (int r = 0; r < MAXRUN; ++r)   // the weights of run r sit at the start of its scores
                if (r < nrun) mma_f16_ts(tb + COL_ACC + b * 80, SC2 ? tb + COL_P : tb + COL_SC + r * G * 16, at(dbv, vp + (cta_head + r * ncta) * 2048), idesc_r,
                           (j >= 1 || r > 0) ? 1u : 0u);
            }
          }
          mma_commit(bar(B_ACC_FULL + b));
          mma_commit(bar(B_MMA_DONE));
        }
        __syncwarp();
      }
    } else {
      // =========================== score issuer: Q_g K_c,g^T per feature group g for this CTA's key runs c (opens phase A) ===========================
      const uint32_t idesc_s = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 16);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      for (int j = 0; j < ntiles; ++j) {
        if (has_intra) {
          const int s = j & 1;
          const uint32_t qa = sbase + OFF_QRAW + s * 16384;
          if (!SC2) ok = ok && mma_done(j - 1);   // the apply MMA of tile j - 1 has read the weights; their columns take the scores
          ok = ok && wwait(B_K_FULL + s, (j >> 1) & 1) && wwait(B_Q_FULL + s, (j >> 1) & 1);
          if (lane == 0) {
            if (ok) {
              tc_fence_after();
              // per key run and feature group: the 64 / G features of the group in steps of 16
              constexpr int ksg = 4 / G;
#pragma unroll
              for (int r = 0; r < MAXRUN; ++r) {
                if (r < nrun) {
                  const uint32_t ka = sbase + OFF_KRAW + s * 16384 + (cta_head + r * ncta) * 2048;
#pragma unroll
                  for (int ks = 0; ks < 4; ++ks)
                    mma_f16_ss(tb + COL_SC + (SC2 ? s : r * G + ks / ksg) * 16, at(dk, qa + ks * 32), at(dk, ka + ks * 32), idesc_s, (ks % ksg) > 0 ? 1u : 0u);
                }
              }
            }
            mma_commit(bar(B_SC_FULL + s));
          }
          __syncwarp();
        }

      }
    }
  } else if (warp < W_Q0) {
    regs_release<56>();
    // =========================== key teams (thread = token; a team of four warps builds NM of the block pairs) ===========================
    const int m = (warp - W_K0) >> 2;   // team: with two accumulator tiles, tile m; with one, its block pair m
    const int t = ((warp - W_K0) & 3) * 32 + lane;
    int pg[NM], ph[NM];
#pragma unroll
    for (int e = 0; e < NM; ++e) {
      pg[e] = args.bp.g[cta_head * NBP + NM * m + e];
      ph[e] = args.bp.h[cta_head * NBP + NM * m + e];
    }
    const unsigned short* rs = reinterpret_cast<const unsigned short*>(args.rscale) + (size_t)bh * args.T;
    unsigned short r_next = (m == 0 && t < args.T) ? rs[t] : (unsigned short)0;
    for (int j = 0; j < ntiles; ++j) {
      const int b = j & 1;
      const uint32_t kraw = sbase + OFF_KRAW + b * 16384;
      ok = ok && wwait(B_K_FULL + b, (j >> 1) & 1);
      TICK(0);
      ok = ok && mma_done(j - 1);       // the update of tile j - 1 has read the products (and column 64 of its values)
      TICK(1);
      if (ok) {
        if (m == 0) {                   // column 64 of the value operand: r of this token
          sts16(sbase + OFF_COL64 + sw128_offset(t, 2 * b), r_next);
          const int tn = (j + 1) * CT + t;
          r_next = (j + 1 < ntiles && tn < args.T) ? rs[tn] : (unsigned short)0;
        }
#pragma unroll
        for (int e = 0; e < NM; ++e) {
          const uint4 ra = lds128(kraw + sw128_offset(t, pg[e]));
          const uint4 rb = lds128(kraw + sw128_offset(t, ph[e]));
          const uint32_t ga[4] = {ra.x, ra.y, ra.z, ra.w}, gb[4] = {rb.x, rb.y, rb.z, rb.w};
          uint32_t pr[32];
          products8x8<false>(ga, gb, 0u, pr);
          const uint32_t dst = sbase + OFF_PSIK + (NM * m + e) * 16384;
#pragma unroll
          for (int i = 0; i < 8; ++i) sts128(dst + sw128_offset(t, i), pr[4 * i], pr[4 * i + 1], pr[4 * i + 2], pr[4 * i + 3]);
        }
        fence_async_smem();
      }
      TICK(2);
      phase_a_arrive();
      TICK(3);
    }
    if (warp == W_K0) TOCK(1);
  } else if (warp < W_S0) {
    regs_take<88>();
    // =========================== query team (thread = token): weighted query products, intra-tile weights ===========================
    const uint32_t q4 = warp & 3;
    const int t = q4 * 32 + lane;
    int pg[NBP], ph[NBP];
    uint32_t pw[NBP];
#pragma unroll
    for (int e = 0; e < NBP; ++e) {
      pg[e] = args.bp.g[cta_head * NBP + e];
      ph[e] = args.bp.h[cta_head * NBP + e];
      pw[e] = args.bp.w[cta_head * NBP + e] == 1 ? 0x3F803F80u : 0x40004000u;
    }
    for (int j = 0; j < ntiles; ++j) {
      const int b = j & 1;
      const uint32_t qraw = sbase + OFF_QRAW + b * 16384;
      ok = ok && wwait(B_Q_FULL + b, (j >> 1) & 1);
      TICK(0);
      ok = ok && mma_done(j - 1);       // the read of tile j - 1 has used the products, its apply the weights
      TICK(1);
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int e = 0; e < NBP; ++e) {
          const uint4 ra = lds128(qraw + sw128_offset(t, pg[e]));
          const uint4 rb = lds128(qraw + sw128_offset(t, ph[e]));
          const uint32_t ga[4] = {ra.x, ra.y, ra.z, ra.w}, gb[4] = {rb.x, rb.y, rb.z, rb.w};
          uint32_t pr[32];
          products8x8<true>(ga, gb, pw[e], pr);
          tmem_st32(tmem_addr(tb, q4 * 32, COL_PSIQ + e * 32), pr);
        }
      }
      TICK(2);
      if (has_intra) {                  // weights P_c = sum_g (Q_g K_c,g^T)^2, causal inside the tile
        ok = ok && wwait(B_SC_FULL + b, (j >> 1) & 1);
        TICK(3);
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int r = 0; r < MAXRUN; ++r) {        // w = sum over the feature groups of (q_g . k_g)^2, masked
            if (r >= nrun) break;
            float w[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) w[c] = 0.f;
#pragma unroll
            for (int a = 0; a < G; ++a) {
              uint32_t y[16];
              tmem_ld16(tmem_addr(tb, q4 * 32, COL_SC + (SC2 ? b : r * G + a) * 16), y);
              tmem_wait_ld(y);
#pragma unroll
              for (int c = 0; c < 16; ++c) w[c] = fmaf(__uint_as_float(y[c]), __uint_as_float(y[c]), w[c]);
            }
            const int key0 = (cta_head + r * ncta) * 16;
            uint32_t pk[8];
#pragma unroll
            for (int c = 0; c < 16; c += 2) pk[c >> 1] = pack_bf16(key0 + c <= t ? w[c] : 0.f, key0 + c + 1 <= t ? w[c + 1] : 0.f);
            tmem_st8(tmem_addr(tb, q4 * 32, SC2 ? COL_P : COL_SC + r * G * 16), pk);   // (over the scores just read, unless the weights have their own columns)
          }
        }
      }
      tmem_wait_st();
      tc_fence_before();
      TICK(4);
      phase_a_arrive();
      TICK(5);
    }
    if (warp == W_Q0) TOCK(2);
  } else if (warp < W_E0) {
    regs_take<88>();
    // =========================== state team (thread = state row of both accumulator tiles) ===========================
    const uint32_t q4 = warp & 3;
    const int f = q4 * 32 + lane;
    for (int j = 0; j < ntiles; ++j) {
      ok = ok && mma_done(j - 1);       // the update of tile j - 1 is complete, and so is the read that used the old snapshot
      TICK(0);
      if (ok && j >= 1) {
        tc_fence_after();
#pragma unroll
        for (int m = 0; m < NM; ++m) {
          uint32_t pk[32], zc[4];
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            uint32_t y[16];
            tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + m * 80 + h * 16), y);
            if (h == 3) tmem_ld4(tmem_addr(tb, q4 * 32, COL_S + m * 80 + 64), zc);
            tmem_wait_ld(y);
#pragma unroll
            for (int c = 0; c < 8; ++c) pk[h * 8 + c] = pack_bf16(__uint_as_float(y[2 * c]), __uint_as_float(y[2 * c + 1]));
          }
          tmem_wait_ld(zc);
          const uint32_t snap = sbase + OFF_SNAP + m * 16384;
#pragma unroll
          for (int c = 0; c < 8; ++c) sts128(snap + sw128_offset(f, c), pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
          sts16(sbase + OFF_COL64 + sw128_offset(f, 2 * (2 + m)), __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(zc[0]))));
        }
        tc_fence_before();
        fence_async_smem();
      }
      TICK(1);
      phase_a_arrive();
      TICK(2);
    }
    if (warp == W_S0) TOCK(3);
  } else if (warp < W_O0) {
    regs_take<88>();
    // =========================== share team (thread = token): this CTA's [N | D] of a tile, staged for the bulk store ===========================
    // Outside the lockstep: it follows the MMA issuer through a pair of barriers per accumulator buffer.  The team
    // touches no global memory: a store it had to see completed before the tile could be published would put a trip
    // to L2 into every iteration, and the MMA issuer waits for this team before it reuses an accumulator buffer.
    const uint32_t q4 = warp & 3;
    const int t = q4 * 32 + lane;
    const uint32_t stg = sbase + OFF_STG;
    for (int j = 0; j < ntiles; ++j) {
      const int b = j & 1;
      ok = ok && wwait(B_ACC_FULL + b, (j >> 1) & 1);
      if (!ok) break;
      TICK(0);
      tc_fence_after();
      const bool valid = has_intra || j >= 1;                    // nothing was accumulated otherwise
      uint32_t dn[4], y[4][16];
#pragma unroll
      for (int h = 0; h < 4; ++h) tmem_ld16(tmem_addr(tb, q4 * 32, COL_ACC + b * 80 + h * 16), y[h]);
      tmem_ld4(tmem_addr(tb, q4 * 32, COL_ACC + b * 80 + 64), dn);
#pragma unroll
      for (int h = 0; h < 4; ++h) tmem_wait_ld(y[h]);
      tmem_wait_ld(dn);
      tc_fence_before();
      mbar_arrive(bar(B_ACC_FREE + b));
      float mx4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int h = 0; h < 4; ++h)
#pragma unroll
        for (int c = 0; c < 16; ++c) mx4[h] = fmaxf(mx4[h], fabsf(__uint_as_float(y[h][c])));
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      // numerators as fp16 relative to a power of two larger than the largest of the row
      const float scale = valid ? __uint_as_float((__float_as_uint(mx) & 0x7F800000u) + 0x00800000u) : 1.f;
      const float inv = (valid && mx > 0.f) ? 1.f / scale : 0.f;
      uint32_t w[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const __half2 hh = __floats2half2_rn(__uint_as_float(y[e >> 3][2 * (e & 7)]) * inv, __uint_as_float(y[e >> 3][2 * (e & 7) + 1]) * inv);
        w[e] = *reinterpret_cast<const uint32_t*>(&hh);
      }
      TICK(1);
      if (j >= 1) ok = wwait(B_STG_FREE, (j - 1) & 1);            // the store of tile j - 1 has read the staging tile
      if (!ok) break;
      TICK(2);
#pragma unroll
      for (int c = 0; c < 8; ++c) sts128(stg + sw128_offset(t, c), w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
      asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(stg + 16384 + t * 8), "f"(valid ? __uint_as_float(dn[0]) : 0.f), "f"(scale) : "memory");
      fence_async_smem();
      mbar_arrive(bar(B_STG_FULL + b));
      TICK(3);
    }
    if (warp == W_E0) TOCK(4);
  } else {
    regs_take<80>();
    // =========================== combine team: this CTA's rows of every tile, summed over the nine shares ===========================
    // A thread waits for the nine shares of a tile and adds up one 16-byte piece of one of the 15 (CTA 8: 8) query
    // rows of the tile that this CTA finishes; the counter of the next tile is read together with the shares of this
    // one, so that a tile costs one trip to L2.
    const int et = tid - W_O0 * 32;
    const int r_in = et >> 3, piece = et & 7;
    __nv_bfloat16* outp = args.out + (size_t)bh * args.T * D;
    const unsigned* cnt = args.counter + (size_t)bh * ntiles;
    if (et == 127) {
      store_thread();
    } else if (r_in < kRowSlots) {
      unsigned have = 0;                                          // shares of tile j seen so far
      for (int j = 0; j < ntiles; ++j) {
        if (have < (unsigned)ncta) ok = wait_count_global(cnt + j, (unsigned)ncta, abort_flag);
        if (!ok) break;
        have = (unsigned)ncta;
        if (j + 1 < ntiles) asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(have) : "l"(cnt + j + 1) : "memory");
#pragma unroll
        for (int r0 = 0; r0 < kRowsPerCta; r0 += kRowSlots) {     // this CTA's rows of the tile, kRowSlots at a time
          const int r_cta = r0 + r_in;
          const int trow = cta_head * kRowsPerCta + r_cta;        // query row of the tile
          if (r_cta >= kRowsPerCta || trow >= CT) continue;
          const size_t in_tile = (size_t)trow * 128 + ((piece ^ (trow & 7)) * 16);
          const size_t row = (size_t)j * CT + trow;
          uint4 pk[NCTA];
          float2 ds[NCTA];
#pragma unroll
          for (int s = 0; s < NCTA; ++s) {
            {
              const unsigned char* blk = args.share + (((size_t)bh * ncta + s) * ntiles + j) * kShareBytes;
              pk[s] = __ldcg(reinterpret_cast<const uint4*>(blk + in_tile));
              ds[s] = __ldcg(reinterpret_cast<const float2*>(blk + 16384 + trow * 8));
            }
          }
          float acc[8], den = 0.f;
#pragma unroll
          for (int c = 0; c < 8; ++c) acc[c] = 0.f;
#pragma unroll
          for (int s = 0; s < NCTA; ++s) {
            {
              den += ds[s].x;
              const uint32_t w4[4] = {pk[s].x, pk[s].y, pk[s].z, pk[s].w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 f2 = __half22float2(*reinterpret_cast<const __half2*>(&w4[e]));
                acc[2 * e] = fmaf(f2.x, ds[s].y, acc[2 * e]);
                acc[2 * e + 1] = fmaf(f2.y, ds[s].y, acc[2 * e + 1]);
              }
            }
          }
          const float inv = den > 0.f ? 1.f / den : 0.f;
          if (row < (size_t)args.T) {
            uint4 o;
            o.x = pack_bf16(acc[0] * inv, acc[1] * inv); o.y = pack_bf16(acc[2] * inv, acc[3] * inv);
            o.z = pack_bf16(acc[4] * inv, acc[5] * inv); o.w = pack_bf16(acc[6] * inv, acc[7] * inv);
            reinterpret_cast<uint4*>(outp + row * D)[piece] = o;
          }
        }
      }
    }
  }

  // ---------------- teardown ----------------
  if (!ok && args.device_status != nullptr) atomicExch(args.device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if ((warp == W_U || warp == W_R) && lane == 0) {
    mma_commit(bar(B_DRAIN));
    mbar_wait(bar(B_DRAIN), 0);
  }
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, TMEM_COLS);
}

// The block pairs (g <= h) the state holds, in the order they are dealt out to the CTAs of a head: all 36 for the
// full lift, those inside a feature group for the blockwise map (runs of 8 features, 8 / groups runs per group).
int fill_block_pairs(BlockPairs& bp, int groups) {
  const int per = 8 / groups;
  int n = 0;
  for (int g = 0; g < 8; ++g)
    for (int h = g; h < 8; ++h) {
      if (g / per != h / per) continue;
      bp.g[n] = (unsigned char)g;
      bp.h[n] = (unsigned char)h;
      bp.w[n] = (unsigned char)(g == h ? 1 : 2);
      ++n;
    }
  return n;
}

// How a head is cut: CTAs per head and accumulator tiles (of two block pairs) per CTA.  The full lift: 36 pairs, nine
// CTAs of four.  Two feature groups: 20 pairs, ten CTAs of two while ten per head fit the GPU in one wave, else five of
// four.  Four groups: 12 pairs, six CTAs of two.
struct SplitPlan {
  int ncta, nm;
};
SplitPlan split_plan(int groups, size_t BH) {
  if (groups == 1) return {9, 2};
  if (groups == 2) return 10 * BH <= 148 ? SplitPlan{10, 1} : SplitPlan{5, 2};
  return {6, 1};
}

size_t al256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

// workspace: counters [BH][ntiles] + ticket | V' [BH][T][64] bf16 | r [BH][T] bf16 | shares [BH][ncta][ntiles][17 KB]
size_t tc_split_workspace_bytes(const Problem& p) {
  const size_t BH = (size_t)p.B * p.H, nt = (size_t)(p.T + CT - 1) / CT;
  const size_t ncta = (size_t)split_plan(p.groups, BH).ncta;
  return al256((BH * nt + 1) * sizeof(unsigned)) + al256(BH * p.T * D * 2) + al256(BH * p.T * 2) + al256(BH * ncta * nt * kShareBytes) +
         (KATA_SPLIT_PROF ? al256(BH * ncta * 5 * 8 * 8) : 0);
}

int tc_split_ctas_per_head(const Problem& p) { return split_plan(p.groups, (size_t)p.B * p.H).ncta; }

bool tc_split_supported(const Problem& p) {
  return p.dtype == KATA_BF16 && p.d_k == 64 && p.d_v == 64 && p.feature_order == 2 && (p.groups == 1 || p.groups == 2 || p.groups == 4);
}

void tc_chunked_split(const Problem& p, void* workspace, int* device_status, LaunchCtx& ctx) {
  const size_t BH = (size_t)p.B * p.H;
  const int ntiles = (p.T + CT - 1) / CT;
  const SplitPlan plan = split_plan(p.groups, BH);
  unsigned char* w8 = static_cast<unsigned char*>(workspace);
  const size_t cnt_bytes = al256((BH * ntiles + 1) * sizeof(unsigned));   // + the ticket counter
  __nv_bfloat16* vs = reinterpret_cast<__nv_bfloat16*>(w8 + cnt_bytes);
  __nv_bfloat16* rscale = reinterpret_cast<__nv_bfloat16*>(w8 + cnt_bytes + al256(BH * p.T * D * 2));
  unsigned char* sh = w8 + cnt_bytes + al256(BH * p.T * D * 2) + al256(BH * p.T * 2);
  CUtensorMap tmQ, tmK, tmV;
  if (!make_tile_map(&tmQ, p.q, (int)BH, p.T, CT) || !make_tile_map(&tmK, p.k, (int)BH, p.T, CT) || !make_tile_map(&tmV, vs, (int)BH, p.T, CT)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  auto kern = p.groups == 1 ? tc_split_kernel<2, 1, 9> : p.groups == 4 ? tc_split_kernel<1, 4, 6> : plan.nm == 1 ? tc_split_kernel<1, 2, 10> : tc_split_kernel<2, 2, 5>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  SplitArgs a{};
  a.out = static_cast<__nv_bfloat16*>(p.out);
  a.rscale = rscale;
  a.counter = reinterpret_cast<unsigned*>(w8);
  a.share = sh;
  a.prof = reinterpret_cast<long long*>(sh + al256(BH * plan.ncta * (size_t)ntiles * kShareBytes));
  a.device_status = device_status;
  a.T = p.T;
  a.ntiles = ntiles;
  a.ncta = plan.ncta;
  a.groups = p.groups;
  if (fill_block_pairs(a.bp, p.groups) != plan.ncta * 2 * plan.nm) {
    ctx.status = KATA_ERR_UNSUPPORTED_SHAPE;
    return;
  }
  if (cudaMemsetAsync(a.counter, 0, cnt_bytes, ctx.stream) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  const size_t n_rows = BH * p.T;
  split_prescale_kernel<<<(unsigned)((n_rows + 31) / 32), 256, 0, ctx.stream>>>(
      static_cast<const __nv_bfloat16*>(p.k), static_cast<const __nv_bfloat16*>(p.v), vs, rscale, n_rows);
  note_launch(ctx);
  kern<<<(unsigned)(BH * plan.ncta), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, tmV, a);
  note_launch(ctx);
}

}  // namespace kata
