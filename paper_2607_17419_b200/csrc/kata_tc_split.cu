// Chunked (linear-state) KATA forward on the Blackwell tensor cores with the FEATURE axis of the state split over
// the CTAs of a head (bf16, d_k = d_v = 64, sequential inter-chunk recurrence, whole sequence in one pass).
//
// Algorithm 1 / section "Chunkwise forward", with the rank-one lift psi(u) = u u^T written as 8 x 8 blocks: the 64
// features of a row are cut into 8 runs of 8, and a "block pair" (g, h), g <= h, is the 64 products
// u[8g+i] u[8h+j].  <psi(q), psi(k)> = (q.k)^2 = sum over the 36 block pairs of w_gh <Q_gh, K_gh> with w = 1 on
// the diagonal pairs (which hold both (i,j) and (j,i)) and w = 2 off it.  One CTA owns 4 block pairs = 256 state
// rows (two M = 128 accumulator tiles S[m], 80 fp32 TMEM columns each: 64 value columns, the normaliser column,
// padding); nine CTAs make a head.  With k' scale r = 1/||k||^2 folded into the values (V' = r V) and the
// normaliser carried as column 64 of every B operand, per tile of 128 tokens a CTA does
//   update   S[m] += Psi(K)_m^T [V' | r]      A = the products, built by token threads in shared memory (MN-major),
//                                             B = the TMA-loaded tile of scaled values, N = 80
//   snapshot B_m = bf16(S[m])                 TMEM -> shared memory, the B operand of the next tile's read
//   read     ACC  = Psi(Q)_m [S | Z]_m        A = the weighted query products in TMEM, N = 80
//   intra    ACC += P_c [V' | r]_c            P_c = (Q K_c^T)^2 masked causally for the 16 keys c of the tile this
//                                             CTA owns (the eight 16-key runs of a tile go to eight of the CTAs)
// ACC is this CTA's share of [N | D] of the tile's 128 queries; the shares are summed
//   (a) inside a thread-block cluster through distributed shared memory (every CTA owns 128 / CS query rows), then
//   (b) from cluster to cluster ("links" of a head) through fp32 scratch in global memory: a link adds what the
//       link before it left (release/acquire progress counters; a link never waits for a later one), and the last
//       link applies the gate/normalise step out = N / D (0 where D = 0) and writes the output.
// The query norm cancels between N and D and is never applied.
//
// Why links: a head needs nine CTAs (36 block pairs / 4), and 16 clusters of 8 or 9 CTAs do not fit the GPCs of a
// B200 at once.  Clusters of 4 do: a head is one single CTA (link 0, its own launch) and two clusters of 4.
//
// A light pre-pass writes V' = r V and r (bf16) once per head, so that the nine CTAs of a head load the scaled values
// with TMA as they are.
// Warps (896 threads): 0 TMA producer, 1 update issuer, 2 read issuer, 3 score issuer; 4-11 key teams (team m builds
// the products of accumulator tile m; team 0 also places r); 12-15 query team; 16-19 state team (TMEM -> bf16
// snapshot, both accumulator tiles in turn); 20-23 intra-tile weights and the exchange of shares; 24-27 owner sums,
// link hand-off and output.  Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cstdlib>

#include "kata_common.cuh"
#include "kata_tmap.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int CT = 128;            // tokens per tile
constexpr int NBP = 4;             // block pairs per CTA
constexpr int NTHREADS = 896;
constexpr int W_TMA = 0, W_U = 1, W_R = 2, W_I = 3, W_K0 = 4, W_Q0 = 12, W_S0 = 16, W_E0 = 20, W_O0 = 24;
constexpr int MAX_CTAS = 12;       // CTAs of a head over all links
constexpr int kPublish = 8;        // tiles between two publications of a link's progress

// ---- TMEM columns ----
constexpr uint32_t COL_S = 0;      // 2 x 80: state tiles (lanes = state rows)
constexpr uint32_t COL_PSIQ = 160; // 128: weighted query products as bf16 pairs (lanes = tokens), 32 per block pair
constexpr uint32_t COL_ACC = 288;  // 2 x 80: this CTA's share of [N | D] (lanes = tokens)
constexpr uint32_t COL_SC = 448;   // 16 fp32 scores
constexpr uint32_t COL_P = 464;    // 8: bf16 weights
constexpr uint32_t TMEM_COLS = 512;

// ---- shared memory (1024-byte aligned tiles of 128-byte rows, 128B swizzle) ----
constexpr uint32_t OFF_PSIK = 0;        // 4 block pairs x [128 tokens][64 products]
constexpr uint32_t OFF_KRAW = 65536;    // key tile
constexpr uint32_t OFF_QRAW = 81920;    // query tile
constexpr uint32_t OFF_VP = 98304;      // 2 x value tile (scaled in place)
constexpr uint32_t OFF_SNAP = 131072;   // 2 x [128 state rows][64 values] bf16
constexpr uint32_t OFF_COL64 = 163840;  // column 64 of the four B operands above: 32 bytes of every row each
constexpr uint32_t OFF_RECV = 180224;   // 128 rows x 68 floats: shares received for the rows this CTA owns
constexpr uint32_t RECV_ROW = 272;
constexpr uint32_t OFF_BAR = OFF_RECV + 128 * RECV_ROW;
constexpr uint32_t OFF_MISC = OFF_BAR + 512;
constexpr uint32_t SMEM_BYTES = OFF_MISC + 64;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(SMEM_ALLOC <= 232448, "shared memory");

// Every barrier has waiters that consume each of its phases in order.
enum {
  B_K_FULL = 0,      // key tile landed
  B_Q_FULL = 1,      // query tile landed
  B_V_FULL = 2,      // [2] tile of scaled values landed
  B_SC_FULL = 4,     // intra-tile scores in TMEM
  B_MMA_DONE = 5,    // update, read and apply MMAs of a tile complete (two commits)
  B_RECV_FULL = 6,   // every share of the rows this CTA owns has arrived (transaction bytes; armed by the owner team)
  B_RECV_EMPTY = 7,  // [4] the owner with that rank has summed what this CTA sent
  B_DRAIN = 11,
  B_COUNT = 12
};


struct BlockPairs {
  unsigned char g[MAX_CTAS * NBP], h[MAX_CTAS * NBP], w[MAX_CTAS * NBP];   // w = 0: unused slot
};

struct SplitArgs {
  __nv_bfloat16* out;
  float* scrN;            // [links - 1][BH][Tpad][64]
  float* scrD;            // [links - 1][BH][Tpad]
  unsigned* progress;     // [links][BH][4]: tiles completed by each owner of a link
  int* device_status;
  int T, ntiles, BH;
  int n_links;            // links of a head over all launches
  int link0, cta0;        // first link / first CTA (within the head) of this launch
  int ctas;               // CTAs of a head in this launch (a multiple of the cluster size)
  int cs_prev;            // cluster size of the launch before (owners of link0 - 1)
  int trigger;            // 1: let the next launch in the stream start at once
  const __nv_bfloat16* rscale;   // [BH][T] bf16: 1 / ||k||^2 (pre-pass)
  BlockPairs bp;
};

// ---- cluster helpers ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t raddr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(raddr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void arrive_remote(uint32_t rbar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(rbar) : "memory");
}
// Bounded wait whose acquire covers writes made by other CTAs of the cluster before their arrival.  Bounded by a
// poll count (hint 1 us per poll): reading the global timer after a failed first try costs more than most waits last.
__device__ __forceinline__ bool wait_cluster_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  uint32_t ok;
  asm volatile(
      "{\n\t"
      ".reg .pred p, q;\n\t"
      ".reg .u32 i;\n\t"
      "mov.u32 i, 0;\n\t"
      "KATA_CWAIT_%=:\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, 1000;\n\t"
      "@p bra KATA_CDONE_%=;\n\t"
      "add.u32 i, i, 1;\n\t"
      "setp.lt.u32 q, i, %3;\n\t"
      "@q bra KATA_CWAIT_%=;\n\t"
      "KATA_CDONE_%=:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kSpinLimit)
      : "memory");
  if (ok == 0) *abort_flag = 1;
  return ok != 0;
}
// Bounded wait for a progress counter in global memory (written with release by another CTA).
__device__ __forceinline__ bool wait_progress(const unsigned* p, unsigned want, volatile int* abort_flag) {
  unsigned v, t0, t1;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  if (v >= want) return true;
  asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t0));
  for (;;) {
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    if (v >= want) return true;
    asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t1));
    if (*abort_flag != 0 || t1 - t0 > 10u * kWaitLimitNs) {   // a producer that is not resident yet may take long
      *abort_flag = 1;
      return false;
    }
    __nanosleep(200);
  }
}

// Shared-memory accesses of buffers that other agents refill (TMA, MMA operands, other CTAs): by address in the shared
// window (a generic-address load is not ordered with the mbarrier arrival that hands the buffer back).  Not volatile:
// a volatile shared access costs a round trip each (measured: ten times the time of the same code with weak accesses).
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
  uint4 r;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(saddr) : "memory");
  return r;
}
__device__ __forceinline__ float4 lds128f(uint32_t saddr) {
  float4 r;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(saddr) : "memory");
  return r;
}
__device__ __forceinline__ float lds32f(uint32_t saddr) {
  float r;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(r) : "r"(saddr) : "memory");
  return r;
}
__device__ __forceinline__ void sts128(uint32_t saddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t saddr, unsigned short v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(saddr), "h"(v) : "memory");
}

// Values loaded from a buffer are kept in registers across the arrival that hands the buffer back to its producer.
// Neither the assembler nor the hardware makes that arrival wait for loads whose results nobody has used yet (seen
// here: key runs that came from the NEXT tile, the refill having overtaken the load), so the loaded words are folded
// into one word that is stored before the arrival: the store cannot issue until every load has returned.
template <int N>
__device__ __forceinline__ void consume_before_arrive(uint32_t sink_addr, const uint32_t (&w)[N]) {
  uint32_t x = w[0];
#pragma unroll
  for (int i = 1; i < N; ++i) x ^= w[i];
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(sink_addr), "r"(x) : "memory");
}

// Register budget per warp group (the kernel is launched with 72 registers per thread for 896 threads): the four
// issuer warps and the key teams give registers up, the teams that hold tiles of TMEM in registers take them.
template <int N> __device__ __forceinline__ void regs_release() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_take() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
static_assert(128 * 40 + 256 * 56 + 512 * 88 <= 896 * 72, "register budget");

// 64 products a[i] b[j] (i, j < 8) of two runs of 8 bf16 (4 words each), scaled by the bf16 pair `wgt`, as 8 chunks of
// 8 bf16 (chunk i = a[i] * b[0..7]).  One rounding per product (the scale is 0, 1 or 2).
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

// Asynchronous store of 16 bytes into the shared memory of a CTA of the cluster; the bytes count towards the
// transaction count of the mbarrier `rbar` of that CTA (no arrival of its own).
__device__ __forceinline__ void st_async_v4(uint32_t raddr, uint32_t rbar, float a, float b, float c, float d) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(raddr), "f"(a),
               "f"(b), "f"(c), "f"(d), "r"(rbar)
               : "memory");
}

// The kernel walks the tiles in lockstep.  Tile j is two phases:
//   A  everything the MMAs of the tile read is put in place: key products (key teams), weighted query products
//      (query team), the snapshot of the state after tile j - 1 (state team), the intra-tile weights (score MMA
//      first, then the exchange team); one named barrier (kBarA) ends the phase;
//   B  the update, read and apply MMAs of the tile are issued back to back (two issuing threads) and commit to
//      one mbarrier (B_MMA_DONE), which every team waits for before it touches its buffers again.  Under phase B
//      the exchange team sends the shares of tile j - 1, the owner team sums those of tile j - 2, and the TMA
//      producer fetches the keys and queries of tile j + 1 (buffers free since phase A) and the values of tile
//      j + 2.
// Two synchronisations per tile instead of a web of point-to-point hand-offs: every hand-off between warps costs
// several hundred cycles from arrival to the waiter's next instruction, and a pipeline whose every buffer is single
// (shared memory and TMEM are full) turns each of them into a round trip.
constexpr int kBarA = 2;
constexpr int kBarAThreads = 32 * W_O0;     // every warp but the owner team

template <int CS>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_split_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ SplitArgs args) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  auto bar = [&](int i) { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; };
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(base + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base + OFF_MISC + 4);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = CS == 1 ? 0u : cluster_ctarank();
  const int bh = blockIdx.x / args.ctas;
  const int cta_launch = blockIdx.x % args.ctas;              // CTA of the head within this launch
  const int cta_head = args.cta0 + cta_launch;                // ... within the head
  const int link = args.link0 + cta_launch / CS;
  const bool last_link = link == args.n_links - 1;
  const int ntiles = args.ntiles;
  const int chunk = cta_head - 1;                             // 16-key run of every tile this CTA weighs (link 0: none)
  const bool has_intra = chunk >= 0 && chunk < 8;
  constexpr int RPO = CT / CS;                                // query rows of a tile this CTA owns
  constexpr uint32_t RECV_BYTES = 128 * RECV_ROW;             // what the owner receives per tile

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(bar(B_K_FULL), 1);
    mbar_init(bar(B_Q_FULL), 1);
    mbar_init(bar(B_V_FULL), 1);
    mbar_init(bar(B_V_FULL + 1), 1);
    mbar_init(bar(B_SC_FULL), 1);
    mbar_init(bar(B_MMA_DONE), 2);
    mbar_init(bar(B_RECV_FULL), 1);
    for (int i = 0; i < 4; ++i) mbar_init(bar(B_RECV_EMPTY + i), 1);
    mbar_init(bar(B_DRAIN), 3);
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
  if (args.trigger) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                 // every CTA's barriers exist before anything arrives on them from outside
  tc_fence_after();
  const uint32_t tb = *tmem_base_s;
  bool ok = true;
  // the wait that opens tile j for every team: the MMAs of tile j - 1 are complete
  auto mma_done = [&](int j) { return j == 0 ? true : wait_or_abort_counted(bar(B_MMA_DONE), (j - 1) & 1, abort_flag); };
  // end of phase A.  A team that gave up keeps arriving, so that nobody is left waiting at the named barrier.
  auto phase_a_done = [&]() { asm volatile("bar.sync %0, %1;" ::"n"(kBarA), "n"(kBarAThreads) : "memory"); };

  if (warp < W_K0) {
    regs_release<40>();
    if (warp == W_TMA) {
      // =========================== TMA producer ===========================
      for (int j = 0; j < ntiles; ++j) {
        const int b = j & 1;
        if (lane == 0 && ok) {
          if (j == 0) {
            mbar_arrive_expect_tx(bar(B_K_FULL), 16384);
            tma_load_3d(base + OFF_KRAW, &tmK, bar(B_K_FULL), 0, 0, bh);
            mbar_arrive_expect_tx(bar(B_Q_FULL), 16384);
            tma_load_3d(base + OFF_QRAW, &tmQ, bar(B_Q_FULL), 0, 0, bh);
            mbar_arrive_expect_tx(bar(B_V_FULL), 16384);
            tma_load_3d(base + OFF_VP, &tmV, bar(B_V_FULL), 0, 0, bh);
            if (ntiles > 1) {
              mbar_arrive_expect_tx(bar(B_V_FULL + 1), 16384);
              tma_load_3d(base + OFF_VP + 16384, &tmV, bar(B_V_FULL + 1), 0, CT, bh);
            }
          }
          // tiles three ahead into L2, so that the loads below find them there
          if (j + 3 < ntiles) {
            asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(&tmK), "r"(0), "r"((j + 3) * CT), "r"(bh) : "memory");
            asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(&tmQ), "r"(0), "r"((j + 3) * CT), "r"(bh) : "memory");
            asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(&tmV), "r"(0), "r"((j + 3) * CT), "r"(bh) : "memory");
          }
        }
        phase_a_done();                 // keys and queries of tile j have been read (teams) and multiplied (score MMA)
        if (lane == 0 && ok && j + 1 < ntiles) {
          mbar_arrive_expect_tx(bar(B_K_FULL), 16384);
          tma_load_3d(base + OFF_KRAW, &tmK, bar(B_K_FULL), 0, (j + 1) * CT, bh);
          mbar_arrive_expect_tx(bar(B_Q_FULL), 16384);
          tma_load_3d(base + OFF_QRAW, &tmQ, bar(B_Q_FULL), 0, (j + 1) * CT, bh);
        }
        if (j + 2 < ntiles) {
          ok = ok && mma_done(j + 1);   // the MMAs of tile j are done with the value tile
          if (lane == 0 && ok) {
            mbar_arrive_expect_tx(bar(B_V_FULL + b), 16384);
            tma_load_3d(base + OFF_VP + b * 16384, &tmV, bar(B_V_FULL + b), 0, (j + 2) * CT, bh);
          }
        }
      }
    } else if (warp == W_U) {
      // =========================== update issuer: S[m] += Psi(K)_m^T [V' | r] ===========================
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 80);
      const uint64_t da = smem_desc(0, 16384, 1024, kSwizzle128B);      // second run of 64 state rows: next block pair
      for (int j = 0; j < ntiles; ++j) {
        const int b = j & 1;
        phase_a_done();
        ok = ok && wait_or_abort_counted(bar(B_V_FULL + b), (j >> 1) & 1, abort_flag);
        if (lane == 0) {
          if (ok) {
            tc_fence_after();
            const uint32_t vp = sbase + OFF_VP + b * 16384;
            const uint64_t db = smem_desc(0, sbase + OFF_COL64 + 32 * b - vp, 1024, kSwizzle128B);
#pragma unroll
            for (int m = 0; m < 2; ++m) {
              const uint32_t pa = sbase + OFF_PSIK + m * 32768;
#pragma unroll
              for (int ks = 0; ks < 8; ++ks)
                mma_f16_ss(tb + COL_S + m * 80, at(da, pa + ks * 2048), at(db, vp + ks * 2048), idesc, (j > 0 || ks > 0) ? 1u : 0u);
            }
          }
          mma_commit(bar(B_MMA_DONE));
        }
        __syncwarp();
      }
    } else if (warp == W_R) {
      // =========================== read issuer: ACC = Psi(Q) [S | Z] + P_c [V' | r]_c ===========================
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 80);
      for (int j = 0; j < ntiles; ++j) {
        const int b = j & 1;
        phase_a_done();
        if (has_intra) ok = ok && wait_or_abort_counted(bar(B_V_FULL + b), (j >> 1) & 1, abort_flag);
        if (lane == 0) {
          if (ok) {
            tc_fence_after();
            if (j >= 1) {
#pragma unroll
              for (int m = 0; m < 2; ++m) {
                const uint32_t sn = sbase + OFF_SNAP + m * 16384;
                const uint64_t db = smem_desc(0, sbase + OFF_COL64 + 32 * (2 + m) - sn, 1024, kSwizzle128B);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                  mma_f16_ts(tb + COL_ACC + b * 80, tb + COL_PSIQ + m * 64 + ks * 8, at(db, sn + ks * 2048), idesc, (m > 0 || ks > 0) ? 1u : 0u);
              }
            }
            if (has_intra) {
              const uint32_t vp = sbase + OFF_VP + b * 16384;
              const uint64_t db = smem_desc(0, sbase + OFF_COL64 + 32 * b - vp, 1024, kSwizzle128B);
              mma_f16_ts(tb + COL_ACC + b * 80, tb + COL_P, at(db, vp + chunk * 2048), idesc, j >= 1 ? 1u : 0u);
            }
          }
          mma_commit(bar(B_MMA_DONE));
        }
        __syncwarp();
      }
    } else {
      // =========================== score issuer: Q K_c^T for this CTA's 16 keys (opens phase A) ===========================
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 16);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      const uint32_t qa = sbase + OFF_QRAW, ka = sbase + OFF_KRAW + (has_intra ? chunk : 0) * 2048;
      for (int j = 0; j < ntiles; ++j) {
        if (has_intra) {
          ok = ok && mma_done(j);       // the apply MMA of tile j - 1 has read the weights; their columns may be rewritten
          ok = ok && wait_or_abort_counted(bar(B_K_FULL), j & 1, abort_flag) && wait_or_abort_counted(bar(B_Q_FULL), j & 1, abort_flag);
          if (lane == 0) {
            if (ok) {
              tc_fence_after();
#pragma unroll
              for (int ks = 0; ks < 4; ++ks) mma_f16_ss(tb + COL_SC, at(dk, qa + ks * 32), at(dk, ka + ks * 32), idesc, ks > 0 ? 1u : 0u);
            }
            mma_commit(bar(B_SC_FULL));
          }
          __syncwarp();
        }
        phase_a_done();
      }
    }
  } else if (warp < W_Q0) {
    regs_release<56>();
    // =========================== key teams (thread = token; team m = accumulator tile m) ===========================
    const int m = (warp - W_K0) >> 2;
    const int t = ((warp - W_K0) & 3) * 32 + lane;
    int pg[2], ph[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      pg[e] = args.bp.g[cta_head * NBP + 2 * m + e];
      ph[e] = args.bp.h[cta_head * NBP + 2 * m + e];
    }
    const uint32_t kraw = sbase + OFF_KRAW;
    const unsigned short* rs = reinterpret_cast<const unsigned short*>(args.rscale) + (size_t)bh * args.T;
    unsigned short r_next = (m == 0 && t < args.T) ? rs[t] : (unsigned short)0;
    for (int j = 0; j < ntiles; ++j) {
      const int b = j & 1;
      ok = ok && mma_done(j);           // the update of tile j - 1 has read the products (and column 64 of its values)
      ok = ok && wait_or_abort_counted(bar(B_K_FULL), j & 1, abort_flag);
      if (ok) {
        if (m == 0) {                   // column 64 of the value operand: r of this token
          sts16(sbase + OFF_COL64 + sw128_offset(t, 2 * b), r_next);
          const int tn = (j + 1) * CT + t;
          r_next = (j + 1 < ntiles && tn < args.T) ? rs[tn] : (unsigned short)0;
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const uint4 ra = lds128(kraw + sw128_offset(t, pg[e]));
          const uint4 rb = lds128(kraw + sw128_offset(t, ph[e]));
          const uint32_t ga[4] = {ra.x, ra.y, ra.z, ra.w}, gb[4] = {rb.x, rb.y, rb.z, rb.w};
          uint32_t pr[32];
          products8x8<false>(ga, gb, 0u, pr);
          const uint32_t dst = sbase + OFF_PSIK + (2 * m + e) * 16384;
#pragma unroll
          for (int i = 0; i < 8; ++i) sts128(dst + sw128_offset(t, i), pr[4 * i], pr[4 * i + 1], pr[4 * i + 2], pr[4 * i + 3]);
        }
        fence_async_smem();
      }
      phase_a_done();
    }
  } else if (warp < W_S0) {
    regs_take<88>();
    // =========================== query team (thread = token) ===========================
    const uint32_t q4 = warp & 3;
    const int t = q4 * 32 + lane;
    int pg[NBP], ph[NBP];
    uint32_t pw[NBP];
#pragma unroll
    for (int e = 0; e < NBP; ++e) {
      pg[e] = args.bp.g[cta_head * NBP + e];
      ph[e] = args.bp.h[cta_head * NBP + e];
      const int w = args.bp.w[cta_head * NBP + e];
      pw[e] = w == 0 ? 0u : w == 1 ? 0x3F803F80u : 0x40004000u;
    }
    const uint32_t qraw = sbase + OFF_QRAW;
    for (int j = 0; j < ntiles; ++j) {
      ok = ok && mma_done(j);           // the read of tile j - 1 has used the products
      ok = ok && wait_or_abort_counted(bar(B_Q_FULL), j & 1, abort_flag);
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
        tmem_wait_st();
        tc_fence_before();
      }
      phase_a_done();
    }
  } else if (warp < W_E0) {
    regs_take<88>();
    // =========================== state team (thread = state row of both accumulator tiles) ===========================
    const uint32_t q4 = warp & 3;
    const int f = q4 * 32 + lane;
    for (int j = 0; j < ntiles; ++j) {
      ok = ok && mma_done(j);           // the update of tile j - 1 is complete, and so is the read that used the old snapshot
      if (ok && j >= 1) {
        tc_fence_after();
#pragma unroll
        for (int m = 0; m < 2; ++m) {
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
      phase_a_done();
    }
  } else if (warp < W_O0) {
    regs_take<88>();
    // =========================== intra-tile weights and the exchange of shares (thread = token) ===========================
    const uint32_t q4 = warp & 3;
    const int t = q4 * 32 + lane;
    const uint32_t owner = (uint32_t)(t / RPO);
    const uint32_t recv_local = sbase + OFF_RECV + (rank * RPO + (t % RPO)) * RECV_ROW;
    const uint32_t recv_remote = map_to_rank(recv_local, owner);
    const uint32_t full_remote = map_to_rank(smem_u32(bar(B_RECV_FULL)), owner);
    for (int j = 0; j <= ntiles; ++j) {
      ok = ok && mma_done(j);           // observed here, like every team, before the tile's named barrier
      // ---- phase A of tile j: weights P = (Q K_c^T)^2, causal inside the tile ----
      if (j < ntiles) {
        if (has_intra) {
          ok = ok && wait_or_abort_counted(bar(B_SC_FULL), j & 1, abort_flag);
          if (ok) {
            tc_fence_after();
            uint32_t y[16], pk[8];
            tmem_ld16(tmem_addr(tb, q4 * 32, COL_SC), y);
            tmem_wait_ld(y);
#pragma unroll
            for (int c = 0; c < 16; c += 2) {
              float a = __uint_as_float(y[c]), bq = __uint_as_float(y[c + 1]);
              a = (chunk * 16 + c <= t) ? a * a : 0.f;
              bq = (chunk * 16 + c + 1 <= t) ? bq * bq : 0.f;
              pk[c >> 1] = pack_bf16(a, bq);
            }
            tmem_st8(tmem_addr(tb, q4 * 32, COL_P), pk);
            tmem_wait_st();
            tc_fence_before();
          }
        }
        phase_a_done();
      }
      // ---- under phase B of tile j: this CTA's share of tile j - 1 goes to the owners of its rows ----
      if (j >= 1) {
        const int jj = j - 1, b = jj & 1;
        if (ok && jj >= 1) ok = wait_cluster_or_abort(bar(B_RECV_EMPTY + owner), (jj - 1) & 1, abort_flag);
        if (ok) {
          tc_fence_after();
          const bool valid = has_intra || jj >= 1;               // nothing was accumulated otherwise
#pragma unroll 1
          for (int h = 0; h < 2; ++h) {
            uint32_t y[32];
            tmem_ld32(tmem_addr(tb, q4 * 32, COL_ACC + b * 80 + h * 32), y);
            tmem_wait_ld(y);
#pragma unroll
            for (int c = 0; c < 8; ++c)
              st_async_v4(recv_remote + h * 128 + c * 16, full_remote, valid ? __uint_as_float(y[4 * c]) : 0.f,
                          valid ? __uint_as_float(y[4 * c + 1]) : 0.f, valid ? __uint_as_float(y[4 * c + 2]) : 0.f,
                          valid ? __uint_as_float(y[4 * c + 3]) : 0.f);
          }
          uint32_t dn[4];
          tmem_ld4(tmem_addr(tb, q4 * 32, COL_ACC + b * 80 + 64), dn);
          tmem_wait_ld(dn);
          tc_fence_before();
          st_async_v4(recv_remote + 256, full_remote, valid ? __uint_as_float(dn[0]) : 0.f, 0.f, 0.f, 0.f);
        }
      }
    }
  } else {
    regs_take<88>();
    // =========================== owner: sums of the shares, link hand-off, output ===========================
    const int et = tid - W_O0 * 32;                            // 0..127
    const size_t tpad = (size_t)ntiles * CT;
    const float* inN = link > 0 ? args.scrN + ((size_t)(link - 1) * args.BH + bh) * tpad * 64 : nullptr;
    const float* inD = link > 0 ? args.scrD + ((size_t)(link - 1) * args.BH + bh) * tpad : nullptr;
    float* outN = !last_link ? args.scrN + ((size_t)link * args.BH + bh) * tpad * 64 : nullptr;
    float* outD = !last_link ? args.scrD + ((size_t)link * args.BH + bh) * tpad : nullptr;
    // owners of the link before: the rows this CTA owns lie inside the rows of one of them
    const int cs_in = link > args.link0 ? CS : args.cs_prev;
    const unsigned* prog_in = link > 0 ? args.progress + ((size_t)(link - 1) * args.BH + bh) * 4 + (rank * RPO) / (CT / cs_in) : nullptr;
    unsigned* prog_out = args.progress + ((size_t)link * args.BH + bh) * 4 + rank;
    __nv_bfloat16* outp = args.out + (size_t)bh * args.T * D;
    constexpr int N_ITEMS = RPO * 4 / 128;                     // (row, 16 columns) items per thread: 1 (clusters of 4) or 4
    // what the link before left for the first item of the next tile, fetched one tile ahead
    float4 pre[4];
    float pre_d = 0.f;
    auto prefetch = [&](int j) {
      const int row = et >> 2, qu = et & 3;
      const size_t grow = (size_t)j * CT + rank * RPO + row;
#pragma unroll
      for (int c = 0; c < 4; ++c) pre[c] = *reinterpret_cast<const float4*>(inN + grow * 64 + qu * 16 + c * 4);
      if (qu == 0) pre_d = inD[grow];
    };
    if (et == 0 && ntiles > 0) mbar_arrive_expect_tx(bar(B_RECV_FULL), RECV_BYTES);
    if (inN != nullptr && ntiles > 0) {
      ok = wait_progress(prog_in, 1u, abort_flag);
      if (ok) prefetch(0);
    }
    for (int j = 0; j < ntiles && ok; ++j) {
      ok = wait_cluster_or_abort(bar(B_RECV_FULL), j & 1, abort_flag);
      if (!ok) break;
#pragma unroll 1
      for (int k = 0; k < N_ITEMS; ++k) {
        const int item = et + k * 128;
        const int row = item >> 2, qu = item & 3;              // row among the owned rows, 16 of the 64 columns
        float acc[16], dsum = 0.f;
#pragma unroll
        for (int c = 0; c < 16; ++c) acc[c] = 0.f;
#pragma unroll
        for (int s = 0; s < CS; ++s) {
          const uint32_t src = sbase + OFF_RECV + (s * RPO + row) * RECV_ROW;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float4 x = lds128f(src + qu * 64 + c * 16);
            acc[4 * c] += x.x; acc[4 * c + 1] += x.y; acc[4 * c + 2] += x.z; acc[4 * c + 3] += x.w;
          }
          if (qu == 0) dsum += lds32f(src + 256);
        }
        const size_t grow = (size_t)j * CT + rank * RPO + row;      // token of the head
        if (inN != nullptr) {
          if (k == 0) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              acc[4 * c] += pre[c].x; acc[4 * c + 1] += pre[c].y; acc[4 * c + 2] += pre[c].z; acc[4 * c + 3] += pre[c].w;
            }
            if (qu == 0) dsum += pre_d;
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float4 x = *reinterpret_cast<const float4*>(inN + grow * 64 + qu * 16 + c * 4);
              acc[4 * c] += x.x; acc[4 * c + 1] += x.y; acc[4 * c + 2] += x.z; acc[4 * c + 3] += x.w;
            }
            if (qu == 0) dsum += inD[grow];
          }
        }
        if (!last_link) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            *reinterpret_cast<float4*>(outN + grow * 64 + qu * 16 + c * 4) = make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
          if (qu == 0) outD[grow] = dsum;
        } else {
          // the four threads of a row are neighbours in a warp: the denominator comes from the first of them
          const float den = __shfl_sync(0xffffffffu, dsum, lane & ~3);
          const float inv = den > 0.f ? 1.f / den : 0.f;
          if (grow < (size_t)args.T) {
            uint4 o0, o1;
            o0.x = pack_bf16(acc[0] * inv, acc[1] * inv);   o0.y = pack_bf16(acc[2] * inv, acc[3] * inv);
            o0.z = pack_bf16(acc[4] * inv, acc[5] * inv);   o0.w = pack_bf16(acc[6] * inv, acc[7] * inv);
            o1.x = pack_bf16(acc[8] * inv, acc[9] * inv);   o1.y = pack_bf16(acc[10] * inv, acc[11] * inv);
            o1.z = pack_bf16(acc[12] * inv, acc[13] * inv); o1.w = pack_bf16(acc[14] * inv, acc[15] * inv);
            uint4* dst = reinterpret_cast<uint4*>(outp + grow * D + qu * 16);
            dst[0] = o0;
            dst[1] = o1;
          }
        }
      }
      // every thread of the team has read its shares (and written its rows): the buffer is armed for the next tile
      // and handed back to the senders, and one thread publishes the tile to the next link (its release covers
      // the team's writes, which the barrier orders before it; every kPublish tiles and at the end: a release at
      // GPU scope waits for the whole team's stores to land, and the next link is content to run a few tiles behind)
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et == 0 && j + 1 < ntiles) mbar_arrive_expect_tx(bar(B_RECV_FULL), RECV_BYTES);
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (et < CS) arrive_remote(map_to_rank(smem_u32(bar(B_RECV_EMPTY + rank)), (uint32_t)et));
      if (et == 0 && !last_link && (((j + 1) % kPublish) == 0 || j + 1 == ntiles))
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(prog_out), "r"((unsigned)(j + 1)) : "memory");
      if (inN != nullptr && j + 1 < ntiles) {
        ok = wait_progress(prog_in, (unsigned)(j + 2), abort_flag);
        if (ok) prefetch(j + 1);
      }
    }
  }

  // ---------------- teardown ----------------
  if (!ok && args.device_status != nullptr) atomicExch(args.device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp >= W_U && warp <= W_I && lane == 0) {
    mma_commit(bar(B_DRAIN));
    mbar_wait(bar(B_DRAIN), 0);
  }
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, TMEM_COLS);
  cluster_sync_all();                 // no CTA leaves while others may still write into its shared memory
}

// The 36 block pairs (g <= h) of the rank-one lift in the order they are dealt out, four to a CTA.
void fill_block_pairs(BlockPairs& bp, int* n_ctas) {
  int n = 0;
  for (int g = 0; g < 8; ++g)
    for (int h = g; h < 8; ++h) {
      bp.g[n] = (unsigned char)g;
      bp.h[n] = (unsigned char)h;
      bp.w[n] = (unsigned char)(g == h ? 1 : 2);
      ++n;
    }
  *n_ctas = (n + NBP - 1) / NBP;
  for (; n < MAX_CTAS * NBP; ++n) bp.g[n] = bp.h[n] = bp.w[n] = 0;
}

constexpr int kLinks = 3;              // a single CTA, then two clusters of four

}  // namespace

static size_t al256(size_t x) { return (x + 255) / 256 * 256; }

// workspace: progress counters | V' [BH][T][64] bf16 | r [BH][T] bf16 | N scratch [links - 1][BH][Tpad][64] fp32 | D scratch
size_t tc_split_workspace_bytes(const Problem& p) {
  const size_t BH = (size_t)p.B * p.H, tpad = (size_t)((p.T + CT - 1) / CT) * CT;
  return al256(kLinks * BH * 4 * sizeof(unsigned)) + al256(BH * p.T * D * 2) + al256(BH * p.T * 2) +
         (kLinks - 1) * BH * tpad * 65 * sizeof(float);
}

bool tc_split_supported(const Problem& p) {
  return p.dtype == KATA_BF16 && p.d_k == 64 && p.d_v == 64 && p.feature_order == 2 && p.groups == 1;
}

void tc_chunked_split(const Problem& p, void* workspace, int* device_status, LaunchCtx& ctx) {
  const int BH = p.B * p.H;
  const int ntiles = (p.T + CT - 1) / CT;
  const size_t tpad = (size_t)ntiles * CT;
  unsigned char* w8 = static_cast<unsigned char*>(workspace);
  const size_t prog_bytes = al256(kLinks * (size_t)BH * 4 * sizeof(unsigned));
  __nv_bfloat16* vs = reinterpret_cast<__nv_bfloat16*>(w8 + prog_bytes);
  __nv_bfloat16* rscale = reinterpret_cast<__nv_bfloat16*>(w8 + prog_bytes + al256((size_t)BH * p.T * D * 2));
  float* scr = reinterpret_cast<float*>(w8 + prog_bytes + al256((size_t)BH * p.T * D * 2) + al256((size_t)BH * p.T * 2));
  CUtensorMap tmQ, tmK, tmV;
  if (!make_tile_map(&tmQ, p.q, BH, p.T, CT) || !make_tile_map(&tmK, p.k, BH, p.T, CT) || !make_tile_map(&tmV, vs, BH, p.T, CT)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  if (cudaFuncSetAttribute(tc_split_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
      cudaFuncSetAttribute(tc_split_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  SplitArgs a{};
  a.out = static_cast<__nv_bfloat16*>(p.out);
  a.progress = reinterpret_cast<unsigned*>(w8);
  a.scrN = scr;
  a.scrD = scr + (size_t)(kLinks - 1) * BH * tpad * 64;
  a.rscale = rscale;
  a.device_status = device_status;
  a.T = p.T;
  a.ntiles = ntiles;
  a.BH = BH;
  a.n_links = kLinks;
  int n_ctas = 0;
  fill_block_pairs(a.bp, &n_ctas);
  if (cudaMemsetAsync(a.progress, 0, prog_bytes, ctx.stream) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  const size_t n_rows = (size_t)BH * p.T;
  split_prescale_kernel<<<(unsigned)((n_rows + 31) / 32), 256, 0, ctx.stream>>>(
      static_cast<const __nv_bfloat16*>(p.k), static_cast<const __nv_bfloat16*>(p.v), vs, rscale, n_rows);
  note_launch(ctx);
  // launch 1: link 0, one CTA per head; launch 2: links 1 and 2, two clusters of four per head, allowed to start
  // while launch 1 runs (it consumes what launch 1 produces tile by tile)
  for (int launch = 0; launch < 2; ++launch) {
    const int cs = launch == 0 ? 1 : 4;
    a.link0 = launch == 0 ? 0 : 1;
    a.cta0 = launch == 0 ? 0 : 1;
    a.ctas = launch == 0 ? 1 : 8;
    a.cs_prev = 1;
    a.trigger = launch == 0 ? 1 : 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(BH * a.ctas));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = SMEM_ALLOC;
    cfg.stream = ctx.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = launch == 0 ? 1 : 2;
    const cudaError_t err = launch == 0 ? cudaLaunchKernelEx(&cfg, tc_split_kernel<1>, tmQ, tmK, tmV, a)
                                        : cudaLaunchKernelEx(&cfg, tc_split_kernel<4>, tmQ, tmK, tmV, a);
    if (err != cudaSuccess) {
      cudaGetLastError();
      ctx.status = KATA_ERR_CUDA;
      return;
    }
    ++ctx.launches;
  }
}

}  // namespace kata
