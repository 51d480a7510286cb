// First-order feature (rows of q, k used as features as they are; appendix "Associative-scan kernel": matched
// d x d states, already-feature-mapped inputs) on the Blackwell tensor cores: bf16, d_k = d_v = 64.
//   o_t = sum_{i<=t} (q_t . k_i) v_i / sum_{i<=t} (q_t . k_i)
// One CTA owns one head and one group of 128-token tiles and walks the group in order.  Per tile:
//   scores   P = tril(Q K^T)                       SS MMA, fp32 in TMEM, masked and rounded to bf16 by 8 warps
//   intra    [O | D]  = P [V | 1]                  A = P from TMEM, B = the value tile read MN-major with a column
//                                                  of ones behind it (a static tile reached through the leading
//                                                  byte offset of the descriptor), N = 80
//   inter    [O | D] += Q [S | Z]^T                B = bf16 snapshot of the state before the tile (80 rows x 64)
//   update   [S | Z]^T += [V | 1]^T K              A = the same value tile and ones column (M = 128 rows: 64 value
//                                                  columns, the normaliser row, zero rows), B = the key tile;
//                                                  fp32 accumulators stay in TMEM for the whole group
//   out      O / D                                 (0 where D = 0)
// A head of many tiles and few heads: the chunk axis is cut into groups of tiles and the CTAs (one per SM) take
// groups until none is left.  A group is walked twice.  Pass 0 builds the state of the group alone (keys and values
// are the only loads) and publishes it; the look-back then adds up the states of the groups before it (a chained
// scan over the group states: every eighth group is an anchor that publishes the sum of everything up to itself,
// the others add the anchor and the groups after it, in order); pass 1 starts from that sum and writes the outputs,
// with the keys and values of the group still in L2 where the groups are small.  One launch; the sum does not depend
// on the order in which the CTAs run.  HBM-bound: q, k, v in, o out, 512 bytes per token.
//
// Warps (512 threads): 0 TMA producer; 1, 2, 3, 7 MMA issuers (scores, intra, update, inter: one thread gets an MMA
// out about every hundred cycles whatever its size, so every group of MMAs has its own); 4-6 state snapshot (TMEM
// -> bf16 rows in shared memory, 32 rows each) and state export; 4-7 state import; 8-15 weights and epilogue (two
// warps per lane quadrant, one per half of the columns).  All waits are bounded.
#include <cuda.h>

#include "kata_common.cuh"
#include "kata_tmap.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int CT = 128;            // tokens per tile
constexpr int NTHREADS = 512;
constexpr int NSTAGE = 3;
constexpr int SROWS = 80;          // state rows kept: 64 value columns, the normaliser row, 15 zero rows
constexpr int W_MMA_A = 1, W_MMA_B = 2, W_MMA_U = 3, W_SNAP0 = 4, W_MMA_R = 7, W_BLD0 = 8;

constexpr uint32_t COL_S = 0;      // 64 fp32: [S | Z]^T, lanes = (v, z, 0..), columns = feature a
constexpr uint32_t COL_P = 64;     // 2 x 128 fp32 scores; the bf16 weights overwrite columns [0,64) of a buffer
constexpr uint32_t COL_O = 320;    // 2 x 80: 64 outputs, column 64 = normaliser
constexpr uint32_t TMEM_COLS = 512;

constexpr uint32_t STAGE_BYTES = 49152;               // Q, K, V tiles of 16 KB, 128B swizzle
constexpr uint32_t OFF_ONES = NSTAGE * STAGE_BYTES;   // [128 tokens][64 columns] bf16: column 0 = 1, the rest 0
constexpr uint32_t OFF_SP = OFF_ONES + 16384;         // 2 x (80 rows x 128 B): state snapshots, K-major
constexpr uint32_t SP_BYTES = SROWS * 128;
constexpr uint32_t OFF_BAR = OFF_SP + 2 * SP_BYTES;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 256;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(SMEM_ALLOC > 116 * 1024, "one CTA per SM is assumed (the CTA allocates all of TMEM)");

// Every barrier has waiters that consume each of its phases in order, and no barrier can complete a second phase
// before its waiters have seen the first (a parity wait cannot tell phases two apart): where the producer of a
// phase does not depend on the waiter's progress, the barrier is split by buffer or committed once.
enum {
  BAR_FULL = 0,      // [3] tiles of the stage landed
  BAR_EMPTY = 3,     // [3] stage free: the issuers' commits
  BAR_S_FULL = 6,    // [2] scores in TMEM
  BAR_P_FULL = 8,    // [2] weights stored (256 threads)
  BAR_P_EMPTY = 10,  // [2] weights consumed by the intra MMA: the buffer may take new scores
  BAR_O_FULL = 12,   // [2] intra + inter result complete
  BAR_O_EMPTY = 14,  // [2] result read by the epilogue (256 threads)
  BAR_U_DONE = 16,   // state update of a tile complete (state-only pass: of the whole group)
  BAR_SNAP_LD = 17,  // state copied out of TMEM (96 threads): the next update may run
  BAR_SNAP_ST = 18,  // [2] snapshot stored into buffer 0 / 1 (96 threads): the inter MMA that reads it may run
  BAR_DRAIN = 20,
  BAR_R_DONE = 21,   // [2] inter-tile part of the result issued and complete: the intra MMAs may add to it
  BAR_COUNT = 23
};

struct OArgs {
  __nv_bfloat16* out;
  int* device_status;
  int Tlen;
  int n_tiles;
  int tiles_per_group;
  int n_groups;
  // more than one group: group states [BH][n_groups][80][64] of the groups alone and of the anchor groups with
  // everything before them, one flag per group, the ticket counter, B * H
  float* local_state;
  float* anchor_state;
  int* flags;
  unsigned* ticket;
  int BH;
};

constexpr int kAnchorEvery = 8;

// One fp32 state row (64 features) as a bf16 row of a snapshot (128B swizzle: chunk index xor row-in-atom).
__device__ __forceinline__ void snap_store_row(unsigned char* sp, int row, const uint32_t (&lo)[32], const uint32_t (&hi)[32]) {
  unsigned char* dst = sp + row * 128;
  const uint32_t rx = (uint32_t)row & 7u;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint32_t* z = c < 4 ? &lo[8 * c] : &hi[8 * (c - 4)];
    uint4 w;
    w.x = pack_bf16(__uint_as_float(z[0]), __uint_as_float(z[1]));
    w.y = pack_bf16(__uint_as_float(z[2]), __uint_as_float(z[3]));
    w.z = pack_bf16(__uint_as_float(z[4]), __uint_as_float(z[5]));
    w.w = pack_bf16(__uint_as_float(z[6]), __uint_as_float(z[7]));
    *reinterpret_cast<uint4*>(dst + (((uint32_t)c ^ rx) << 4)) = w;
  }
}

__global__ void __launch_bounds__(NTHREADS, 1)
tc_order1_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const OArgs args) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  auto bar = [&](int i) { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; };
  auto qtile = [&](int s) { return base + s * STAGE_BYTES; };
  auto ktile = [&](int s) { return base + s * STAGE_BYTES + 16384; };
  auto vtile = [&](int s) { return base + s * STAGE_BYTES + 32768; };
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool fused = args.flags != nullptr;
  constexpr size_t E = (size_t)SROWS * D;
  if (tid == 0) {
    abort_s = 0;
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  // the ones column (element 0 of chunk 0 of every token row of the static tile) and zeroed snapshots
  for (uint32_t i = tid; i < (16384 + 2 * SP_BYTES) / 16; i += NTHREADS)
    *reinterpret_cast<uint4*>(base + OFF_ONES + i * 16) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  if (tid < CT) *reinterpret_cast<uint16_t*>(base + OFF_ONES + sw128_offset(tid, 0)) = (uint16_t)0x3F80;
  fence_async_smem();
  if (warp == 0) {
    tmem_alloc(&tmem_base_s, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tmem_base_s;
  // More than one group: the CTAs take groups until none is left.  Groups are dealt in the order in which they are
  // asked for, earlier groups of every head first: the groups that a CTA waits for belong to CTAs that are working
  // on them or are done with them, whatever the size of the grid.
  __shared__ unsigned ticket_s;
  bool bars_live = false, dead = false;
  for (;;) {
  int bh = blockIdx.x, grp = 0;
  if (fused) {
    __syncthreads();
    if (tid == 0) ticket_s = atomicAdd(args.ticket, 1u);
    __syncthreads();
    if (ticket_s >= (unsigned)args.BH * (unsigned)args.n_groups) break;
    grp = (int)(ticket_s / (unsigned)args.BH);
    bh = (int)(ticket_s % (unsigned)args.BH);
  }
  const int t_begin = grp * args.tiles_per_group;
  const int n = min(args.n_tiles, t_begin + args.tiles_per_group) - t_begin;   // tiles of this group
  const size_t slot = (size_t)bh * args.n_groups + grp;
  // Pass 0 builds the state of the group alone (keys and values only) and publishes it, pass 1 starts from the sum
  // of the groups before it and writes the outputs; the last group of a head has no pass 0.
  const int pass_first = fused && grp + 1 < args.n_groups ? 0 : 1;
  for (int pass = pass_first; pass <= 1; ++pass) {
  bool ok = true;
  const bool wo = pass == 1;
  float* fin = pass == 0 ? args.local_state + slot * E : nullptr;
  const bool lookback = fused && pass == 1 && grp > 0;
  const bool resume = lookback;

  if (tid == 0) {
    // (one thread: initialising the barriers from as many threads at once gave barriers that did not work)
    if (bars_live)
      for (int i = 0; i < BAR_COUNT; ++i) mbar_inval(bar(i));
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(bar(BAR_FULL + i), 1);
      mbar_init(bar(BAR_EMPTY + i), wo ? 4 : 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_S_FULL + i), 1);
      mbar_init(bar(BAR_P_FULL + i), 256);
      mbar_init(bar(BAR_P_EMPTY + i), 1);
      mbar_init(bar(BAR_O_FULL + i), 1);
      mbar_init(bar(BAR_O_EMPTY + i), 256);
      mbar_init(bar(BAR_R_DONE + i), 1);
    }
    mbar_init(bar(BAR_U_DONE), 1);
    mbar_init(bar(BAR_SNAP_LD), 96);
    mbar_init(bar(BAR_SNAP_ST), 96);
    mbar_init(bar(BAR_SNAP_ST + 1), 96);
    mbar_init(bar(BAR_DRAIN), 4);
    fence_mbar_init();
  }
  __syncthreads();

  if (lookback) {
    // Look-back: the nearest anchor group at or before grp - 1 holds the sum of everything up to itself (group 0 is
    // its own anchor); the groups between it and this one are added in order, so the sum does not depend on who was
    // first.  All threads take part (the loads of up to eight group states are in flight together); the sum goes
    // through the first stage buffer, which is idle between the passes.  An anchor adds its own state for the groups
    // behind it.
    const int anchor = (grp - 1) / kAnchorEvery * kAnchorEvery;
    const int cnt = grp - anchor;                                   // 1 .. 8
    bool got = true;
    for (int g2 = anchor; g2 < grp && got; ++g2)
      got = wait_flag(args.flags + (slot - grp + g2), (g2 == anchor && anchor > 0) ? umma::kFlagAnchor : umma::kFlagLocal, abort_flag);
    const bool publish = grp % kAnchorEvery == 0 && grp + 1 < args.n_groups;
    float4* scratch = reinterpret_cast<float4*>(base);
    if (got) {
      for (int i = tid; i < (int)(E / 4); i += NTHREADS) {
        float4 part[kAnchorEvery];
#pragma unroll
        for (int u = 0; u < kAnchorEvery; ++u)
          if (u < cnt) {
            const float* sb = (u == 0 && anchor > 0) ? args.anchor_state : args.local_state;
            part[u] = __ldcg(reinterpret_cast<const float4*>(sb + (slot - grp + anchor + u) * E) + i);
          }
        float4 acc = part[0];
#pragma unroll
        for (int u = 1; u < kAnchorEvery; ++u)
          if (u < cnt) { acc.x += part[u].x; acc.y += part[u].y; acc.z += part[u].z; acc.w += part[u].w; }
        scratch[i] = acc;
        if (publish) {
          const float4 own = __ldcg(reinterpret_cast<const float4*>(args.local_state + slot * E) + i);
          reinterpret_cast<float4*>(args.anchor_state + slot * E)[i] = make_float4(acc.x + own.x, acc.y + own.y, acc.z + own.z, acc.w + own.w);
        }
      }
    }
    fence_async_smem();   // the stage buffer goes back to the TMA
    __syncthreads();
    if (publish && tid == 0) publish_flag(args.flags + slot, *abort_flag ? umma::kFlagPoison : umma::kFlagAnchor);
  }
  if (resume) {
    // the state before the first tile: into the accumulators and, as bf16, into snapshot 0
    if (warp >= W_SNAP0 && warp < W_SNAP0 + 4) {
      const uint32_t q4 = warp & 3;
      const int row = q4 * 32 + lane;
      uint32_t lo[32], hi[32];
      if (row < SROWS && !*abort_flag) {
        const float4* src = reinterpret_cast<const float4*>(base) + (size_t)row * (D / 4);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float4 a = src[c], b = src[8 + c];
          lo[4 * c] = __float_as_uint(a.x); lo[4 * c + 1] = __float_as_uint(a.y);
          lo[4 * c + 2] = __float_as_uint(a.z); lo[4 * c + 3] = __float_as_uint(a.w);
          hi[4 * c] = __float_as_uint(b.x); hi[4 * c + 1] = __float_as_uint(b.y);
          hi[4 * c + 2] = __float_as_uint(b.z); hi[4 * c + 3] = __float_as_uint(b.w);
        }
        snap_store_row(base + OFF_SP, row, lo, hi);
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) lo[c] = hi[c] = 0u;
      }
      tmem_st32(tmem_addr(tb, q4 * 32, COL_S), lo);
      tmem_st32(tmem_addr(tb, q4 * 32, COL_S + 32), hi);
      tmem_wait_st();
      fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*abort_flag) ok = false;
  }

  if (warp == 0) {
    // =========================== TMA producer ===========================
    if (lane == 0) {
      for (int j = 0; j < n && ok; ++j) {
        const int s = j % NSTAGE;
        ok = wait_or_abort_counted(bar(BAR_EMPTY + s), ((j / NSTAGE) & 1) ^ 1, abort_flag);
        if (!ok) break;
        const int tok = (t_begin + j) * CT;
        mbar_arrive_expect_tx(bar(BAR_FULL + s), wo ? 49152u : 32768u);
        if (wo) tma_load_3d(qtile(s), &tmQ, bar(BAR_FULL + s), 0, tok, bh);
        tma_load_3d(ktile(s), &tmK, bar(BAR_FULL + s), 0, tok, bh);
        tma_load_3d(vtile(s), &tmV, bar(BAR_FULL + s), 0, tok, bh);
      }
      // The barriers are initialised again for the next pass, so no arrival may still be on its way when this pass
      // ends: the last phases of the stage barriers, which no load waits for, are waited for here (a tcgen05.commit
      // arrives some time after its MMAs; only a completed phase says that all its arrivals are in).
      for (int j = (n > NSTAGE ? n - NSTAGE : 0); j < n && ok; ++j)      // the last tile of every stage that was used
        ok = wait_or_abort_counted(bar(BAR_EMPTY + j % NSTAGE), (j / NSTAGE) & 1, abort_flag);
    }
  } else if (warp == W_MMA_A) {
    // =========================== scores P = Q K^T ===========================
    // Four issuer warps, one per MMA group of a tile: a thread gets an MMA out about every hundred cycles whatever
    // its size, and the groups of a tile do not depend on one another.  Every lane waits, lane 0 issues (a warp of
    // waiters is woken sooner than a single waiting lane).
    if (wo) {
      const uint32_t idQK = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 128);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      for (int j = 0; j < n && ok; ++j) {
        const int s = j % NSTAGE, b = j & 1;
        ok = wait_or_abort_counted(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort_counted(bar(BAR_P_EMPTY + b), ((j >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          const uint32_t qa = smem_u32(qtile(s)), ka = smem_u32(ktile(s));
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            mma_f16_ss(tb + COL_P + b * 128, at(dk, qa + ks * 32), at(dk, ka + ks * 32), idQK, ks > 0);
          mma_commit(bar(BAR_S_FULL + b));
          mma_commit(bar(BAR_EMPTY + s));
        }
        __syncwarp();
      }
      // (as for the stage barriers: the weights barriers of the last two tiles, which no score MMA waits for)
      for (int j = n; j < n + 2 && ok; ++j)
        if (j >= 2) ok = wait_or_abort_counted(bar(BAR_P_EMPTY + (j & 1)), ((j >> 1) & 1) ^ 1, abort_flag);
    }
  } else if (warp == W_MMA_U) {
    // =========================== state update [S | Z]^T += [V | 1]^T K ===========================
    const uint32_t idU = instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 64);     // A and B MN-major (token = K)
    const uint32_t ones = smem_u32(base + OFF_ONES);
    for (int j = 0; j < n && ok; ++j) {
      const int s = j % NSTAGE;
      const bool upd = j + 1 < n || fin != nullptr;
      ok = wait_or_abort_counted(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag);
      // the accumulators are free once the snapshot of the previous state has left TMEM
      if (ok && upd && wo && j > 0) ok = wait_or_abort_counted(bar(BAR_SNAP_LD), (j - 1) & 1, abort_flag);
      if (!ok) break;
      if (lane == 0) {
        const uint32_t ka = smem_u32(ktile(s)), va = smem_u32(vtile(s));
        if (upd) {
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            // A: 8 tokens x 64 columns per 1 KB atom (SBO), columns 64..127 in the static ones tile (LBO);
            // B: the key tile, features on N
            mma_f16_ss(tb + COL_S, smem_desc(va + ks * 2048, ones - va, 1024, kSwizzle128B),
                       smem_desc(ka + ks * 2048, 16384, 1024, kSwizzle128B), idU, (resume || j > 0 || ks > 0) ? 1u : 0u);
          // state-only pass: nobody looks at the state between the tiles, one commit after the last update
          if (wo || j + 1 == n) mma_commit(bar(BAR_U_DONE));
        }
        mma_commit(bar(BAR_EMPTY + s));
      }
      __syncwarp();
    }
  } else if (warp == W_MMA_R) {
    // =========================== inter-tile part [O | D] = Q [S | Z]^T (opens the accumulator of the tile) ===========================
    if (wo) {
      const uint32_t idR = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 80);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      const uint32_t spa = smem_u32(base + OFF_SP);
      for (int j = 0; j < n && ok; ++j) {
        const int s = j % NSTAGE, b = j & 1;
        ok = wait_or_abort_counted(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort_counted(bar(BAR_O_EMPTY + b), ((j >> 1) & 1) ^ 1, abort_flag);
        // the snapshot after tile j - 1 went to buffer j & 1; it is that buffer's ((j - 1) / 2)-th
        if (ok && j > 0) ok = wait_or_abort_counted(bar(BAR_SNAP_ST + (j & 1)), ((j - 1) >> 1) & 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          if (resume || j > 0) {
            const uint32_t qa = smem_u32(qtile(s));
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_f16_ss(tb + COL_O + b * 80, at(dk, qa + ks * 32), at(dk, spa + (j & 1) * SP_BYTES + ks * 32), idR, ks > 0);
          }
          mma_commit(bar(BAR_R_DONE + b));
          mma_commit(bar(BAR_EMPTY + s));
        }
        __syncwarp();
      }
    }
  } else if (warp == W_MMA_B) {
    // =========================== intra-tile part [O | D] += P [V | 1] ===========================
    if (wo) {
      const uint32_t idPV = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 80);    // A tmem, B MN-major
      const uint32_t ones = smem_u32(base + OFF_ONES);
      for (int j = 0; j < n && ok; ++j) {
        const int s = j % NSTAGE, b = j & 1;
        ok = wait_or_abort_counted(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort_counted(bar(BAR_P_FULL + b), (j >> 1) & 1, abort_flag) &&
             wait_or_abort_counted(bar(BAR_R_DONE + b), (j >> 1) & 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          const uint32_t va = smem_u32(vtile(s));
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            mma_f16_ts(tb + COL_O + b * 80, tb + COL_P + b * 128 + ks * 8,
                       smem_desc(va + ks * 2048, ones - va, 1024, kSwizzle128B), idPV, (resume || j > 0 || ks > 0) ? 1u : 0u);
          mma_commit(bar(BAR_P_EMPTY + b));
          mma_commit(bar(BAR_O_FULL + b));
          mma_commit(bar(BAR_EMPTY + s));
        }
        __syncwarp();
      }
    }
  } else if (warp >= W_SNAP0 && warp < W_SNAP0 + 3) {
    // =========================== state snapshot / export (rows 0..95) ===========================
    const uint32_t q4 = warp & 3;
    const int row = q4 * 32 + lane;
    for (int j = wo ? 0 : n - 1; j < n && ok; ++j) {
      if (!(j + 1 < n || fin != nullptr)) break;          // the last update is skipped when nobody needs it
      ok = wait_or_abort_counted(bar(BAR_U_DONE), wo ? (j & 1) : 0, abort_flag);
      // the snapshot buffer written below was read by the inter MMA of tile j - 1
      if (ok && wo && j > 0 && j + 1 < n) ok = wait_or_abort_counted(bar(BAR_O_FULL + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      uint32_t lo[32], hi[32];
      if (wo && j + 1 < n) {
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S), lo);
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + 32), hi);
        tmem_wait_ld(lo);
        tmem_wait_ld(hi);
        tc_fence_before();
        mbar_arrive(bar(BAR_SNAP_LD));
        if (row < SROWS) snap_store_row(base + OFF_SP + ((j + 1) & 1) * SP_BYTES, row, lo, hi);
        fence_async_smem();
        mbar_arrive(bar(BAR_SNAP_ST + ((j + 1) & 1)));
      } else if (j + 1 == n) {
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S), lo);
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + 32), hi);
        tmem_wait_ld(lo);
        tmem_wait_ld(hi);
        if (row < SROWS) {
          float4* dst = reinterpret_cast<float4*>(fin + (size_t)row * D);
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            dst[c] = make_float4(__uint_as_float(lo[4 * c]), __uint_as_float(lo[4 * c + 1]), __uint_as_float(lo[4 * c + 2]),
                                 __uint_as_float(lo[4 * c + 3]));
            dst[8 + c] = make_float4(__uint_as_float(hi[4 * c]), __uint_as_float(hi[4 * c + 1]),
                                     __uint_as_float(hi[4 * c + 2]), __uint_as_float(hi[4 * c + 3]));
          }
        }
      }
    }
    if (fused && pass == 0) {
      // the group's own state is in place: tell the groups behind it
      asm volatile("bar.sync 6, 96;" ::: "memory");
      if (warp == W_SNAP0 && lane == 0) publish_flag(args.flags + slot, *abort_flag ? umma::kFlagPoison : umma::kFlagLocal);
    }
  } else if (warp >= W_BLD0 && wo) {
    // =========================== weights and epilogue (256 threads) ===========================
    const uint32_t q4 = warp & 3;
    const int ch = (warp - W_BLD0) >> 2;         // column half
    const int rowl = q4 * 32 + lane;             // token of the tile (= TMEM lane)
    auto epilogue = [&](int jj) -> bool {
      const int bb = jj & 1;
      if (!wait_or_abort_counted(bar(BAR_O_FULL + bb), (jj >> 1) & 1, abort_flag)) return false;
      tc_fence_after();
      uint32_t o[32], dn[16];
      tmem_ld32(tmem_addr(tb, q4 * 32, COL_O + bb * 80 + ch * 32), o);
      tmem_ld16(tmem_addr(tb, q4 * 32, COL_O + bb * 80 + 64), dn);
      tmem_wait_ld(o);
      tmem_wait_ld(dn);
      tc_fence_before();
      mbar_arrive(bar(BAR_O_EMPTY + bb));
      const float den = __uint_as_float(dn[0]);
      const float inv = den != 0.f ? 1.f / den : 0.f;
      const int tok = (t_begin + jj) * CT + rowl;
      if (tok < args.Tlen) {
        __nv_bfloat16* dst = args.out + ((size_t)bh * args.Tlen + tok) * D + ch * 32;
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint4 pkt;
          pkt.x = pack_bf16(__uint_as_float(o[c]) * inv, __uint_as_float(o[c + 1]) * inv);
          pkt.y = pack_bf16(__uint_as_float(o[c + 2]) * inv, __uint_as_float(o[c + 3]) * inv);
          pkt.z = pack_bf16(__uint_as_float(o[c + 4]) * inv, __uint_as_float(o[c + 5]) * inv);
          pkt.w = pack_bf16(__uint_as_float(o[c + 6]) * inv, __uint_as_float(o[c + 7]) * inv);
          *reinterpret_cast<uint4*>(dst + c) = pkt;
        }
      }
      return true;
    };
    for (int j = 0; j < n && ok; ++j) {
      const int b = j & 1;
      ok = wait_or_abort_counted(bar(BAR_S_FULL + b), (j >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t scol = tmem_addr(tb, q4 * 32, COL_P + b * 128 + ch * 64);
      uint32_t ya[32], yb[32], pk[32];
      tmem_ld32(scol, ya);
      tmem_ld32(scol + 32, yb);
      tmem_wait_ld(ya);
      tmem_wait_ld(yb);
      // causal mask inside the tile: key c contributes to token rowl when c <= rowl
#pragma unroll
      for (int c = 0; c < 32; c += 2) {
        const int k0 = ch * 64 + c, k1 = ch * 64 + 32 + c;
        pk[c / 2] = pack_bf16(k0 <= rowl ? __uint_as_float(ya[c]) : 0.f, k0 + 1 <= rowl ? __uint_as_float(ya[c + 1]) : 0.f);
        pk[16 + c / 2] = pack_bf16(k1 <= rowl ? __uint_as_float(yb[c]) : 0.f, k1 + 1 <= rowl ? __uint_as_float(yb[c + 1]) : 0.f);
      }
      // the weights overwrite score columns [0,64) of the buffer, which the column-half-0 warp of this
      // quadrant reads: both warps of the quadrant must have their scores in registers first
      tc_fence_before();
      asm volatile("bar.sync %0, 64;" ::"r"(1 + (int)q4) : "memory");
      tc_fence_after();
      tmem_st32(tmem_addr(tb, q4 * 32, COL_P + b * 128 + ch * 32), pk);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL + b));
      if (j > 0) ok = epilogue(j - 1);
    }
    if (ok) ok = epilogue(n - 1);
  }

  // ---------------- end of the pass ----------------
  if (!ok && args.device_status != nullptr) atomicExch(args.device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if ((warp == W_MMA_A || warp == W_MMA_B || warp == W_MMA_U || warp == W_MMA_R) && lane == 0) {
    mma_commit(bar(BAR_DRAIN));
    mbar_wait(bar(BAR_DRAIN), 0);
  }
  __syncthreads();
  bars_live = true;
  if (*abort_flag) {
    if (fused && tid == 0) publish_flag(args.flags + slot, umma::kFlagPoison);
    dead = true;
    break;
  }
  }
  if (!fused || dead) break;
  }
  if (warp == 0) tmem_dealloc(tb, TMEM_COLS);
}

}  // namespace

size_t tc_order1_state_elems() { return (size_t)SROWS * D; }
int tc_order1_tile() { return CT; }

// plan: groups of chunks of C tokens; every group but the last must cover whole 128-token tiles.
void tc_order1(const Problem& p, const ScanPlan& plan, bool use_scan, int C, float* ws, int* device_status,
               LaunchCtx& ctx) {
  const int BH = p.B * p.H;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_tile_map(&tmQ, p.q, BH, p.T, CT) || !make_tile_map(&tmK, p.k, BH, p.T, CT) || !make_tile_map(&tmV, p.v, BH, p.T, CT)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  if (cudaFuncSetAttribute(tc_order1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  OArgs a;
  a.out = static_cast<__nv_bfloat16*>(p.out);
  a.device_status = device_status;
  a.Tlen = p.T;
  a.n_tiles = (p.T + CT - 1) / CT;
  const int NG = use_scan ? plan.n_groups : 1;
  a.n_groups = NG;
  a.tiles_per_group = NG > 1 ? (int)((long long)plan.chunks_per_group * C / CT) : a.n_tiles;
  const size_t E = tc_order1_state_elems();
  float* bufA = ws;
  float* bufB = NG > 1 ? ws + (size_t)BH * NG * E : nullptr;
  a.local_state = nullptr;
  a.anchor_state = nullptr;
  a.flags = nullptr;
  a.ticket = nullptr;
  a.BH = BH;
  if (NG > 1) {
    // One launch: every CTA builds the state of its group alone, publishes it, adds up the groups before it (a chained
    // scan with an anchor every eight groups) and walks its tiles again, now with the keys and values in L2.
    int* flags = reinterpret_cast<int*>(ws + 2 * (size_t)BH * NG * E);
    if (cudaMemsetAsync(flags, 0, ((size_t)BH * NG + 1) * sizeof(int), ctx.stream) != cudaSuccess) {
      cudaGetLastError();
      ctx.status = KATA_ERR_CUDA;
      return;
    }
    a.local_state = bufA;
    a.anchor_state = bufB;
    a.flags = flags;
    a.ticket = reinterpret_cast<unsigned*>(flags + (size_t)BH * NG);
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      sms = 148;
    }
    const unsigned total = (unsigned)BH * NG;
    tc_order1_kernel<<<dim3(total < (unsigned)sms ? total : (unsigned)sms), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, tmV, a);
    note_launch(ctx);
    return;
  }
  // one group: one CTA per head walks all its tiles
  tc_order1_kernel<<<dim3(BH), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, tmV, a);
  note_launch(ctx);
}

}  // namespace kata
