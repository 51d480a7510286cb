// Chunked (linear-state) KATA forward on the Blackwell tensor cores, token-major, bf16, d_k = d_v = 64,
// whole sequence in one pass (the sequential inter-chunk recurrence of the chunked form).
//
// One CTA owns one head and a slice of 8 value columns and walks the sequence in tiles of 128 tokens.
// The feature state is never expanded: with k' = k / ||k||^2 the state of the slice is
//   S[(b,v), a] = sum_t k'[t,b] v[t,v] k[t,a]   and   Z[b, a] = sum_t k'[t,b] k[t,a]       (a, b < 64, v < 8)
// which is the rank-one lift <psi(q), psi(k)> = (q.k)^2 contracted in two stages.  S and Z are symmetric in
// (a, b), so only the 16 x 16 blocks with a-block <= b-block are kept (160 + 64 accumulator columns in TMEM).
// Per tile of 128 tokens:
//   update   S += W^T K          W[t,(b,v)] = k[t,b] v'[t,v] (v' = v / ||k||^2), one bf16 row per token, built
//                                by token threads in shared memory (MN-major A operand); B = the TMA-loaded
//                                key tile as it is; fp32 accumulators stay in TMEM for the whole sequence
//   snapshot S' = bf16(S)        after each update the accumulators are copied to shared memory as the B operand
//                                of the read (off-diagonal blocks doubled, which stands for the dropped half)
//   read     Y[t,(b,v)] = sum_a q[t,a] S'[(b,v),a]     tokens on the TMEM lanes, 8 pieces of 80 columns;
//            N_inter[t,v] = sum_b q[t,b] Y[t,(b,v)]    then is a dot product inside one thread
//   intra    P = (Q K^T)^2 masked causally, [O | D] += P [V' | 1/||k||^2]   as in the quadratic form
//   out      (N_inter + O) / (D_inter + D)             (0 where the denominator is 0)
// The query norm cancels and is never applied.
// Compiled three more times with KATA_STREAM_EXPORT and KATA_STREAM_MODE set (kept as separate builds so that the
// plain kernel's code stays as it is, and each build carries only what it needs):
//   mode 1 (kata_tc_stream_export.cu)   state before the first token / after the last token in the public layouts
//   mode 2 (kata_tc_stream_restart.cu)  a group of tiles restarted from a scanned prefix state (pass 3 of the scan forms)
//   mode 3 (kata_tc_stream_state.cu)    state only: what a group of tiles adds to the state (pass 1); no queries, no
//                                       reads, no intra tile, and a third key stage in the space they leave
//
// Warps (768 threads, 80 registers each): 0 TMA producer and update-MMA issuer (b-block 3, Z); 1 update-MMA
// issuer (b-blocks 0-2); 2 read-MMA issuer; 3 intra-tile MMA issuer; 4-11 W builders in two teams (even / odd
// 16-token steps into a ring of three buffers; warp = b-block, lanes = 16 tokens x 2 halves of the block), which
// also copy shares of the snapshot; 12-19 readers in two teams (even / odd read pieces, thread = token), the
// first team writes the output; 20-23 key scales, query tile to TMEM, weights P, the last share of the snapshot.
// The snapshot is double-buffered, so the reads of tile j + 1 overlap the update of tile j + 1; only the copy
// out of TMEM (twelve warps, at most 64 columns each) sits between two updates.  All waits are bounded.
#include <cuda.h>

#include "kata_common.cuh"
#include "kata_tmap.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int CT = 128;          // tokens per tile
constexpr int VS = 8;            // value columns per CTA
constexpr int NSLICE = D / VS;
constexpr int NTHREADS = 768;
constexpr int WARP_UB = 0, WARP_U = 1, WARP_R = 2, WARP_I = 3, WARP_BLD0 = 4, WARP_RD0 = 12, WARP_AUX0 = 20;

// ---- TMEM columns ----
constexpr uint32_t COL_S = 0;     // b-block beta at 8 beta (beta + 1): 16 (beta + 1) columns (a < 16 (beta + 1))
constexpr uint32_t COL_Z = 160;   // 64 columns, lanes 0..63 = b
constexpr uint32_t COL_Y = 224;   // 2 x 80: read pieces
constexpr uint32_t COL_P = 384;   // 64 fp32 scores; the bf16 weights overwrite columns [0,32)
constexpr uint32_t COL_O = 448;   // 16: intra-tile numerator (8) and denominator (column 8)
constexpr uint32_t COL_Q = 464;   // 32: the query tile as bf16 pairs
constexpr uint32_t TMEM_COLS = 512;

// ---- shared memory ----
constexpr uint32_t OFF_K = 0;             // 2 stages x K tile 16 KB, 128B swizzle
constexpr uint32_t OFF_Q = 32768;         // Q tile 16 KB (staging for the copy to TMEM)
constexpr uint32_t OFF_VP = 49152;        // 2 stages x 4 KB: [128 keys][8 bf16] v', then [128 keys][8 bf16] (1/||k||^2, 0..)
constexpr uint32_t OFF_W = 57344;         // 3 x 18 KB: [4 tiles][2 M-atoms][2 groups of 8 tokens][1 KB], then the Z rows
constexpr uint32_t W_BYTES = 18432;       //   [2 groups of 8 tokens][1 KB]; MN-major 128B swizzle
constexpr int NWBUF = 3;
constexpr uint32_t OFF_ZERO = 112640;     // 2 KB of zeros: the missing second M-atom of the Z tile
constexpr uint32_t OFF_SP = 114688;       // 2 x (5 blocks x 80 rows x 128 B): the snapshots, K-major 128B swizzle
constexpr uint32_t SP_BLOCK = 10240;
constexpr uint32_t SP_BYTES = 5 * SP_BLOCK;
constexpr uint32_t OFF_R2 = 217088;       // 2 stages x 128 x (bf16 1/||k||^2 twice)
constexpr uint32_t OFF_PART = 218112;     // 9 x 128 fp32: partial sums of the second reader team
constexpr uint32_t OFF_BAR = 222720;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 320;     // BAR_COUNT barriers and three more of the state-only build
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(OFF_W + NWBUF * W_BYTES == OFF_ZERO && OFF_ZERO + 2048 == OFF_SP, "layout");

// Blockwise map (Section 3.3) with G feature groups of 64 / G features: only the 16 x 16 state blocks whose a-block
// and b-block lie in the same group exist.  b-block beta keeps the a-blocks first(beta) .. beta.
template <int G>
struct Geo {
  static constexpr int BPG = 4 / G;                                       // b-blocks per feature group
  __host__ __device__ static constexpr int first(int beta) { return beta / BPG * BPG; }
  __host__ __device__ static constexpr int nblk(int beta) { return beta - first(beta) + 1; }
  __host__ __device__ static constexpr uint32_t col_s(int beta) {         // first accumulator column of b-block beta
    uint32_t c = 0;
    for (int i = 0; i < beta; ++i) c += 16u * nblk(i);
    return c;
  }
  static constexpr uint32_t Z = col_s(4);                                 // G = 1: 160, 2: 96, 4: 64
  static constexpr uint32_t Y = Z + 64;
  static constexpr uint32_t P = G == 1 ? 384u : Y + 160u;                 // scores of one intra-tile piece
  static constexpr int NP = G == 4 ? 4 : 2;                               // intra-tile pieces of KH keys:
  static constexpr int KH = CT / NP;                                      //   G x KH score columns (64, 128, 128)
  static_assert(P + G * KH <= 448, "TMEM columns");
};
static_assert(Geo<1>::col_s(1) == 16 && Geo<1>::col_s(2) == 48 && Geo<1>::col_s(3) == 96 && Geo<1>::Z == COL_Z &&
              Geo<1>::Y == COL_Y && Geo<1>::P == COL_P, "the plain feature keeps its layout");

// Every barrier has waiters that consume each of its phases in order.
enum {
  BAR_K_FULL = 0,     // [2] key tile landed
  BAR_K_EMPTY = 2,    // [2] stage free: the two update issuers' and the intra issuer's commits
  BAR_PREP = 4,       // [2] key scales and v' of the tile written
  BAR_QT_FULL = 6,    // query tile copied to TMEM
  BAR_W_FULL = 7,     // [3] W step built
  BAR_W_EMPTY = 10,   // [3] W step consumed
  BAR_U_DONE = 13,    // update of the tile complete
  BAR_R_DONE = 14,    // all read pieces of the tile complete
  BAR_SNAP_LD = 15,   // accumulators copied out of TMEM: the next update may run
  BAR_SNAP_ST = 16,   // snapshot stored: the next read may run
  BAR_Y_FULL = 17,    // [2]
  BAR_Y_EMPTY = 19,   // [2]
  BAR_S_FULL = 21,    // scores of a 64-key half in TMEM
  BAR_P_FULL = 22,    // weights of the half stored
  BAR_PV0 = 23,       // first half applied (its weights may be overwritten)
  BAR_O_FULL = 24,    // intra-tile result complete
  BAR_O_EMPTY = 25,   // intra-tile result read
  BAR_PART_FULL = 26, // partial sums of the second reader team written
  BAR_PART_EMPTY = 27,// ... and read
  BAR_Q_FULL = 28,    // query tile landed in shared memory
  BAR_QS_EMPTY = 29,  // ... and copied out of it
  BAR_Q_FREE = 30,    // the readers hold all their multipliers of the tile: the TMEM copy may be replaced
  BAR_DRAIN = 31,
  BAR_COUNT = 32
};

struct SArgs {
  const __nv_bfloat16* v;
  __nv_bfloat16* out;
  int* device_status;
  int Tlen;
#ifdef KATA_STREAM_EXPORT
  int layout;          // KATA_LAYOUT_DIRECT / KATA_LAYOUT_PACKED
  float* s_final;      // state after the last token, [BH][n_psi][64] in the public layout (null: not exported)
  float* z_final;      // [BH][n_psi]
  const float* s_init; // state before the first token, same layout (null: zero)
  const float* z_init;
  // groups of tiles (reduce-then-scan over the chunk axis): grid z = group
  const float* init_compact;   // [BH][n_groups][8 slices][224 columns][128 lanes]: group g starts from slot g - 1
  float* final_compact;        // same shape: the state a group leaves behind (null: not kept)
  int write_out;               // 0: state only (no queries, no output)
  int tiles_per_group;
  int n_groups;
#endif
};

__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmul2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Rounds 16 fp32 accumulator columns (scaled by sc) to bf16 and stores them as the 16-byte chunks c and c + 1 of a
// 128-byte snapshot row (128B swizzle: chunk index xor row-in-atom rx).
__device__ __forceinline__ void snap_store16(unsigned char* row, uint32_t c, uint32_t rx, const uint32_t* z, float sc) {
#pragma unroll
  for (int h8 = 0; h8 < 2; ++h8) {
    uint4 w;
    w.x = pack_bf16(__uint_as_float(z[8 * h8]) * sc, __uint_as_float(z[8 * h8 + 1]) * sc);
    w.y = pack_bf16(__uint_as_float(z[8 * h8 + 2]) * sc, __uint_as_float(z[8 * h8 + 3]) * sc);
    w.z = pack_bf16(__uint_as_float(z[8 * h8 + 4]) * sc, __uint_as_float(z[8 * h8 + 5]) * sc);
    w.w = pack_bf16(__uint_as_float(z[8 * h8 + 6]) * sc, __uint_as_float(z[8 * h8 + 7]) * sc);
    *reinterpret_cast<uint4*>(row + (((c + h8) ^ rx) << 4)) = w;
  }
}

// Snapshot placement of read piece p (8 values of b, b-block p / 2): block and byte offset inside the 128-byte rows.
// Pieces of the b-blocks 0 and 2 share rows (32 + 96 bytes), the two pieces of b-block 1 share rows (64 + 64).
__device__ __forceinline__ uint32_t sp_block(int p) { return (0x43102210u >> (4 * p)) & 0xFu; }   // 0,1,2,2,0,1,3,4
__device__ __forceinline__ uint32_t sp_koff(int p) { return p == 3 ? 64u : (p == 4 || p == 5) ? 32u : 0u; }

#ifdef KATA_STREAM_EXPORT
// Row of entry (a, b) of the exported state (a, b in the same feature group): the g blocks follow one another, each
// the direct m x m layout or the packed upper triangle (rows of la <= lb, off-diagonal entries times sqrt(2)).
template <int G>
__device__ __forceinline__ int state_row(int a, int b, bool packed) {
  constexpr int m = D / G;
  const int gb = a / m, la = a - gb * m, lb = b - gb * m;
  return packed ? gb * (m * (m + 1) / 2) + la * m - la * (la - 1) / 2 + (lb - la) : gb * m * m + la * m + lb;
}

// The state after the last token, from the TMEM accumulators to the public layout (one call per thread of the
// four auxiliary warps; kept out of line so that it does not weigh on the register allocation of the main loop).
template <int G>
__device__ __noinline__ void export_state(uint32_t tb, uint32_t q4, int t, float* s_final, float* z_final, int layout,
                                          int bh, int v0, int slice) {
  using geo = Geo<G>;
  tc_fence_after();
  const bool packed = layout == KATA_LAYOUT_PACKED;
  constexpr int m = D / G;
  const int n_psi = G * (packed ? m * (m + 1) / 2 : m * m);
  float* sf = s_final + (size_t)bh * n_psi * D + v0;
  const int vv = t & 7;
  uint32_t scol = tmem_addr(tb, q4 * 32, COL_S);
#pragma unroll 1
  for (int be = 0; be < 4; ++be) {
    const int b = 16 * be + (t >> 3);
#pragma unroll 1
    for (int al = geo::first(be); al <= be; ++al, scol += 16) {
      uint32_t z[16];
      tmem_ld16(scol, z);
      tmem_wait_ld(z);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int a = 16 * al + i;
        const float val = __uint_as_float(z[i]);
        if (packed) {
          if (a <= b) sf[(size_t)state_row<G>(a, b, true) * D + vv] = (a == b) ? val : val * 1.41421356237309504880f;
        } else {
          sf[(size_t)state_row<G>(a, b, false) * D + vv] = val;
          if (al < be) sf[(size_t)state_row<G>(b, a, false) * D + vv] = val;     // the dropped half of the symmetric state
        }
      }
    }
  }
  if (slice == 0 && q4 < 2) {
    float* zf = z_final + (size_t)bh * n_psi;
    const int b = t, bz = b >> 4, fz = geo::first(bz);
#pragma unroll 1
    for (int al = 0; al < 4; ++al) {      // the load is warp-wide: every lane walks all four a-blocks
      uint32_t z[16];
      tmem_ld16(tmem_addr(tb, q4 * 32, geo::Z + 16 * al), z);
      tmem_wait_ld(z);
      if (al < fz || al >= fz + geo::BPG) continue;      // a-block outside the feature group of this lane's b
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int a = 16 * al + i;
        const float val = __uint_as_float(z[i]);
        if (packed) {
          if (a <= b) zf[state_row<G>(a, b, true)] = (a == b) ? val : val * 1.41421356237309504880f;
        } else {
          zf[state_row<G>(a, b, false)] = val;
        }
      }
    }
  }
}

// The accumulators as they are (up to 224 columns x 128 lanes, column-major) for the scan over groups of tiles.
template <int G>
__device__ __noinline__ void export_compact(uint32_t tb, uint32_t q4, int t, float* dst) {
  tc_fence_after();
#pragma unroll 1
  for (int c = 0; c < (int)Geo<G>::Z + 64; c += 16) {
    uint32_t z[16];
    tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + c), z);
    tmem_wait_ld(z);
#pragma unroll
    for (int i = 0; i < 16; ++i) dst[(size_t)(c + i) * 128 + t] = __uint_as_float(z[i]);
  }
}

// The state before the first token, from the public layout (or, with comp, from the column-major copy of the
// accumulators that export_compact writes) into the TMEM accumulators (the inverse of export_state; same thread
// <-> row mapping), and its bf16 snapshot into snapshot buffer 0, which the reads of the first tile use.  One
// call per thread of the four auxiliary warps, before the pipeline starts.
template <int G>
__device__ __noinline__ void import_state(uint32_t tb, unsigned char* sp, uint32_t q4, int t, const float* s_init,
                                          const float* z_init, int layout, int bh, int v0, const float* comp) {
  using geo = Geo<G>;
  const bool packed = layout == KATA_LAYOUT_PACKED;
  constexpr int m = D / G;
  const int n_psi = G * (packed ? m * (m + 1) / 2 : m * m);
  const float* sf = comp ? nullptr : s_init + (size_t)bh * n_psi * D + v0;
  const float* zf = comp ? nullptr : z_init + (size_t)bh * n_psi;
  // entry (a, b) of the symmetric state: DIRECT its own row, PACKED the row of (min, max) with sqrt(2) taken out
  auto srow = [&](int a, int b, float& scale) -> int {
    if (!packed) { scale = 1.f; return state_row<G>(a, b, false); }
    const int lo = a < b ? a : b, hi = a < b ? b : a;
    scale = lo == hi ? 1.f : 0.70710678118654752440f;
    return state_row<G>(lo, hi, true);
  };
  const int bloc = t >> 3, vv = t & 7;
  uint32_t scol = tmem_addr(tb, q4 * 32, COL_S);
  int col = 0;
#pragma unroll 1
  for (int be = 0; be < 4; ++be) {
    const int b = 16 * be + bloc;
    const int p = 2 * be + (bloc >> 3);
    unsigned char* row = sp + sp_block(p) * SP_BLOCK + (bloc & 7) * 1024 + vv * 128;
#pragma unroll 1
    for (int al = geo::first(be); al <= be; ++al, scol += 16, col += 16) {
      uint32_t z[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (comp != nullptr) {
          z[i] = __float_as_uint(comp[(size_t)(col + i) * 128 + t]);
        } else {
          float scale;
          const int r = srow(16 * al + i, b, scale);
          z[i] = __float_as_uint(scale * sf[(size_t)r * D + vv]);
        }
      }
      tmem_st16(scol, z);
      snap_store16(row, (sp_koff(p) >> 4) + 2 * (al - geo::first(be)), (uint32_t)vv, z, al < be ? 2.f : 1.f);
    }
  }
  if (q4 < 2) {
    const int b = t, bz = b >> 4, fz = geo::first(bz), pz = b >> 3;
    unsigned char* rowz = sp + sp_block(pz) * SP_BLOCK + 8 * 1024 + (b & 7) * 128;
#pragma unroll 1
    for (int al = 0; al < 4; ++al) {
      const bool same = al >= fz && al < fz + geo::BPG;      // a-block in the feature group of b
      uint32_t z[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (comp != nullptr) {
          z[i] = __float_as_uint(comp[(size_t)(geo::Z + 16 * al + i) * 128 + t]);
        } else if (same) {
          float scale;
          const int r = srow(16 * al + i, b, scale);
          z[i] = __float_as_uint(scale * zf[r]);
        } else {
          z[i] = 0u;
        }
      }
      tmem_st16(tmem_addr(tb, q4 * 32, geo::Z + 16 * al), z);
      if (al >= fz && al <= bz) snap_store16(rowz, (sp_koff(pz) >> 4) + 2 * (al - fz), (uint32_t)(b & 7), z, al < bz ? 2.f : 1.f);
    }
  } else {
    // lanes 64..127 of the Z accumulators: rows of the zero atom, kept at zero
    uint32_t z[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) z[i] = 0u;
#pragma unroll 1
    for (int al = 0; al < 4; ++al) tmem_st16(tmem_addr(tb, q4 * 32, geo::Z + 16 * al), z);
  }
  tmem_wait_st();
  fence_async_smem();
}
#endif

template <int G>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_stream_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const SArgs args) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  auto bar = [&](int i) { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; };
  unsigned char* const qtile = base + OFF_Q;
  auto ktile = [&](int s) { return base + OFF_K + s * 16384; };
  auto wbuf = [&](int b) { return base + OFF_W + b * W_BYTES; };
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  using geo = Geo<G>;
  constexpr uint32_t COL_Z = geo::Z, COL_Y = geo::Y, COL_P = geo::P;     // (the namespace constants are those of G = 1)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slice = blockIdx.x, bh = blockIdx.y;
  const int v0 = slice * VS;
#ifdef KATA_STREAM_EXPORT
  // a group of tiles of the sequence (grid z); wo = false: only the state of the group is computed
  const int grp = blockIdx.z;
  const int t0 = grp * args.tiles_per_group;
  const int nch = min((args.Tlen + CT - 1) / CT, t0 + args.tiles_per_group) - t0;
  if (nch <= 0) return;
  constexpr bool wo = KATA_STREAM_MODE != 3;
#if KATA_STREAM_MODE != 1
  const size_t comp_elems = (size_t)224 * 128;
#endif
#if KATA_STREAM_MODE == 2
  const float* comp_in = (args.init_compact != nullptr && grp > 0)
      ? args.init_compact + ((((size_t)bh * args.n_groups + (grp - 1)) * NSLICE + slice) * comp_elems) : nullptr;
#endif
#if KATA_STREAM_MODE == 3
  float* comp_out = args.final_compact + ((((size_t)bh * args.n_groups + grp) * NSLICE + slice) * comp_elems);
#endif
#else
  constexpr int t0 = 0;
  constexpr bool wo = true;
  const int nch = (args.Tlen + CT - 1) / CT;
#endif
#if defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE == 3
  // The state-only build has the query and snapshot areas to spare: a third key stage (tile, scales, barriers), so
  // that a key tile is requested two tiles ahead (with two stages the chain stage free -> TMA -> key scales ->
  // first W step is as long as the tile itself).
  constexpr int NKS = 3;
  auto kst = [&](int j) { return j % 3; };
  auto kph = [&](int j) { return (uint32_t)((j / 3) & 1); };
  auto kfull = [&](int s) { return s < 2 ? bar(BAR_K_FULL + s) : bar(BAR_COUNT); };
  auto kempty = [&](int s) { return s < 2 ? bar(BAR_K_EMPTY + s) : bar(BAR_COUNT + 1); };
  auto kprep = [&](int s) { return s < 2 ? bar(BAR_PREP + s) : bar(BAR_COUNT + 2); };
  auto vptile = [&](int s) { return s < 2 ? base + OFF_VP + s * 4096 : base + OFF_SP; };
  auto r2pair = [&](int s) { return s < 2 ? reinterpret_cast<uint32_t*>(base + OFF_R2) + s * CT : reinterpret_cast<uint32_t*>(base + OFF_SP + 4096); };
#else
  constexpr int NKS = 2;
  auto kst = [&](int j) { return j & 1; };
  auto kph = [&](int j) { return (uint32_t)((j >> 1) & 1); };
  auto kfull = [&](int s) { return bar(BAR_K_FULL + s); };
  auto kempty = [&](int s) { return bar(BAR_K_EMPTY + s); };
  auto kprep = [&](int s) { return bar(BAR_PREP + s); };
  auto vptile = [&](int s) { return base + OFF_VP + s * 4096; };
  auto r2pair = [&](int s) { return reinterpret_cast<uint32_t*>(base + OFF_R2) + s * CT; };
#endif

  if (tid == 0) {
    abort_s = 0;
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(BAR_K_FULL + s), 1);
      mbar_init(bar(BAR_K_EMPTY + s), wo ? 3 : 2);
      mbar_init(bar(BAR_PREP + s), 128);
      mbar_init(bar(BAR_Y_FULL + s), 1);
      mbar_init(bar(BAR_Y_EMPTY + s), 128);
    }
    if (NKS == 3) {
      mbar_init(kfull(2), 1);
      mbar_init(kempty(2), 2);
      mbar_init(kprep(2), 128);
    }
    for (int s = 0; s < NWBUF; ++s) {
      mbar_init(bar(BAR_W_FULL + s), 128);
      mbar_init(bar(BAR_W_EMPTY + s), 2);
    }
    mbar_init(bar(BAR_QT_FULL), 128);
    mbar_init(bar(BAR_U_DONE), 2);
    mbar_init(bar(BAR_R_DONE), 1);
    mbar_init(bar(BAR_SNAP_LD), 384);
    mbar_init(bar(BAR_SNAP_ST), 384);
    mbar_init(bar(BAR_S_FULL), 1);
    mbar_init(bar(BAR_P_FULL), 128);
    mbar_init(bar(BAR_PV0), 1);
    mbar_init(bar(BAR_O_FULL), 1);
    mbar_init(bar(BAR_O_EMPTY), 128);
    mbar_init(bar(BAR_PART_FULL), 128);
    mbar_init(bar(BAR_PART_EMPTY), 128);
    mbar_init(bar(BAR_Q_FULL), 1);
    mbar_init(bar(BAR_QS_EMPTY), 128);
    mbar_init(bar(BAR_Q_FREE), 256);
    mbar_init(bar(BAR_DRAIN), 4);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
  }
  // zero: the zero atom of the Z tile and the snapshots (state 0, pad rows)
  for (uint32_t i = tid; i < (2048 + 2 * SP_BYTES) / 16; i += NTHREADS)
    *reinterpret_cast<uint4*>(base + OFF_ZERO + i * 16) = make_uint4(0u, 0u, 0u, 0u);
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
#if defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE != 3
  // accumulators and snapshot 0 start from a given state: the public one (mode 1) or a scanned prefix (mode 2)
#if KATA_STREAM_MODE == 1
  const bool resume = args.s_init != nullptr;
  const float* comp_in = nullptr;
#else
  const bool resume = comp_in != nullptr;
  // This build is launched as a programmatic dependent launch behind the scan rounds: up to here the CTA touched
  // only its own shared memory and TMEM; the prefix states are visible from here on.
  cudaGridDependencySynchronize();
#endif
  if (resume) {
    if (warp >= WARP_AUX0)
      import_state<G>(tb, base + OFF_SP, warp & 3, (warp & 3) * 32 + lane, args.s_init, args.z_init, args.layout, bh, v0,
                   comp_in);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }
#else
  constexpr bool resume = false;
#endif

  if (warp == WARP_UB || warp == WARP_U) {
    // =========================== update issuers: S += W^T K ===========================
    // Two threads share the MMAs of one 16-token step (their accumulators are disjoint): warp 1 the b-blocks
    // 0..2, warp 0 b-block 3 and Z.  Warp 0 is also the TMA producer of the query and key tiles.
    if (lane == 0) {
      // A: MN-major, 128B swizzle: 64 rows x 8 tokens per 1 KB atom; next 8 tokens +1 KB (SBO), next 64 rows +2 KB (LBO)
      const uint64_t dA = smem_desc(0, 2048, 1024, kSwizzle128B);
      // B: the key tile read MN-major (N = feature a, K = token): one atom of 64 features x 8 tokens per 1 KB
      const uint64_t dB = smem_desc(0, 16384, 1024, kSwizzle128B);
      const bool producer = (warp == WARP_UB);
      auto load_k = [&](int j) -> bool {
        const int s = kst(j);
        if (!wait_or_abort_counted(kempty(s), kph(j) ^ 1, abort_flag)) return false;
        mbar_arrive_expect_tx(kfull(s), 16384);
        tma_load_3d(ktile(s), &tmK, kfull(s), 0, (t0 + j) * CT, bh);
        return true;
      };
      auto load_q = [&](int j) -> bool {     // one staging buffer: free once the previous tile was copied to TMEM
        if (!wait_or_abort_counted(bar(BAR_QS_EMPTY), (j & 1) ^ 1, abort_flag)) return false;
        mbar_arrive_expect_tx(bar(BAR_Q_FULL), 16384);
        tma_load_3d(qtile, &tmQ, bar(BAR_Q_FULL), 0, (t0 + j) * CT, bh);
        return true;
      };
      if (producer) {
        ok = load_k(0) && (!wo || load_q(0));
        if (ok && nch > 1) ok = load_k(1);
        if (ok && NKS == 3 && nch > 2) ok = load_k(2);
      }
      uint32_t wbi = 0, wph = 0;             // W buffer of the step and the parity of its phase
      for (int j = 0; j < nch && ok; ++j) {
        const int s = kst(j);
        ok = wait_or_abort_counted(kfull(s), kph(j), abort_flag);
        if (ok && wo && j > 0) ok = wait_or_abort_counted(bar(BAR_SNAP_LD), (j - 1) & 1, abort_flag);
        // the key stage of tile j - 1 is free once that tile's consumers are through: refill it (with tile j + 1;
        // with tile j + 2 where there are three stages)
        if (ok && producer && j > 0 && j + NKS - 1 < nch) ok = load_k(j + NKS - 1);
#pragma unroll 1
        for (int sc = 0; sc < 8 && ok; ++sc) {
          ok = wait_or_abort_counted(bar(BAR_W_FULL + wbi), wph, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t wa = smem_u32(wbuf(wbi)), ka = smem_u32(ktile(s)) + sc * 2048;
          const uint64_t db = at(dB, ka);
          const uint32_t acc = (resume || j > 0 || sc > 0) ? 1u : 0u;
          // b-block beta: N = its a-blocks, the B operand starts at the first feature of its group (32 bytes per a-block)
          if (producer) {
            mma_f16_ss(tb + COL_S + geo::col_s(3), at(dA, wa + 3 * 4096), db + 2 * geo::first(3),
                       instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 16 * geo::nblk(3)), acc);
            // Z rows: 64 rows of this buffer, the other 64 rows of the tile read the zero atom (LBO reaches it)
            mma_f16_ss(tb + COL_Z, smem_desc(wa + 16384, smem_u32(base + OFF_ZERO) - (wa + 16384), 1024, kSwizzle128B), db,
                       instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 64), acc);
          } else {
            mma_f16_ss(tb + COL_S + 0, at(dA, wa), db, instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 16), acc);
            mma_f16_ss(tb + COL_S + geo::col_s(1), at(dA, wa + 4096), db + 2 * geo::first(1),
                       instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 16 * geo::nblk(1)), acc);
            mma_f16_ss(tb + COL_S + geo::col_s(2), at(dA, wa + 2 * 4096), db + 2 * geo::first(2),
                       instr_desc(kFmtBF16, kFmtBF16, 1, 1, 128, 16 * geo::nblk(2)), acc);
          }
          mma_commit(bar(BAR_W_EMPTY + wbi));
          if (++wbi == NWBUF) { wbi = 0; wph ^= 1; }
        }
        if (!ok) break;
        // state-only pass: nobody looks at the state between the tiles, one commit after the last update (a parity
        // wait cannot tell phases two apart)
        if (wo || j + 1 == nch) mma_commit(bar(BAR_U_DONE));
        mma_commit(kempty(s));
        // the query staging buffer is free once tile j was copied to TMEM (at the end of tile j - 1)
        if (producer && wo && j + 1 < nch) ok = load_q(j + 1);
      }
    }
  } else if (warp == WARP_R) {
    // =========================== read issuer: Y = Q S'^T, 8 pieces ===========================
    if (lane == 0 && wo) {
      const uint32_t idR = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 80);
      const uint64_t dS = smem_desc(0, 16, 1024, kSwizzle128B);
      const uint32_t spa = smem_u32(base + OFF_SP);
      for (int j = 0; j < nch && ok; ++j) {
        ok = wait_or_abort_counted(bar(BAR_QT_FULL), j & 1, abort_flag);
        if (ok && j > 0) ok = wait_or_abort_counted(bar(BAR_SNAP_ST), (j - 1) & 1, abort_flag);
#pragma unroll 1
        for (int p = 0; p < 8; ++p) {
          if (!ok) break;
          const int g = 8 * j + p, yb = g & 1;
          ok = wait_or_abort_counted(bar(BAR_Y_EMPTY + yb), ((g >> 1) & 1) ^ 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sbase = spa + (j & 1) * SP_BYTES + sp_block(p) * SP_BLOCK + sp_koff(p);
#pragma unroll 1
          for (int al = geo::first(p >> 1); al <= (p >> 1); ++al)
            mma_f16_ts(tb + COL_Y + yb * 80, tb + COL_Q + al * 8, at(dS, sbase + (al - geo::first(p >> 1)) * 32), idR,
                       al > geo::first(p >> 1));
          mma_commit(bar(BAR_Y_FULL + yb));
        }
        if (!ok) break;
        mma_commit(bar(BAR_R_DONE));
      }
    }
  } else if (warp == WARP_I) {
    // =========================== intra-tile issuer: scores and [O | D] ===========================
    if (lane == 0 && wo) {
      constexpr int NP = geo::NP, KH = geo::KH;
      const uint32_t idQK = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, KH);
      const uint32_t idPV = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 16);
      const uint64_t dK = smem_desc(0, 16, 1024, kSwizzle128B);
      for (int j = 0; j < nch && ok; ++j) {
        const int s = j & 1;
        ok = wait_or_abort_counted(bar(BAR_K_FULL + s), (j >> 1) & 1, abort_flag) &&
             wait_or_abort_counted(bar(BAR_QT_FULL), j & 1, abort_flag) &&
             wait_or_abort_counted(bar(BAR_PREP + s), (j >> 1) & 1, abort_flag);
        // the weights of the previous tile's second half are read by its last apply MMAs
        if (ok && j > 0) ok = wait_or_abort_counted(bar(BAR_O_FULL), (j - 1) & 1, abort_flag);
        const uint32_t ka = smem_u32(ktile(s)), va = smem_u32(vptile(s));
#pragma unroll
        for (int h = 0; h < NP; ++h) {
          if (!ok) break;
          // the weights of piece h - 1 alias the score columns: its apply MMAs must be through
          if (h > 0) ok = wait_or_abort_counted(bar(BAR_PV0), (j * (NP - 1) + h - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)   // 16 features per step; group ks / (4 / G) has its own KH score columns
            mma_f16_ts(tb + COL_P + (ks / (4 / G)) * KH, tb + COL_Q + ks * 8, at(dK, ka + h * KH * 128 + ks * 32), idQK,
                       (ks % (4 / G)) > 0);
          mma_commit(bar(BAR_S_FULL));
          ok = wait_or_abort_counted(bar(BAR_P_FULL), h & 1, abort_flag);
          if (ok && h == 0 && j > 0) ok = wait_or_abort_counted(bar(BAR_O_EMPTY), (j - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < KH / 16; ++ks)
            // MN-major, no swizzle: 8 keys x 16 bytes per core matrix, next 8 keys +128 (LBO), columns 8..15 +2048 (SBO)
            mma_f16_ts(tb + COL_O, tb + COL_P + ks * 8, smem_desc(va + h * KH * 16 + ks * 256, 128, 2048, kSwizzleNone), idPV,
                       (h > 0 || ks > 0) ? 1u : 0u);
          if (h < NP - 1) mma_commit(bar(BAR_PV0));
        }
        if (!ok) break;
        mma_commit(bar(BAR_O_FULL));
        mma_commit(bar(BAR_K_EMPTY + s));
      }
    }
  } else if (warp < WARP_RD0) {
    // =========================== W builders (+ shares of the snapshot) ===========================
    // Two teams of four warps: team 0 (warps 4-7) builds the even 16-token steps, team 1 the odd steps, into a
    // ring of three buffers.  Warp = b-block, lanes = 16 tokens x 2 halves of the block.
    const int beta = warp & 3;
    const int team = (warp - WARP_BLD0) >> 2;
    const uint32_t q4 = warp & 3;
    const int tk = lane & 15, half = lane >> 4;
    const int row_t = q4 * 32 + lane, bloc = row_t >> 3, vv = row_t & 7;    // snapshot: row of a state tile
    uint32_t wbi = team, wph = 0;                                           // buffer and phase parity of the next step
    // snapshot share of team 0: b-block 1 and the Z rows; of team 1: b-blocks 2 and 0 (b-block 3: warps 20-23).
    // The buffer written was read by the reads of tile jp - 1.  They are complete: warps 20-23 wait for them
    // before they scale tile jp + 1, and the callers have waited for those scales (BAR_PREP).
    auto snapshot_share = [&](int jp) -> bool {
      if (!wait_or_abort_counted(bar(BAR_U_DONE), jp & 1, abort_flag)) return false;
      tc_fence_after();
      unsigned char* sp = base + OFF_SP + ((jp + 1) & 1) * SP_BYTES;
      auto rowp = [&](int p) { return sp + sp_block(p) * SP_BLOCK + (bloc & 7) * 1024 + vv * 128; };
      if constexpr (G > 1) {
        // b-blocks 0 and 2 are diagonal blocks only; b-block 1 is [a-block 0 doubled | diagonal] for G = 2, diagonal
        // for G = 4; a Z row keeps the a-blocks of its group
        if (team == 1) {
          uint32_t e[16], c0[16];
          tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + geo::col_s(2)), e);
          tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + 0), c0);
          const int p2 = 4 + (bloc >> 3), p0 = bloc >> 3;
          tmem_wait_ld(e);
          tmem_wait_ld(c0);
          tc_fence_before();
          mbar_arrive(bar(BAR_SNAP_LD));
          snap_store16(rowp(p2), sp_koff(p2) >> 4, vv, e, 1.f);
          snap_store16(rowp(p0), sp_koff(p0) >> 4, vv, c0, 1.f);
        } else {
          uint32_t c1[16 * geo::nblk(1)];
          const uint32_t col1 = tmem_addr(tb, q4 * 32, COL_S + 16);
          if constexpr (geo::nblk(1) == 2) tmem_ld32(col1, c1); else tmem_ld16(col1, c1);
          const int p1 = 2 + (bloc >> 3);
          unsigned char* r1 = rowp(p1);
          const uint32_t k1 = sp_koff(p1) >> 4;
          auto store1 = [&]() {
            if constexpr (geo::nblk(1) == 2) {
              snap_store16(r1, k1, vv, c1, 2.f);
              snap_store16(r1, k1 + 2, vv, c1 + 16, 1.f);
            } else {
              snap_store16(r1, k1, vv, c1, 1.f);
            }
          };
          if (q4 < 2) {
            // Z rows: lane = b; row 64 + (b % 8) of piece b / 8
            uint32_t z0[32], z1[32];
            tmem_ld32(tmem_addr(tb, q4 * 32, COL_Z), z0);
            tmem_wait_ld(c1);
            store1();
            tmem_ld32(tmem_addr(tb, q4 * 32, COL_Z + 32), z1);
            tmem_wait_ld(z0);
            tmem_wait_ld(z1);
            tc_fence_before();
            mbar_arrive(bar(BAR_SNAP_LD));
            const int b = row_t, bz = b >> 4, fz = geo::first(bz), pz = b >> 3;
            unsigned char* rowz = sp + sp_block(pz) * SP_BLOCK + 8 * 1024 + (b & 7) * 128;
            const uint32_t cz = sp_koff(pz) >> 4;
            const uint32_t rz = (uint32_t)(b & 7);
#pragma unroll
            for (int al = 0; al < 4; ++al)
              if (al >= fz && al <= bz)
                snap_store16(rowz, cz + 2 * (al - fz), rz, (al < 2 ? z0 : z1) + 16 * (al & 1), al < bz ? 2.f : 1.f);
          } else {
            tmem_wait_ld(c1);
            tc_fence_before();
            mbar_arrive(bar(BAR_SNAP_LD));
            store1();
          }
        }
      } else if (team == 1) {
        uint32_t e[32], f[16], c0[16];
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + 48), e);
        tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + 80), f);
        tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + 0), c0);
        const int p2 = 4 + (bloc >> 3), p0 = bloc >> 3;
        unsigned char* row2 = rowp(p2);
        const uint32_t c2 = sp_koff(p2) >> 4;
        tmem_wait_ld(e);
        tmem_wait_ld(f);
        tmem_wait_ld(c0);
        tc_fence_before();
        mbar_arrive(bar(BAR_SNAP_LD));
        snap_store16(row2, c2, vv, e, 2.f);
        snap_store16(row2, c2 + 2, vv, e + 16, 2.f);
        snap_store16(row2, c2 + 4, vv, f, 1.f);
        snap_store16(rowp(p0), sp_koff(p0) >> 4, vv, c0, 1.f);
      } else {
        uint32_t c1[32];
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + 16), c1);
        const int p1 = 2 + (bloc >> 3);
        unsigned char* r1 = rowp(p1);
        const uint32_t k1 = sp_koff(p1) >> 4;
        if (q4 < 2) {
          // Z rows: lane = b; row 64 + (b % 8) of piece b / 8, features a < 16 (b / 16 + 1)
          uint32_t z0[32];
          tmem_ld32(tmem_addr(tb, q4 * 32, COL_Z), z0);
          tmem_wait_ld(c1);
          snap_store16(r1, k1, vv, c1, 2.f);
          snap_store16(r1, k1 + 2, vv, c1 + 16, 1.f);
          tmem_ld32(tmem_addr(tb, q4 * 32, COL_Z + 32), c1);
          tmem_wait_ld(z0);
          tmem_wait_ld(c1);
          tc_fence_before();
          mbar_arrive(bar(BAR_SNAP_LD));
          const int b = row_t, bz = b >> 4, pz = b >> 3;
          unsigned char* rowz = sp + sp_block(pz) * SP_BLOCK + 8 * 1024 + (b & 7) * 128;
          const uint32_t cz = sp_koff(pz) >> 4;
          const uint32_t rz = (uint32_t)(b & 7);
          snap_store16(rowz, cz, rz, z0, 0 < bz ? 2.f : 1.f);
          if (1 <= bz) snap_store16(rowz, cz + 2, rz, z0 + 16, 1 < bz ? 2.f : 1.f);
          if (2 <= bz) snap_store16(rowz, cz + 4, rz, c1, 2 < bz ? 2.f : 1.f);
          if (3 <= bz) snap_store16(rowz, cz + 6, rz, c1 + 16, 1.f);
        } else {
          tmem_wait_ld(c1);
          tc_fence_before();
          mbar_arrive(bar(BAR_SNAP_LD));
          snap_store16(r1, k1, vv, c1, 2.f);
          snap_store16(r1, k1 + 2, vv, c1 + 16, 1.f);
        }
      }
      fence_async_smem();
      mbar_arrive(bar(BAR_SNAP_ST));
      return true;
    };
    for (int j = 0; j < nch && ok; ++j) {
      const int s = kst(j);
      ok = wait_or_abort_counted(kfull(s), kph(j), abort_flag) && wait_or_abort_counted(kprep(s), kph(j), abort_flag);
      // team 1 copies its share of the state after tile j - 1 before its first step of tile j, team 0 after
      // its first step: either way right when the update of tile j - 1 completes
      if (ok && wo && team == 1 && j > 0) ok = snapshot_share(j - 1);
#pragma unroll 1
      for (int sc = team; sc < 8 && ok; sc += 2) {
        const int t = sc * 16 + tk;
        const uint4 kraw = *reinterpret_cast<const uint4*>(ktile(s) + sw128_offset(t, 2 * beta + half));
        const uint4 vp = *reinterpret_cast<const uint4*>(vptile(s) + t * 16);
        const uint32_t rr = r2pair(s)[t];
        const uint32_t kw[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
        ok = wait_or_abort_counted(bar(BAR_W_EMPTY + wbi), wph ^ 1, abort_flag);
        if (!ok) break;
        unsigned char* wrow = wbuf(wbi) + (tk >> 3) * 1024 + (tk & 7) * 128;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint32_t kbb = __byte_perm(kw[i >> 1], 0u, (i & 1) ? 0x3232 : 0x1010);
          uint4 w;
          w.x = mul_bf16x2(kbb, vp.x);
          w.y = mul_bf16x2(kbb, vp.y);
          w.z = mul_bf16x2(kbb, vp.z);
          w.w = mul_bf16x2(kbb, vp.w);
          *reinterpret_cast<uint4*>(wrow + beta * 4096 + half * 2048 + ((i ^ (tk & 7)) << 4)) = w;
        }
        {
          uint4 w;
          w.x = mul_bf16x2(kw[0], rr);
          w.y = mul_bf16x2(kw[1], rr);
          w.z = mul_bf16x2(kw[2], rr);
          w.w = mul_bf16x2(kw[3], rr);
          *reinterpret_cast<uint4*>(wrow + 16384 + (((2 * beta + half) ^ (tk & 7)) << 4)) = w;
        }
        fence_async_smem();
        mbar_arrive(bar(BAR_W_FULL + wbi));
        // this team's next step is two steps on: two buffers further in the ring of three
        wbi += 2;
        if (wbi >= NWBUF) { wbi -= NWBUF; wph ^= 1; }
        if (wo && sc == 0 && j > 0) ok = snapshot_share(j - 1);
      }
    }
  } else if (warp < WARP_AUX0) {
    // =========================== readers and epilogue (thread = token) ===========================
    // Two teams: team 0 (warps 12-15) folds the even pieces (TMEM buffer 0), team 1 the odd pieces (buffer 1)
    // and hands its partial sums to team 0 through shared memory; team 0 writes the output.
    const uint32_t q4 = warp & 3;
    const int team = (warp - WARP_RD0) >> 2;
    const int t = q4 * 32 + lane;
    float* part = reinterpret_cast<float*>(base + OFF_PART);
    const uint32_t ycol = tmem_addr(tb, q4 * 32, COL_Y + team * 80);
    for (int j = 0; j < nch && ok && wo; ++j) {
      ok = wait_or_abort_counted(bar(BAR_QT_FULL), j & 1, abort_flag);    // the multipliers come from the TMEM copy of the query tile
      if (!ok) break;
      tc_fence_after();
      float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      float accz = 0.f;
#pragma unroll 1
      for (int p = team; p < 8; p += 2) {
        const int g = 8 * j + p;
        // q[t, 8p .. 8p+7]: the multipliers of this piece
        uint32_t qw[4];
        tmem_ld4(tmem_addr(tb, q4 * 32, COL_Q + 4 * p), qw);
        tmem_wait_ld(qw);
        if (p >= 6) {          // last piece of this team: the query tile in TMEM may be replaced
          tc_fence_before();
          mbar_arrive(bar(BAR_Q_FREE));
        }
        ok = wait_or_abort_counted(bar(BAR_Y_FULL + team), (g >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        uint32_t y0[16], y1[16], y2[16];
        tmem_ld16(ycol, y0);
        tmem_ld16(ycol + 16, y1);
        tmem_ld16(ycol + 32, y2);
        auto fold = [&](const uint32_t (&y)[16], int i0) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const int b = i0 + i;
            const float qb = (b & 1) ? bf_hi(qw[b >> 1]) : bf_lo(qw[b >> 1]);
            const float2 qq = make_float2(qb, qb);
#pragma unroll
            for (int vv = 0; vv < 4; ++vv)
              acc[vv] = __ffma2_rn(qq, make_float2(__uint_as_float(y[8 * i + 2 * vv]), __uint_as_float(y[8 * i + 2 * vv + 1])),
                                   acc[vv]);
          }
        };
        tmem_wait_ld(y0);
        fold(y0, 0);
        tmem_ld16(ycol + 48, y0);
        tmem_wait_ld(y1);
        fold(y1, 2);
        tmem_ld16(ycol + 64, y1);
        tmem_wait_ld(y2);
        fold(y2, 4);
        tmem_wait_ld(y0);
        fold(y0, 6);
        tmem_wait_ld(y1);
        tc_fence_before();
        mbar_arrive(bar(BAR_Y_EMPTY + team));
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float qb = (i & 1) ? bf_hi(qw[i >> 1]) : bf_lo(qw[i >> 1]);
          accz = fmaf(qb, __uint_as_float(y1[i]), accz);
        }
      }
      if (!ok) break;
      if (team == 1) {
        ok = wait_or_abort_counted(bar(BAR_PART_EMPTY), (j & 1) ^ 1, abort_flag);
        if (!ok) break;
        part[0 * CT + t] = acc[0].x; part[1 * CT + t] = acc[0].y;
        part[2 * CT + t] = acc[1].x; part[3 * CT + t] = acc[1].y;
        part[4 * CT + t] = acc[2].x; part[5 * CT + t] = acc[2].y;
        part[6 * CT + t] = acc[3].x; part[7 * CT + t] = acc[3].y;
        part[8 * CT + t] = accz;
        mbar_arrive(bar(BAR_PART_FULL));
        continue;
      }
      ok = wait_or_abort_counted(bar(BAR_PART_FULL), j & 1, abort_flag);
      if (!ok) break;
      acc[0].x += part[0 * CT + t]; acc[0].y += part[1 * CT + t];
      acc[1].x += part[2 * CT + t]; acc[1].y += part[3 * CT + t];
      acc[2].x += part[4 * CT + t]; acc[2].y += part[5 * CT + t];
      acc[3].x += part[6 * CT + t]; acc[3].y += part[7 * CT + t];
      accz += part[8 * CT + t];
      mbar_arrive(bar(BAR_PART_EMPTY));
      ok = wait_or_abort_counted(bar(BAR_O_FULL), j & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      uint32_t o[16];
      tmem_ld16(tmem_addr(tb, q4 * 32, COL_O), o);
      tmem_wait_ld(o);
      tc_fence_before();
      mbar_arrive(bar(BAR_O_EMPTY));
      const float den = accz + __uint_as_float(o[8]);
      const float inv = den > 0.f ? 1.f / den : 0.f;
      const int tok = (t0 + j) * CT + t;
      if (tok < args.Tlen) {
        uint4 pkt;
        pkt.x = pack_bf16((acc[0].x + __uint_as_float(o[0])) * inv, (acc[0].y + __uint_as_float(o[1])) * inv);
        pkt.y = pack_bf16((acc[1].x + __uint_as_float(o[2])) * inv, (acc[1].y + __uint_as_float(o[3])) * inv);
        pkt.z = pack_bf16((acc[2].x + __uint_as_float(o[4])) * inv, (acc[2].y + __uint_as_float(o[5])) * inv);
        pkt.w = pack_bf16((acc[3].x + __uint_as_float(o[6])) * inv, (acc[3].y + __uint_as_float(o[7])) * inv);
        *reinterpret_cast<uint4*>(args.out + ((size_t)bh * args.Tlen + tok) * D + v0) = pkt;
      }
    }
  } else {
    // =========================== key scales, query tile, weights, snapshot ===========================
    const uint32_t q4 = warp & 3;
    const int t = q4 * 32 + lane;       // token of the tile, and TMEM lane
    auto load_v = [&](int j) -> uint4 {
      const int tok = (t0 + j) * CT + t;
      if (j < nch && tok < args.Tlen)
        return *reinterpret_cast<const uint4*>(args.v + ((size_t)bh * args.Tlen + tok) * D + v0);
      return make_uint4(0u, 0u, 0u, 0u);
    };
    // key scales and v' of tile j (the value slice was fetched one tile earlier)
    auto prep = [&](int j, const uint4& vraw) -> bool {
      const int s = kst(j);
      if (!wait_or_abort_counted(kfull(s), kph(j), abort_flag)) return false;
      float ss = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(ktile(s) + sw128_offset(t, c));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          ss = fmaf(bf_lo(w[e]), bf_lo(w[e]), ss);
          ss = fmaf(bf_hi(w[e]), bf_hi(w[e]), ss);
        }
      }
      const float r2 = inv_or_zero(ss);
      uint4 vp;
      vp.x = pack_bf16(bf_lo(vraw.x) * r2, bf_hi(vraw.x) * r2);
      vp.y = pack_bf16(bf_lo(vraw.y) * r2, bf_hi(vraw.y) * r2);
      vp.z = pack_bf16(bf_lo(vraw.z) * r2, bf_hi(vraw.z) * r2);
      vp.w = pack_bf16(bf_lo(vraw.w) * r2, bf_hi(vraw.w) * r2);
      *reinterpret_cast<uint4*>(vptile(s) + t * 16) = vp;
      const uint32_t rb = pack_bf16(r2, r2);
      *reinterpret_cast<uint4*>(vptile(s) + 2048 + t * 16) = make_uint4(rb & 0xFFFFu, 0u, 0u, 0u);
      r2pair(s)[t] = rb;
      fence_async_smem();
      mbar_arrive(kprep(s));
      return true;
    };
    // this warp's share of the snapshot of the state after tile j (b-block 3; the other blocks and Z: warps 4-11);
    // the update of tile j is complete (BAR_U_DONE observed by the caller)
    auto snapshot_share = [&](int j) {
      tc_fence_after();
      const int bloc = t >> 3, vv = t & 7;          // row of a state tile = 8 * (b within the block) + v
      unsigned char* sp = base + OFF_SP + ((j + 1) & 1) * SP_BYTES;
      const int p3 = 6 + (bloc >> 3);
      unsigned char* r3 = sp + sp_block(p3) * SP_BLOCK + (bloc & 7) * 1024 + vv * 128;
      if constexpr (G == 1) {
        uint32_t a0[32], a1[32];
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + 96), a0);
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + 128), a1);
        tmem_wait_ld(a0);
        tmem_wait_ld(a1);
        tc_fence_before();
        mbar_arrive(bar(BAR_SNAP_LD));
        snap_store16(r3, 0, vv, a0, 2.f);
        snap_store16(r3, 2, vv, a0 + 16, 2.f);
        snap_store16(r3, 4, vv, a1, 2.f);
        snap_store16(r3, 6, vv, a1 + 16, 1.f);
      } else if constexpr (G == 2) {      // [a-block 2 doubled | diagonal]
        uint32_t a0[32];
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_S + geo::col_s(3)), a0);
        tmem_wait_ld(a0);
        tc_fence_before();
        mbar_arrive(bar(BAR_SNAP_LD));
        snap_store16(r3, 0, vv, a0, 2.f);
        snap_store16(r3, 2, vv, a0 + 16, 1.f);
      } else {                            // the diagonal block
        uint32_t a0[16];
        tmem_ld16(tmem_addr(tb, q4 * 32, COL_S + geo::col_s(3)), a0);
        tmem_wait_ld(a0);
        tc_fence_before();
        mbar_arrive(bar(BAR_SNAP_LD));
        snap_store16(r3, 0, vv, a0, 1.f);
      }
      fence_async_smem();
      mbar_arrive(bar(BAR_SNAP_ST));
    };
    uint4 vnext = load_v(0);
    if (!wo) {
      // state-only pass: key scales and v' of every tile, nothing else
      for (int j = 0; j < nch && ok; ++j) {
        ok = prep(j, vnext);
        vnext = load_v(j + 1);
      }
    }
    for (int j = -1; j < nch && ok && wo; ++j) {
      // ---- scales of the next tile, so that its W rows can be built during this tile's update ----
      if (j + 1 < nch) {
        ok = prep(j + 1, vnext);
        if (!ok) break;
        vnext = load_v(j + 2);
      }
      bool snapped = (j < 0) || (j + 1 >= nch);      // nothing to copy before the first and after the last tile
      // ---- weights P = (q.k)^2, causal, two halves of 64 keys ----
      if (j >= 0) {
#pragma unroll 1
        for (int h = 0; h < geo::NP; ++h) {
          // The copy of the state out of TMEM sits between two updates: serve it first when the update
          // completes while this warp waits for scores.
          ok = false;
          for (uint32_t i = 0; i < kSpinLimit; ++i) {
            if (mbar_test_wait(bar(BAR_S_FULL), h & 1)) { ok = true; break; }
            if (!snapped && mbar_test_wait(bar(BAR_U_DONE), j & 1)) { snapshot_share(j); snapped = true; }
            __nanosleep(64);
            if ((i & 1023u) == 1023u && *abort_flag) break;
          }
          if (!ok) { *abort_flag = 1; break; }
          tc_fence_after();
          const uint32_t scol = tmem_addr(tb, q4 * 32, COL_P);
          if constexpr (G > 1) {
            // 16 keys at a time: the weight of a key is the sum over the groups of its squared scores (group g in
            // columns [g KH, g KH + KH)).  The bf16 weights of keys [16 i, 16 i + 16) go to columns [8 i, 8 i + 8),
            // group-0 scores that this thread has read already.
            constexpr int KH = geo::KH;
#pragma unroll 1
            for (int i = 0; i < KH / 16; ++i) {
              float2 w[8];
              uint32_t y[16], pk[8];
#pragma unroll
              for (int g = 0; g < G; ++g) {
                tmem_ld16(scol + g * KH + 16 * i, y);
                tmem_wait_ld(y);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const float2 sv = make_float2(__uint_as_float(y[2 * e]), __uint_as_float(y[2 * e + 1]));
                  w[e] = g == 0 ? __fmul2_rn(sv, sv) : __ffma2_rn(sv, sv, w[e]);
                }
              }
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const int c = h * KH + 16 * i + 2 * e;
                if (c > t) w[e].x = 0.f;
                if (c + 1 > t) w[e].y = 0.f;
                pk[e] = pack_bf16(w[e].x, w[e].y);
              }
              tmem_st8(scol + 8 * i, pk);
            }
          } else {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t y[32], pk[16];
            tmem_ld32(scol + half * 32, y);
            tmem_wait_ld(y);
#pragma unroll
            for (int jj = 0; jj < 32; jj += 2) {
              const int c = h * 64 + half * 32 + jj;
              const float2 sv = make_float2(__uint_as_float(y[jj]), __uint_as_float(y[jj + 1]));
              float2 w = __fmul2_rn(sv, sv);
              if (c > t) w.x = 0.f;
              if (c + 1 > t) w.y = 0.f;
              pk[jj / 2] = pack_bf16(w.x, w.y);
            }
            tmem_st16(scol + half * 16, pk);
          }
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(bar(BAR_P_FULL));
        }
        if (!ok) break;
      }
      if (j + 1 >= nch) break;
      if (!snapped) {
        ok = wait_or_abort_counted(bar(BAR_U_DONE), j & 1, abort_flag);
        if (!ok) break;
        snapshot_share(j);
      }
      // ---- query tile j + 1 to TMEM, once the reads of tile j are complete, the readers hold their multipliers
      //      (the scores of tile j are complete: see above) and the tile has landed ----
      {
        if (j >= 0) ok = wait_or_abort_counted(bar(BAR_R_DONE), j & 1, abort_flag) && wait_or_abort_counted(bar(BAR_Q_FREE), j & 1, abort_flag);
        if (ok) ok = wait_or_abort_counted(bar(BAR_Q_FULL), (j + 1) & 1, abort_flag);
        if (!ok) break;
        uint32_t qw[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 raw = *reinterpret_cast<const uint4*>(qtile + sw128_offset(t, c));
          qw[4 * c] = raw.x; qw[4 * c + 1] = raw.y; qw[4 * c + 2] = raw.z; qw[4 * c + 3] = raw.w;
        }
        mbar_arrive(bar(BAR_QS_EMPTY));
        tc_fence_after();
        tmem_st32(tmem_addr(tb, q4 * 32, COL_Q), qw);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_QT_FULL));
      }
    }
#if defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE == 1
    // ---- the state after the last token, from the accumulators to the public layout ----
    if (ok && args.s_final != nullptr) {
      ok = wait_or_abort_counted(bar(BAR_U_DONE), (nch - 1) & 1, abort_flag);
      if (ok) export_state<G>(tb, q4, t, args.s_final, args.z_final, args.layout, bh, v0, slice);
    }
#elif defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE == 3
    // ---- what the group adds to the state: the accumulators as they are (the one commit of this build's updates) ----
    if (ok) {
      ok = wait_or_abort_counted(bar(BAR_U_DONE), 0, abort_flag);
      if (ok) export_compact<G>(tb, q4, t, comp_out);
    }
#endif
  }

  // ---------------- teardown ----------------
  if (!ok && args.device_status != nullptr) atomicExch(args.device_status, (int)KATA_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp <= WARP_I && lane == 0) {
    mma_commit(bar(BAR_DRAIN));
    mbar_wait(bar(BAR_DRAIN), 0);
  }
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
}  // namespace

#if defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE == 1
size_t tc_stream_state_elems() { return (size_t)NSLICE * 224 * 128; }
int tc_stream_slices() { return NSLICE; }
int tc_stream_tile() { return CT; }

void tc_chunked_stream_export(const Problem& p, int* device_status, const StreamIO& io, LaunchCtx& ctx) {
#elif defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE == 2
void tc_chunked_stream_restart(const Problem& p, int* device_status, const StreamIO& io, LaunchCtx& ctx) {
#elif defined(KATA_STREAM_EXPORT) && KATA_STREAM_MODE == 3
void tc_chunked_stream_state(const Problem& p, int* device_status, const StreamIO& io, LaunchCtx& ctx) {
#else
void tc_chunked_stream(const Problem& p, int* device_status, LaunchCtx& ctx) {
#endif
  const int BH = p.B * p.H;
  CUtensorMap tmQ, tmK;
  if (!make_tile_map(&tmQ, p.q, BH, p.T, CT) || !make_tile_map(&tmK, p.k, BH, p.T, CT)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  auto kern = p.groups == 1 ? tc_stream_kernel<1> : p.groups == 2 ? tc_stream_kernel<2> : tc_stream_kernel<4>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
#ifdef KATA_STREAM_EXPORT
  const int n_tiles = (p.T + CT - 1) / CT;
  const int n_groups = io.n_groups > 0 ? io.n_groups : 1;
  SArgs a{static_cast<const __nv_bfloat16*>(p.v), static_cast<__nv_bfloat16*>(p.out), device_status, p.T, io.layout,
          io.s_final, io.z_final, io.s_init, io.z_init, io.init_compact, io.final_compact, io.write_out,
          io.n_groups > 0 ? io.tiles_per_group : n_tiles, n_groups};
  const int launch_groups = io.launch_groups > 0 ? io.launch_groups : n_groups;
#if KATA_STREAM_MODE == 2
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(NSLICE, BH, launch_groups);
  cfg.blockDim = dim3(NTHREADS);
  cfg.dynamicSmemBytes = SMEM_ALLOC;
  cfg.stream = ctx.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, tmQ, tmK, a) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  ++ctx.launches;
  return;
#else
  kern<<<dim3(NSLICE, BH, launch_groups), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, a);
#endif
#else
  SArgs a{static_cast<const __nv_bfloat16*>(p.v), static_cast<__nv_bfloat16*>(p.out), device_status, p.T};
  kern<<<dim3(NSLICE, BH, 1), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, a);
#endif
  note_launch(ctx);
}

}  // namespace kata
