// Backward of the quadratic form on the Blackwell tensor cores: bf16, d_k = d_v = 64, full rank-one feature.
//
// With s_ti = q_t . k_i, r_i = 1/||k_i||^2, a_ti = r_i s_ti^2 (i <= t), D_t = sum_i a_ti, o_t = sum_i a_ti v_i / D_t:
//   c_ti = dout_t . v_i,   g_ti = (c_ti - dout_t . o_t) / D_t,   e_ti = 2 g_ti s_ti,   p_ti = s_ti^2 / D_t
//   dq_t = sum_i e_ti k'_i                       (k' = r k, written by the pre-pass)
//   dv_i = r_i sum_t p_ti dout_t
//   dk_i = r_i (u_i - r_i (k_i . u_i) k_i),  u_i = sum_t e_ti q_t      (the second term is the derivative of r_i; it
//                                                                       makes dk_i orthogonal to k_i: o has degree 0 in k_i)
// A pre-pass writes k' and r; then one kernel in two modes, both with a fixed tile of 128 rows on the TMEM lanes and
// tiles of 64 rows streamed past it:
//   MODE_DQ   fixed = 128 queries (Q, dout), streamed = keys (K, V, K', r), twice:  S = Q K^T, C = dout V^T (SS MMAs,
//             N = 64); in the first sweep the weight warps sum D_t = sum_i r_i s^2 and sum_i r_i s^2 c in fp32 (the
//             same weights in both, so dout_t . o_t is consistent with c: their difference is what the gradient is
//             made of) and leave (1/D_t, dout_t . o_t) in the workspace; in the second sweep they form E, and
//             dq += E K' (A = E from TMEM)
//   MODE_DKV  fixed = 128 keys (K, V), streamed = queries (Q, dout, their scalars):  S^T = K Q^T, C^T = V dout^T,
//             the weight warps form P^T and E^T with the scalars of the columns, then dv~ += P^T dout, u += E^T Q
//             (B = the streamed tiles read MN-major), and the epilogue applies r_i and the projection.
// No atomics, every sum in a fixed order.  Warps (384 threads): 0 TMA producer, 1 score-MMA issuer, 2 output-MMA
// issuer, 4-11 weights and epilogue.  All waits are bounded.
#include <cuda.h>
#include <type_traits>

#include "kata_common.cuh"
#include "kata_tmap.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int MT = 128;          // rows of the fixed tile (TMEM lanes)
constexpr int NT = 64;           // rows of a streamed tile
constexpr int NSTAGE = 4;
constexpr int NBUF_MAX = 3;
constexpr int NTHREADS = 384;
constexpr int WARP_BLD0 = 4;
enum { MODE_DQ = 0, MODE_DKV = 1 };

constexpr uint32_t COL_B = 0;      // score buffers of (G + 1) x 64 fp32 columns: [S_0 | .. | S_{G-1} | C] of a streamed tile
                                   // (G feature groups; three buffers for G = 1, two for G = 2, one for G = 4); the
                                   // bf16 weights overwrite columns [0,32) of each block
constexpr uint32_t COL_ACC = 384;  // 2 x 64 fp32 accumulators
constexpr uint32_t TMEM_COLS = 512;

constexpr uint32_t OFF_X1 = 0;                     // fixed tiles: 128 x 64 bf16, 128B swizzle
constexpr uint32_t OFF_X2 = 16384;
constexpr uint32_t OFF_ST = 32768;                 // stages: two streamed tiles of 8 KB, then K' (MODE_DQ)
constexpr uint32_t STAGE_BYTES = 24576;
constexpr uint32_t OFF_SC = OFF_ST + NSTAGE * STAGE_BYTES;   // per stage 512 bytes of scalars of the 64 streamed rows:
                                                             // r_i (MODE_DQ) or (1/D_t, dout_t . o_t) (MODE_DKV)
constexpr uint32_t OFF_PART = OFF_SC + NSTAGE * 512;         // 2 x 128 float2: the column halves of a row meet here
constexpr uint32_t OFF_BAR = OFF_PART + 2048;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 256;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(SMEM_ALLOC > 116 * 1024, "one CTA per SM is assumed (the CTA allocates all of TMEM)");

// Every barrier has waiters that consume each of its phases in order; a producer of a phase always depends on the
// waiter's progress (no barrier can complete two phases ahead of a waiter).
enum {
  BAR_XFULL = 0,     // fixed tiles landed
  BAR_FULL = 1,      // [4] streamed tiles landed (TMA bytes + 32 producer lanes)
  BAR_EMPTY = 5,     // [4] stage free: both issuers' commits
  BAR_SFULL = 9,     // [3] scores in TMEM
  BAR_PFULL = 12,    // [3] weights stored (256 threads)
  BAR_PEMPTY = 15,   // [3] weights consumed: the buffer may take new scores
  BAR_ODONE = 18,
  BAR_DRAIN = 19,
  BAR_COUNT = 20
};

struct BArgs {
  __nv_bfloat16* out0;       // MODE_DQ: dq;  MODE_DKV: dk
  __nv_bfloat16* out1;       // MODE_DKV: dv
  float* stats;              // [BH][T][2]: 1 / D_t, dout_t . o_t (written by MODE_DQ, read by MODE_DKV)
  const float* rk;           // [BH][T]: 1 / ||k_i||^2
  int* device_status;
  int Tlen;
};

// G feature groups of the blockwise map: s_g = q_g . k_g per group, a = r sum_g s_g^2, e_g = 2 g s_g; dq and u are
// formed group by group (N = 64 / G columns of the accumulator, the B operand offset into the 128-byte rows).
template <int MODE, int G>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_bwd_kernel(const __grid_constant__ CUtensorMap tmX1, const __grid_constant__ CUtensorMap tmX2,
              const __grid_constant__ CUtensorMap tmY1, const __grid_constant__ CUtensorMap tmY2,
              const __grid_constant__ CUtensorMap tmY3, const BArgs args) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  auto bar = [&](int i) { return reinterpret_cast<uint64_t*>(base + OFF_BAR) + i; };
  auto y1 = [&](int s) { return base + OFF_ST + s * STAGE_BYTES; };
  auto y2 = [&](int s) { return base + OFF_ST + s * STAGE_BYTES + 8192; };
  auto y3 = [&](int s) { return base + OFF_ST + s * STAGE_BYTES + 16384; };
  auto sc = [&](int s) { return base + OFF_SC + s * 512; };
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  constexpr int NBUF = G == 1 ? 3 : G == 2 ? 2 : 1;
  constexpr uint32_t BW = (G + 1) * 64;            // columns of a score buffer
  constexpr uint32_t CB = G * 64;                  // its C block
  constexpr int MG = D / G;                        // features per group
  static_assert(NBUF * BW <= COL_ACC, "TMEM columns");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  const int n_stream = (args.Tlen + NT - 1) / NT;                 // streamed tiles of the whole sequence
  // MODE_DQ: heaviest (last) query tiles first, keys 0 .. m0 + 127;  MODE_DKV: key tile blockIdx.x (the first are
  // the heaviest), queries m0 .. T - 1
  const int mtile = MODE == MODE_DQ ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
  const int m0 = mtile * MT;
  const int jbeg = MODE == MODE_DQ ? 0 : 2 * mtile;
  const int jend = MODE == MODE_DQ ? min(n_stream, 2 * mtile + 2) : n_stream;
  const int ntiles = jend - jbeg;
  const int nsteps = MODE == MODE_DQ ? 2 * ntiles : ntiles;       // MODE_DQ streams the keys twice

  if (tid == 0) {
    abort_s = 0;
    mbar_init(bar(BAR_XFULL), 1);
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(bar(BAR_FULL + i), 1 + 32);
      mbar_init(bar(BAR_EMPTY + i), 2);
    }
    for (int i = 0; i < NBUF_MAX; ++i) {
      mbar_init(bar(BAR_SFULL + i), 1);
      mbar_init(bar(BAR_PFULL + i), 256);
      mbar_init(bar(BAR_PEMPTY + i), 1);
    }
    mbar_init(bar(BAR_ODONE), 1);
    mbar_init(bar(BAR_DRAIN), 2);
    fence_mbar_init();
    tma_prefetch_desc(&tmX1);
    tma_prefetch_desc(&tmX2);
    tma_prefetch_desc(&tmY1);
    tma_prefetch_desc(&tmY2);
    if (MODE == MODE_DQ) tma_prefetch_desc(&tmY3);
  }
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
    // =========================== TMA producer (+ the scalars of the streamed queries) ===========================
    if (lane == 0) {
      mbar_arrive_expect_tx(bar(BAR_XFULL), 32768);
      tma_load_3d(base + OFF_X1, &tmX1, bar(BAR_XFULL), 0, m0, bh);
      tma_load_3d(base + OFF_X2, &tmX2, bar(BAR_XFULL), 0, m0, bh);
    }
    for (int j = 0; j < nsteps && ok; ++j) {
      const int s = j % NSTAGE;
      const int n0 = (jbeg + j % ntiles) * NT;
      ok = wait_or_abort(bar(BAR_EMPTY + s), ((j / NSTAGE) & 1) ^ 1, abort_flag);
      if (!ok) break;
      if (lane == 0) {
        mbar_arrive_expect_tx(bar(BAR_FULL + s), MODE == MODE_DQ ? 24576u : 16384u);
        tma_load_3d(y1(s), &tmY1, bar(BAR_FULL + s), 0, n0, bh);
        tma_load_3d(y2(s), &tmY2, bar(BAR_FULL + s), 0, n0, bh);
        if (MODE == MODE_DQ) tma_load_3d(y3(s), &tmY3, bar(BAR_FULL + s), 0, n0, bh);
      }
      const int t = n0 + 2 * lane;                       // two streamed rows per lane
      if (MODE == MODE_DKV) {
        // (1 / D_t, dout_t . o_t) of the 64 streamed queries
        float4 st = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* src = args.stats + ((size_t)bh * args.Tlen + t) * 2;
        if (t < args.Tlen) { st.x = src[0]; st.y = src[1]; }
        if (t + 1 < args.Tlen) { st.z = src[2]; st.w = src[3]; }
        *reinterpret_cast<float4*>(sc(s) + lane * 16) = st;
      } else {
        // r_i of the 64 streamed keys
        float2 r2 = make_float2(0.f, 0.f);
        const float* src = args.rk + (size_t)bh * args.Tlen + t;
        if (t < args.Tlen) r2.x = src[0];
        if (t + 1 < args.Tlen) r2.y = src[1];
        *reinterpret_cast<float2*>(sc(s) + lane * 8) = r2;
      }
      mbar_arrive(bar(BAR_FULL + s));
    }
  } else if (warp == 1) {
    // =========================== score MMA issuer: [S | C] ===========================
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 64);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      const uint32_t x1 = smem_u32(base + OFF_X1), x2 = smem_u32(base + OFF_X2);
      ok = wait_or_abort(bar(BAR_XFULL), 0, abort_flag);
      for (int j = 0; j < nsteps && ok; ++j) {
        const int s = j % NSTAGE, b = j % NBUF;
        ok = wait_or_abort(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort(bar(BAR_PEMPTY + b), ((j / NBUF) & 1) ^ 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a1 = smem_u32(y1(s)), a2 = smem_u32(y2(s));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)      // 16 features per step; group ks / (4 / G) has its own 64 score columns
          mma_f16_ss(tb + COL_B + b * BW + (ks / (4 / G)) * 64, at(dk, x1 + ks * 32), at(dk, a1 + ks * 32), idesc,
                     (ks % (4 / G)) > 0);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_f16_ss(tb + COL_B + b * BW + CB, at(dk, x2 + ks * 32), at(dk, a2 + ks * 32), idesc, ks > 0);
        mma_commit(bar(BAR_SFULL + b));
        mma_commit(bar(BAR_EMPTY + s));
      }
    }
  } else if (warp == 2) {
    // =========================== output MMA issuer ===========================
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 64);     // A tmem, B MN-major
      // MN-major, 128B swizzle: 8 streamed rows x 64 columns per 1 KB atom (SBO); 16 rows per MMA
      const uint64_t dmn = smem_desc(0, 8192, 1024, kSwizzle128B);
      for (int j = 0; j < nsteps && ok; ++j) {
        const int s = j % NSTAGE, b = j % NBUF;
        ok = wait_or_abort(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort(bar(BAR_PFULL + b), (j / NBUF) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // group g: N = 64 / G accumulator columns, the B operand starts 2 * 64 / G bytes further into the rows
        const uint32_t idg = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, MG);
        if (MODE == MODE_DQ) {
          if (j >= ntiles) {      // the first sweep only sums the row scalars: nothing to multiply
            const uint32_t kp = smem_u32(y3(s));
#pragma unroll
            for (int g = 0; g < G; ++g)
#pragma unroll
              for (int ks = 0; ks < 4; ++ks)
                mma_f16_ts(tb + COL_ACC + g * MG, tb + COL_B + b * BW + g * 64 + ks * 8,
                           at(dmn, kp + ks * 2048 + g * MG * 2), idg, (j > ntiles || ks > 0) ? 1u : 0u);
          }
        } else {
          const uint32_t qa = smem_u32(y1(s)), ga = smem_u32(y2(s));
          // P^T sits over the first score block for G = 1 and over the C block otherwise; E_g^T over the other / its own
          const uint32_t pcol = G == 1 ? 0u : CB;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)      // dv~ += P^T dout
            mma_f16_ts(tb + COL_ACC, tb + COL_B + b * BW + pcol + ks * 8, at(dmn, ga + ks * 2048), idesc, (j > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
          for (int g = 0; g < G; ++g)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)    // u_g += E_g^T Q_g
              mma_f16_ts(tb + COL_ACC + 64 + g * MG, tb + COL_B + b * BW + (G == 1 ? 64u : (uint32_t)g * 64u) + ks * 8,
                         at(dmn, qa + ks * 2048 + g * MG * 2), idg, (j > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(bar(BAR_PEMPTY + b));
        mma_commit(bar(BAR_EMPTY + s));
      }
      if (ok) mma_commit(bar(BAR_ODONE));
    }
  } else if (warp >= WARP_BLD0) {
    // =========================== weights and epilogue (256 threads) ===========================
    const uint32_t q4 = warp & 3;
    const int ch = (warp - WARP_BLD0) >> 2;      // column half: streamed rows [32 ch, 32 ch + 32) of the tile
    const int rowl = q4 * 32 + lane;             // row of the fixed tile (= TMEM lane)
    const int grow = m0 + rowl;
    float inv_row = 0.f, del_row = 0.f;          // MODE_DQ: the scalars of this query (1 / D_t, dout_t . o_t)
    float sum_d = 0.f, sum_m = 0.f;              // MODE_DQ, first sweep: this warp's share of D_t and of sum a c
    float2* part = reinterpret_cast<float2*>(base + OFF_PART);
    for (int j = 0; j < nsteps && ok; ++j) {
      const int s = j % NSTAGE, b = j % NBUF;
      const int n0 = (jbeg + j % ntiles) * NT + ch * 32;   // first streamed row of this warp's columns
      if (MODE == MODE_DQ && j == ntiles) {
        // between the sweeps: the two column halves of a row meet, the scalars go to registers and to the workspace
        part[ch * MT + rowl] = make_float2(sum_d, sum_m);
        asm volatile("bar.sync %0, 64;" ::"r"(1 + (int)q4) : "memory");
        const float2 other = part[(1 - ch) * MT + rowl];
        const float dt = ch == 0 ? sum_d + other.x : other.x + sum_d;      // fixed order of the halves
        const float mt = ch == 0 ? sum_m + other.y : other.y + sum_m;
        inv_row = dt > 0.f ? 1.f / dt : 0.f;
        del_row = mt * inv_row;
        if (ch == 0 && grow < args.Tlen)
          *reinterpret_cast<float2*>(args.stats + ((size_t)bh * args.Tlen + grow) * 2) = make_float2(inv_row, del_row);
      }
      ok = wait_or_abort(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&     // the column scalars are in the stage
           wait_or_abort(bar(BAR_SFULL + b), (j / NBUF) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if constexpr (G > 1) {
        // one block of 64 score columns per group, then the C block; this warp's 32 columns of each
        const uint32_t bcol = tmem_addr(tb, q4 * 32, COL_B + b * BW + ch * 32);
        uint32_t cvg[32], sg[32], pk[16];
        tmem_ld32(bcol + CB, cvg);
        tmem_wait_ld(cvg);
        const bool first = MODE == MODE_DQ && j < ntiles;
        const bool diag = MODE == MODE_DQ ? (n0 + 31 > m0) : (n0 < m0 + MT - 1);
        auto dead = [&](int c) { return MODE == MODE_DQ ? (n0 + c > grow) : (n0 + c < grow); };
        float2 cf[16], ss[16];
        // two copies of each loop with a causal test, chosen once per tile: the test exists on diagonal tiles only
        auto factors = [&](auto masked) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float2 c2 = make_float2(__uint_as_float(cvg[c]), __uint_as_float(cvg[c + 1]));
            if (MODE == MODE_DQ) {
              // second sweep: 2 (c - dout.o) / D; first sweep: c as it is
              cf[c / 2] = first ? c2 : __fmul2_rn(__fadd2_rn(c2, make_float2(-del_row, -del_row)), make_float2(2.f * inv_row, 2.f * inv_row));
            } else {
              const float4 st = reinterpret_cast<const float4*>(sc(s) + ch * 256)[c / 2];
              cf[c / 2] = __fmul2_rn(__fadd2_rn(c2, make_float2(-st.y, -st.w)), make_float2(2.f * st.x, 2.f * st.z));
            }
            if constexpr (decltype(masked)::value) {
              if (dead(c)) cf[c / 2].x = 0.f;
              if (dead(c + 1)) cf[c / 2].y = 0.f;
            }
            ss[c / 2] = make_float2(0.f, 0.f);
          }
        };
        if (diag && !first) factors(std::true_type{}); else factors(std::false_type{});
#pragma unroll 1
        for (int g = 0; g < G; ++g) {
          tmem_ld32(bcol + g * 64, sg);
          tmem_wait_ld(sg);
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float2 s2 = make_float2(__uint_as_float(sg[c]), __uint_as_float(sg[c + 1]));
            ss[c / 2] = __ffma2_rn(s2, s2, ss[c / 2]);
            const float2 e2 = __fmul2_rn(cf[c / 2], s2);
            pk[c / 2] = pack_bf16(e2.x, e2.y);
          }
          if (first) continue;
          // E_g goes over columns [0,32) of its own block, which the column-half-0 warp reads
          tc_fence_before();
          asm volatile("bar.sync %0, 64;" ::"r"(1 + (int)q4) : "memory");
          tc_fence_after();
          tmem_st16(tmem_addr(tb, q4 * 32, COL_B + b * BW + g * 64 + ch * 16), pk);
        }
        if (first) {
          // a = r_i sum_g s_g^2 for the keys n <= this query; D_t += a, sum += a c
          const float2* cs = reinterpret_cast<const float2*>(sc(s) + ch * 128);
          float2 d2 = make_float2(0.f, 0.f), m2 = make_float2(0.f, 0.f);
          auto sums = [&](auto masked) {
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              float2 a2 = __fmul2_rn(ss[c / 2], cs[c / 2]);
              if constexpr (decltype(masked)::value) {
                if (dead(c)) a2.x = 0.f;
                if (dead(c + 1)) a2.y = 0.f;
              }
              d2 = __fadd2_rn(d2, a2);
              m2 = __ffma2_rn(a2, cf[c / 2], m2);
            }
          };
          if (diag) sums(std::true_type{}); else sums(std::false_type{});
          sum_d += d2.x + d2.y;
          sum_m += m2.x + m2.y;
        } else if (MODE == MODE_DKV) {
          // P^T = sum_g s_g^2 / D_t over the C block (both warps of the quadrant hold its scores since the first sync)
          auto weights = [&](auto masked) {
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
              const float4 st = reinterpret_cast<const float4*>(sc(s) + ch * 256)[c / 2];
              float2 p2 = __fmul2_rn(ss[c / 2], make_float2(st.x, st.z));
              if constexpr (decltype(masked)::value) {
                if (dead(c)) p2.x = 0.f;
                if (dead(c + 1)) p2.y = 0.f;
              }
              pk[c / 2] = pack_bf16(p2.x, p2.y);
            }
          };
          if (diag) weights(std::true_type{}); else weights(std::false_type{});
          tmem_st16(tmem_addr(tb, q4 * 32, COL_B + b * BW + CB + ch * 16), pk);
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(BAR_PFULL + b));
        continue;
      }
      const uint32_t scol = tmem_addr(tb, q4 * 32, COL_B + b * 128 + ch * 32);
      uint32_t sv[32], cv[32], pe[16], pp[16];
      tmem_ld32(scol, sv);
      tmem_ld32(scol + 64, cv);
      tmem_wait_ld(sv);
      tmem_wait_ld(cv);
      if (MODE == MODE_DQ && j < ntiles) {
        // first sweep: a = r_i s^2 for the keys n <= this query; D_t += a, sum += a c
        const float2* cs = reinterpret_cast<const float2*>(sc(s) + ch * 128);
        const bool diag = n0 + 31 > m0;                 // some key of these columns lies after some query of the tile
        float2 d2 = make_float2(0.f, 0.f), m2 = make_float2(0.f, 0.f);
        // two copies of the loop, chosen once per tile: the causal test exists on diagonal tiles only
        auto sums = [&](auto masked) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float2 s2 = make_float2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1]));
            float2 a2 = __fmul2_rn(__fmul2_rn(s2, s2), cs[c / 2]);
            if constexpr (decltype(masked)::value) {
              if (n0 + c > grow) a2.x = 0.f;
              if (n0 + c + 1 > grow) a2.y = 0.f;
            }
            d2 = __fadd2_rn(d2, a2);
            m2 = __ffma2_rn(a2, make_float2(__uint_as_float(cv[c]), __uint_as_float(cv[c + 1])), m2);
          }
        };
        if (diag) sums(std::true_type{}); else sums(std::false_type{});
        sum_d += d2.x + d2.y;
        sum_m += m2.x + m2.y;
        // nothing is stored; the buffer is handed on as it is
        tc_fence_before();
        mbar_arrive(bar(BAR_PFULL + b));
        continue;
      }
      if (MODE == MODE_DQ) {
        // e = 2 (c - dout.o) / D * s, keys n <= this query
        const float2 f2 = make_float2(2.f * inv_row, 2.f * inv_row), nd2 = make_float2(-del_row, -del_row);
        const bool diag = n0 + 31 > m0;
        auto weigh = [&](auto masked) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float2 s2 = make_float2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1]));
            const float2 c2 = make_float2(__uint_as_float(cv[c]), __uint_as_float(cv[c + 1]));
            float2 e2 = __fmul2_rn(__fmul2_rn(__fadd2_rn(c2, nd2), f2), s2);
            if constexpr (decltype(masked)::value) {
              if (n0 + c > grow) e2.x = 0.f;
              if (n0 + c + 1 > grow) e2.y = 0.f;
            }
            pe[c / 2] = pack_bf16(e2.x, e2.y);
          }
        };
        if (diag) weigh(std::true_type{}); else weigh(std::false_type{});
      } else {
        // p = s^2 / D_t, e = 2 (c - dout_t.o_t) / D_t * s with the scalars of the columns (queries t >= this key)
        const float4* cs = reinterpret_cast<const float4*>(sc(s) + ch * 256);
        const bool diag = n0 < m0 + MT - 1;             // some query of these columns lies before some key of the tile
        auto weigh = [&](auto masked) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const float4 st = cs[c / 2];                       // (1/D, dout.o) of queries n0 + c, n0 + c + 1
            const float2 s2 = make_float2(__uint_as_float(sv[c]), __uint_as_float(sv[c + 1]));
            const float2 c2 = make_float2(__uint_as_float(cv[c]), __uint_as_float(cv[c + 1]));
            const float2 t2 = __fmul2_rn(s2, make_float2(st.x, st.z));                    // s / D
            float2 p2 = __fmul2_rn(t2, s2);                                               // s^2 / D
            float2 e2 = __fmul2_rn(__fadd2_rn(c2, make_float2(-st.y, -st.w)), __fadd2_rn(t2, t2));
            if constexpr (decltype(masked)::value) {
              if (n0 + c < grow) { p2.x = 0.f; e2.x = 0.f; }
              if (n0 + c + 1 < grow) { p2.y = 0.f; e2.y = 0.f; }
            }
            pp[c / 2] = pack_bf16(p2.x, p2.y);
            pe[c / 2] = pack_bf16(e2.x, e2.y);
          }
        };
        if (diag) weigh(std::true_type{}); else weigh(std::false_type{});
      }
      // the weights overwrite score columns [0,32) of each half, which the column-half-0 warp of this quadrant
      // reads: both warps of the quadrant must have their scores in registers first
      tc_fence_before();
      asm volatile("bar.sync %0, 64;" ::"r"(1 + (int)q4) : "memory");
      tc_fence_after();
      if (MODE == MODE_DQ) {
        tmem_st16(tmem_addr(tb, q4 * 32, COL_B + b * 128 + ch * 16), pe);
      } else {
        tmem_st16(tmem_addr(tb, q4 * 32, COL_B + b * 128 + ch * 16), pp);
        tmem_st16(tmem_addr(tb, q4 * 32, COL_B + b * 128 + 64 + ch * 16), pe);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_PFULL + b));
    }
    // ---- epilogue ----
    if (ok) ok = wait_or_abort(bar(BAR_ODONE), 0, abort_flag);
    if (ok) {
      tc_fence_after();
      uint32_t a0[32];
      tmem_ld32(tmem_addr(tb, q4 * 32, COL_ACC + ch * 32), a0);
      tmem_wait_ld(a0);
      auto store32 = [&](__nv_bfloat16* dst, const float (&x)[32]) {
#pragma unroll
        for (int c = 0; c < 32; c += 8) {
          uint4 pkt;
          pkt.x = pack_bf16(x[c], x[c + 1]);
          pkt.y = pack_bf16(x[c + 2], x[c + 3]);
          pkt.z = pack_bf16(x[c + 4], x[c + 5]);
          pkt.w = pack_bf16(x[c + 6], x[c + 7]);
          *reinterpret_cast<uint4*>(dst + c) = pkt;
        }
      };
      float x[32];
      if (MODE == MODE_DQ) {
#pragma unroll
        for (int c = 0; c < 32; ++c) x[c] = __uint_as_float(a0[c]);
        if (grow < args.Tlen) store32(args.out0 + ((size_t)bh * args.Tlen + grow) * D + ch * 32, x);
      } else {
        uint32_t u[32];
        tmem_ld32(tmem_addr(tb, q4 * 32, COL_ACC + 64 + ch * 32), u);
        tmem_wait_ld(u);
        // this key's row (32 of its 64 entries), its share of ||k||^2 and of k . u; the halves meet in shared memory
        float kf[32];
        float n2 = 0.f, dot = 0.f;
#pragma unroll
        for (int cix = 0; cix < 4; ++cix) {
          const uint4 raw = *reinterpret_cast<const uint4*>(base + OFF_X1 + sw128_offset(rowl, ch * 4 + cix));
          const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            kf[8 * cix + 2 * e] = __uint_as_float(w[e] << 16);
            kf[8 * cix + 2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
          }
        }
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          n2 = fmaf(kf[c], kf[c], n2);
          dot = fmaf(kf[c], __uint_as_float(u[c]), dot);
        }
        part[ch * MT + rowl] = make_float2(n2, dot);
        asm volatile("bar.sync %0, 64;" ::"r"(1 + (int)q4) : "memory");
        const float2 other = part[(1 - ch) * MT + rowl];
        // fixed order of the two halves
        const float n2t = ch == 0 ? n2 + other.x : other.x + n2;
        const float dott = ch == 0 ? dot + other.y : other.y + dot;
        const float r = inv_or_zero(n2t);
        const float proj = r * dott;
        if (grow < args.Tlen) {
#pragma unroll
          for (int c = 0; c < 32; ++c) x[c] = r * (__uint_as_float(u[c]) - proj * kf[c]);
          store32(args.out0 + ((size_t)bh * args.Tlen + grow) * D + ch * 32, x);
#pragma unroll
          for (int c = 0; c < 32; ++c) x[c] = r * __uint_as_float(a0[c]);
          store32(args.out1 + ((size_t)bh * args.Tlen + grow) * D + ch * 32, x);
        }
      }
    }
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

size_t align256(size_t n) { return (n + 255) / 256 * 256; }

// Pre-pass: one warp per 4 key rows (8 lanes x 16 bytes per row).  k' = k / ||k||^2 (bf16), r = 1 / ||k||^2 (fp32).
__global__ void __launch_bounds__(256) bwd_prescale_kernel(const __nv_bfloat16* __restrict__ k, __nv_bfloat16* __restrict__ ks,
                                                           float* __restrict__ rk, size_t n_rows) {
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
  const float r = inv_or_zero(ss);
  uint4 kc;
  kc.x = pack_bf16(__uint_as_float(kw[0] << 16) * r, __uint_as_float(kw[0] & 0xFFFF0000u) * r);
  kc.y = pack_bf16(__uint_as_float(kw[1] << 16) * r, __uint_as_float(kw[1] & 0xFFFF0000u) * r);
  kc.z = pack_bf16(__uint_as_float(kw[2] << 16) * r, __uint_as_float(kw[2] & 0xFFFF0000u) * r);
  kc.w = pack_bf16(__uint_as_float(kw[3] << 16) * r, __uint_as_float(kw[3] & 0xFFFF0000u) * r);
  *reinterpret_cast<uint4*>(ks + row * D + part * 8) = kc;
  if (part == 0) rk[row] = r;
}

}  // namespace

// workspace: K' [BH][T][64] bf16, r [BH][T] fp32, the row scalars [BH][T][2] fp32
size_t tc_bwd_workspace_bytes(const Problem& p) {
  const size_t rows = (size_t)p.B * p.H * p.T;
  return align256(rows * D * 2) + align256(rows * sizeof(float)) + align256(rows * 2 * sizeof(float));
}

void tc_bwd_quadratic(const Problem& p, const void* dout, void* dq, void* dk, void* dv, void* workspace, int* device_status,
                      LaunchCtx& ctx) {
  const int BH = p.B * p.H;
  const size_t rows = (size_t)BH * p.T;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  __nv_bfloat16* ks = reinterpret_cast<__nv_bfloat16*>(ws);
  float* rk = reinterpret_cast<float*>(ws + align256(rows * D * 2));
  float* stats = reinterpret_cast<float*>(ws + align256(rows * D * 2) + align256(rows * sizeof(float)));
  bwd_prescale_kernel<<<(unsigned)((rows + 31) / 32), 256, 0, ctx.stream>>>(static_cast<const __nv_bfloat16*>(p.k), ks, rk, rows);
  note_launch(ctx);
  CUtensorMap q128, g128, k128, v128, q64, g64, k64, v64, ks64;
  if (!make_tile_map(&q128, p.q, BH, p.T, MT) || !make_tile_map(&g128, dout, BH, p.T, MT) || !make_tile_map(&k128, p.k, BH, p.T, MT) ||
      !make_tile_map(&v128, p.v, BH, p.T, MT) || !make_tile_map(&q64, p.q, BH, p.T, NT) || !make_tile_map(&g64, dout, BH, p.T, NT) ||
      !make_tile_map(&k64, p.k, BH, p.T, NT) || !make_tile_map(&v64, p.v, BH, p.T, NT) || !make_tile_map(&ks64, ks, BH, p.T, NT)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  auto kq = p.groups == 1 ? tc_bwd_kernel<MODE_DQ, 1> : p.groups == 2 ? tc_bwd_kernel<MODE_DQ, 2> : tc_bwd_kernel<MODE_DQ, 4>;
  auto kkv = p.groups == 1 ? tc_bwd_kernel<MODE_DKV, 1> : p.groups == 2 ? tc_bwd_kernel<MODE_DKV, 2> : tc_bwd_kernel<MODE_DKV, 4>;
  if (cudaFuncSetAttribute(kq, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess ||
      cudaFuncSetAttribute(kkv, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  const dim3 grid((p.T + MT - 1) / MT, BH);
  // dq and the row scalars, then dk and dv (which read the scalars)
  BArgs a{static_cast<__nv_bfloat16*>(dq), nullptr, stats, rk, device_status, p.T};
  kq<<<grid, NTHREADS, SMEM_ALLOC, ctx.stream>>>(q128, g128, k64, v64, ks64, a);
  note_launch(ctx);
  BArgs b{static_cast<__nv_bfloat16*>(dk), static_cast<__nv_bfloat16*>(dv), stats, rk, device_status, p.T};
  kkv<<<grid, NTHREADS, SMEM_ALLOC, ctx.stream>>>(k128, v128, q64, g64, q64, b);
  note_launch(ctx);
}

}  // namespace kata
