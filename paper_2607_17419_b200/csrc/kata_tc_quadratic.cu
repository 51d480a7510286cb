// Quadratic ("flash-style") KATA forward on the Blackwell tensor cores (tcgen05 + TMEM), bf16, d_k = d_v = 64.
//
// One CTA = one head x one tile of 128 queries; it walks the key tiles j <= i of 128 keys:
//   scores   S = Q K_j^T                      tcgen05 kind::f16, both operands from TMA-loaded 128B-swizzled tiles,
//                                             fp32 result in TMEM (two buffers)
//   weights  P = S^2 (causal mask on the      packed fp32x2 multiplies on the TMEM read-back; rounded to bf16 and
//            diagonal tile)                   stored back to TMEM
//   apply    [O | D] += P [V/||k||^2 | 1/||k||^2]   tcgen05 kind::f16, A = P from TMEM, B = the value tile (scaled in
//                                             place by the norm warps) plus one extra column group, MN-major, N = 80:
//                                             the normaliser is column 64 of the same accumulator
//   epilogue out = O / D (0 where D = 0)      the gate/normalise step of the readout
// There is no running maximum and no rescaling: the weights are polynomial.  The query norm cancels between
// numerator and denominator and is never applied.  The d^2-wide feature state is never formed.
//
// Warps (512 threads): 0 TMA producer, 1 score-MMA issuer, 2 apply-MMA issuer, 4-7 key norms + value scaling, 8-15 weight
// builders (TMEM lane quadrant = warp % 4, column half = (warp - 8) / 4).  All waits are bounded.
#include <cuda.h>

#include "kata_common.cuh"
#include "kata_umma.cuh"

namespace kata {
namespace {

using namespace umma;

constexpr int D = 64;
constexpr int QT = 128;          // queries per CTA
constexpr int KTILE = 128;       // keys per tile
constexpr int NSTAGE = 3;
constexpr int NTHREADS = 512;

constexpr uint32_t COL_S = 0;    // 2 x 128 fp32 score buffers
constexpr uint32_t COL_P = 256;  // 2 x 64: bf16 weights (128 keys packed in 64 columns)
constexpr uint32_t COL_O = 384;  // 80 fp32 accumulators: 64 outputs, column 64 = normaliser
constexpr uint32_t TMEM_COLS = 512;

constexpr uint32_t OFF_Q = 0;                       // 128 x 64 bf16, 128B swizzle
constexpr uint32_t STAGE_BYTES = 49152;             // K tile 16 KB, V tile 16 KB, scale-column tile 16 KB
constexpr uint32_t OFF_KV = 16384;                  // NSTAGE stages
constexpr uint32_t OFF_BAR = OFF_KV + NSTAGE * STAGE_BYTES;
constexpr uint32_t SMEM_BYTES = OFF_BAR + 256;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;
static_assert(SMEM_ALLOC > 116 * 1024, "one CTA per SM is assumed (the CTA allocates all of TMEM)");

// Every barrier has waiters that consume each of its phases in order (no waiter skips a phase).
enum {
  BAR_QFULL = 0,
  BAR_FULL = 1,      // [4] K and V tiles landed
  BAR_EMPTY = 5,     // [4] stage free: both issuers' commits + 128 norm threads
  BAR_R2FULL = 9,    // [4] values scaled by 1/||k||^2 and the scale column written (128 norm threads)
  BAR_SFULL = 13,    // [2] scores in TMEM
  BAR_SEMPTY = 15,   // [2] scores read (256 builders)
  BAR_PFULL = 17,    // [2] weights stored (256 builders)
  BAR_PEMPTY = 19,   // [2] weights consumed by the apply MMA
  BAR_ODONE = 21,
  BAR_DRAIN = 22,
  BAR_COUNT = 23
};

struct QArgs {
  __nv_bfloat16* out;
  int* device_status;
  int Tlen;
};

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
  const int qtile = gridDim.x - 1 - blockIdx.x;   // heaviest tiles first
  const int bh = blockIdx.y;
  const int q0 = qtile * QT;
  const int ntiles = qtile + 1;                   // key tiles 0..qtile

  if (tid == 0) {
    abort_s = 0;
    mbar_init(bar(BAR_QFULL), 1);
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(bar(BAR_FULL + i), 1);
      mbar_init(bar(BAR_EMPTY + i), 2 + 128);
      mbar_init(bar(BAR_R2FULL + i), 128);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BAR_SFULL + i), 1);
      mbar_init(bar(BAR_SEMPTY + i), 256);
      mbar_init(bar(BAR_PFULL + i), 256);
      mbar_init(bar(BAR_PEMPTY + i), 1);
    }
    mbar_init(bar(BAR_ODONE), 1);
    mbar_init(bar(BAR_DRAIN), 2);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  // the scale-column tiles are zero except for one bf16 per key row, rewritten for every key tile
  for (int i = tid; i < NSTAGE * 1024; i += NTHREADS)
    *reinterpret_cast<uint4*>(rtile(i >> 10) + (i & 1023) * 16) = make_uint4(0u, 0u, 0u, 0u);
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
    if (lane == 0) {
      mbar_arrive_expect_tx(bar(BAR_QFULL), 16384);
      tma_load_3d(base + OFF_Q, &tmQ, bar(BAR_QFULL), 0, q0, bh);
      for (int j = 0; j < ntiles && ok; ++j) {
        const int s = j % NSTAGE;
        ok = wait_or_abort(bar(BAR_EMPTY + s), ((j / NSTAGE) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(bar(BAR_FULL + s), 32768);
        tma_load_3d(ktile(s), &tmK, bar(BAR_FULL + s), 0, j * KTILE, bh);
        tma_load_3d(vtile(s), &tmV, bar(BAR_FULL + s), 0, j * KTILE, bh);
      }
    }
  } else if (warp == 1) {
    // =========================== score MMA issuer: S = Q K^T ===========================
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 0, 128, 128);
      const uint64_t dk = smem_desc(0, 16, 1024, kSwizzle128B);
      const uint32_t qa = smem_u32(base + OFF_Q);
      ok = wait_or_abort(bar(BAR_QFULL), 0, abort_flag);
      for (int j = 0; j < ntiles && ok; ++j) {
        const int s = j % NSTAGE, b = j & 1;
        ok = wait_or_abort(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort(bar(BAR_SEMPTY + b), ((j >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t ka = smem_u32(ktile(s));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          mma_f16_ss(tb + COL_S + b * 128, dk + (uint64_t)(((qa + ks * 32) >> 4) & 0x3FFF),
                     dk + (uint64_t)(((ka + ks * 32) >> 4) & 0x3FFF), idesc, ks > 0);
        mma_commit(bar(BAR_SFULL + b));
        mma_commit(bar(BAR_EMPTY + s));
      }
    }
  } else if (warp == 2) {
    // =========================== apply MMA issuer: O += P V ===========================
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kFmtBF16, kFmtBF16, 0, 1, 128, 80);     // A tmem, B MN-major, N = 64 + 16
      // MN-major, 128B swizzle: 8 key rows per 1024-byte atom (SBO), second group of 64 columns 16 KB on (LBO)
      const uint64_t dmn = smem_desc(0, 16384, 1024, kSwizzle128B);
      for (int j = 0; j < ntiles && ok; ++j) {
        const int s = j % NSTAGE, b = j & 1;
        ok = wait_or_abort(bar(BAR_R2FULL + s), (j / NSTAGE) & 1, abort_flag) &&
             wait_or_abort(bar(BAR_PFULL + b), (j >> 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t va = smem_u32(vtile(s));
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          mma_f16_ts(tb + COL_O, tb + COL_P + b * 64 + ks * 8, dmn + (uint64_t)(((va + ks * 2048) >> 4) & 0x3FFF),
                     idesc, (j > 0 || ks > 0) ? 1u : 0u);
        mma_commit(bar(BAR_PEMPTY + b));
        mma_commit(bar(BAR_EMPTY + s));
      }
      if (ok) mma_commit(bar(BAR_ODONE));
    }
  } else if (warp >= 4 && warp < 8) {
    // =========================== key norms (128 threads, one key each) ===========================
    const int kr = tid - 128;
    for (int j = 0; j < ntiles && ok; ++j) {
      const int s = j % NSTAGE;
      ok = wait_or_abort(bar(BAR_FULL + s), (j / NSTAGE) & 1, abort_flag);
      if (!ok) break;
      const unsigned char* kt = ktile(s);
      float ss0 = 0.f, ss1 = 0.f;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const uint4 raw = *reinterpret_cast<const uint4*>(kt + sw128_offset(kr, ch));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xFFFF0000u);
          ss0 = fmaf(lo, lo, ss0);
          ss1 = fmaf(hi, hi, ss1);
        }
      }
      const float r2 = inv_or_zero(ss0 + ss1);
      unsigned char* vt = vtile(s);
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        uint4* pv = reinterpret_cast<uint4*>(vt + sw128_offset(kr, ch));
        const uint4 raw = *pv;
        uint4 sc;
        sc.x = pack_bf16(__uint_as_float(raw.x << 16) * r2, __uint_as_float(raw.x & 0xFFFF0000u) * r2);
        sc.y = pack_bf16(__uint_as_float(raw.y << 16) * r2, __uint_as_float(raw.y & 0xFFFF0000u) * r2);
        sc.z = pack_bf16(__uint_as_float(raw.z << 16) * r2, __uint_as_float(raw.z & 0xFFFF0000u) * r2);
        sc.w = pack_bf16(__uint_as_float(raw.w << 16) * r2, __uint_as_float(raw.w & 0xFFFF0000u) * r2);
        *pv = sc;
      }
      // column 64 of the B operand: the scale itself (element 0 of 16-byte chunk 0 of this key row)
      *reinterpret_cast<uint16_t*>(rtile(s) + sw128_offset(kr, 0)) = (uint16_t)(pack_bf16(r2, 0.f) & 0xFFFFu);
      fence_async_smem();
      mbar_arrive(bar(BAR_R2FULL + s));
      mbar_arrive(bar(BAR_EMPTY + s));
    }
  } else if (warp >= 8) {
    // =========================== weight builders (256 threads) ===========================
    const uint32_t q4 = warp & 3;
    const int ch = (warp - 8) >> 2;              // column half: keys [64 ch, 64 ch + 64) of the tile
    const int rowl = q4 * 32 + lane;             // query row inside the tile (= TMEM lane)
    const int qrow = q0 + rowl;
    for (int j = 0; j < ntiles && ok; ++j) {
      const int b = j & 1;
      ok = wait_or_abort(bar(BAR_SFULL + b), (j >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t scol = tmem_addr(tb, q4 * 32, COL_S + b * 128 + ch * 64);
      const bool diag = (j == ntiles - 1);
      const int key0 = j * KTILE + ch * 64;
      uint32_t ya[32], yb[32], pk[32];
      auto weigh = [&](const uint32_t (&y)[32], int half) {
#pragma unroll
        for (int jj = 0; jj < 32; jj += 2) {
          const int c = half * 32 + jj;
          const float2 sv = make_float2(__uint_as_float(y[jj]), __uint_as_float(y[jj + 1]));
          float2 w = __fmul2_rn(sv, sv);
          if (diag) {
            if (key0 + c > qrow) w.x = 0.f;
            if (key0 + c + 1 > qrow) w.y = 0.f;
          }
          pk[c / 2] = pack_bf16(w.x, w.y);
        }
      };
      tmem_ld32(scol, ya);
      tmem_wait_ld(ya);
      tmem_ld32(scol + 32, yb);
      weigh(ya, 0);
      tmem_wait_ld(yb);
      tc_fence_before();
      mbar_arrive(bar(BAR_SEMPTY + b));          // this thread's scores are in registers
      weigh(yb, 1);
      ok = wait_or_abort(bar(BAR_PEMPTY + b), ((j >> 1) & 1) ^ 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      tmem_st32(tmem_addr(tb, q4 * 32, COL_P + b * 64 + ch * 32), pk);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_PFULL + b));
    }
    // ---- epilogue: out = O / D ----
    if (ok) ok = wait_or_abort(bar(BAR_ODONE), 0, abort_flag);
    if (ok) {
      tc_fence_after();
      uint32_t o[32], dn[16];
      tmem_ld32(tmem_addr(tb, q4 * 32, COL_O + ch * 32), o);
      tmem_ld16(tmem_addr(tb, q4 * 32, COL_O + 64), dn);
      tmem_wait_ld(o);
      tmem_wait_ld(dn);
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

// [BH][T][64] bf16 tensor, box = 64 columns x 128 rows x 1 head, 128B swizzle; rows beyond T read as zero.
bool make_map(CUtensorMap* tm, const void* ptr, int BH, int T) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
  cuuint32_t box[3] = {(cuuint32_t)D, (cuuint32_t)KTILE, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

void tc_quadratic(const Problem& p, int* device_status, LaunchCtx& ctx) {
  const int BH = p.B * p.H;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_map(&tmQ, p.q, BH, p.T) || !make_map(&tmK, p.k, BH, p.T) || !make_map(&tmV, p.v, BH, p.T)) {
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  if (cudaFuncSetAttribute(tc_quad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_ALLOC) !=
      cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
    return;
  }
  QArgs a{static_cast<__nv_bfloat16*>(p.out), device_status, p.T};
  tc_quad_kernel<<<dim3((p.T + QT - 1) / QT, BH), NTHREADS, SMEM_ALLOC, ctx.stream>>>(tmQ, tmK, tmV, a);
  note_launch(ctx);
}

}  // namespace kata
