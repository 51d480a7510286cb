// C ABI of the KATA forward library: argument validation, scan planning, workspace carve-up and
// dispatch to the SIMT (fp32) or tensor-core (tcgen05) kernels.  Declarations and the contract of
// every entry point are in include/kata.h.
#include <cstdlib>
#include <cstring>
#include <mutex>

#include <cmath>

#include "kata_common.cuh"

namespace kata {
namespace {

thread_local int g_last_launches = 0;
thread_local int g_last_impl = KATA_IMPL_SIMT;

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool dim_ok(int d) { return d == 16 || d == 32 || d == 64; }
inline int ceil_log2(int n) {
  int r = 0;
  while ((1 << r) < n) ++r;
  return r;
}

struct Opts {
  int dtype, feature_order, state_layout, inter_chunk, impl, scan_group, groups;
  void* workspace;
  size_t workspace_bytes;
  float* s_pre;
  float* z_pre;
  const float* s_init;
  const float* z_init;
  int* device_status;
  cudaStream_t stream;
};

int read_opts(const kata_opts* o, Opts& out) {
  if (o == nullptr || o->struct_size != sizeof(kata_opts)) return KATA_ERR_INVALID_ARG;
  out.dtype = o->dtype;
  out.feature_order = o->feature_order == 0 ? 2 : o->feature_order;
  out.state_layout = o->state_layout;
  out.inter_chunk = o->inter_chunk;
  out.impl = o->impl;
  out.scan_group = o->scan_group;
  out.groups = o->feature_groups == 0 ? 1 : o->feature_groups;
  out.workspace = o->workspace;
  out.workspace_bytes = o->workspace_bytes;
  out.s_pre = o->s_pre;
  out.z_pre = o->z_pre;
  out.s_init = o->s_init;
  out.z_init = o->z_init;
  out.device_status = o->device_status;
  out.stream = static_cast<cudaStream_t>(o->stream);
  if (out.dtype != KATA_F32 && out.dtype != KATA_BF16) return KATA_ERR_INVALID_ARG;
  if (out.feature_order != 1 && out.feature_order != 2) return KATA_ERR_INVALID_ARG;
  if (out.state_layout != KATA_LAYOUT_DIRECT && out.state_layout != KATA_LAYOUT_PACKED) return KATA_ERR_INVALID_ARG;
  if (out.inter_chunk < KATA_SEQUENTIAL || out.inter_chunk > KATA_INTER_AUTO) return KATA_ERR_INVALID_ARG;
  if (out.impl < KATA_IMPL_AUTO || out.impl > KATA_IMPL_TENSOR) return KATA_ERR_INVALID_ARG;
  if (out.scan_group < 0) return KATA_ERR_INVALID_ARG;
  if (out.groups != 1 && out.groups != 2 && out.groups != 4) return KATA_ERR_INVALID_ARG;
  if (out.groups != 1 && out.feature_order != 2) return KATA_ERR_INVALID_ARG;
  if ((out.s_pre == nullptr) != (out.z_pre == nullptr)) return KATA_ERR_INVALID_ARG;
  return KATA_OK;
}

int check_shape(int fn, int B, int H, int T, int d_k, int d_v, int C) {
  if (fn < KATA_FN_QUADRATIC || fn > KATA_FN_CHUNK_STATE_SCAN) return KATA_ERR_INVALID_ARG;
  if (B < 1 || H < 1 || T < 1 || d_k < 1 || d_v < 1) return KATA_ERR_INVALID_ARG;
  if ((long long)B * H > 65535) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (!dim_ok(d_k) || !dim_ok(d_v)) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (fn != KATA_FN_QUADRATIC) {
    if (C < 1) return KATA_ERR_INVALID_ARG;
    if (C != kChunk && C != 2 * kChunk) return KATA_ERR_UNSUPPORTED_SHAPE;   // C = 128: see prepare()
  }
  return KATA_OK;
}

bool want_tensor(int fn, const Problem& p, const Opts& o) {
  return o.impl != KATA_IMPL_SIMT && tc_supported(p, fn);
}

// The tensor-core backward covers bf16: the full rank-one feature with d_k = d_v = 64 or narrower rows zero-padded,
// and the blockwise map (g = 2, 4) at d_k = d_v = 64.
bool bwd_tensor(const Problem& p, const Opts& o) {
  if (o.impl == KATA_IMPL_SIMT || p.dtype != KATA_BF16 || p.feature_order != 2) return false;
  // feature blocks depend on the true width: no padding there
  return p.groups == 1 || ((p.groups == 2 || p.groups == 4) && p.d_k == 64 && p.d_v == 64);
}

// Scratch of the backward: the fp32 kernels' row scalars, or the tensor-core kernels' scratch behind seven padded
// tensors (q, k, v, dout, dq, dk, dv) when the rows are narrower than 64.
size_t bwd_workspace(const Problem& p, const Opts& o, size_t* pad_bytes) {
  *pad_bytes = 0;
  if (!bwd_tensor(p, o)) return align_up(simt_bwd_workspace_elems(p.B * p.H, p.T) * sizeof(float));
  Problem pp = p;
  if (p.d_k < 64 || p.d_v < 64) {
    *pad_bytes = align_up((size_t)p.B * p.H * p.T * 64 * 2);
    pp.d_k = 64;
    pp.d_v = 64;
  }
  return 7 * *pad_bytes + align_up(tc_bwd_workspace_bytes(pp));
}

// Chunks per group of the scan forms on the SIMT kernels: enough groups for about two CTAs per SM, at least two.
int simt_scan_group(int BH, int slices, int NC) {
  int ng = (2 * 148 + slices * BH - 1) / (slices * BH);
  if (ng < 2) ng = 2;
  if (ng > NC) ng = NC;
  return (NC + ng - 1) / ng;
}

// Chunks per group of the scan forms on the tensor-core kernel.  One CTA per SM and per (head, value slice, group):
// the first pass runs groups 0 .. ng-2 in its state-only build, the last pass runs all ng groups, each in whole waves
// of 148 CTAs; a group state costs four transfers of 115 KB per CTA.  The smallest modelled time over ng = 2 .. 32
// decides.  The constants are fitted to measured times of the scan form on one batch element of 131072 tokens, 1024
// tiles (ms measured / modelled; heads x groups): 1 x 8: 0.89 / 0.92, 1 x 16: 0.50 / 0.48, 1 x 32: 0.54 / 0.49,
// 4 x 2: 3.40 / 3.69, 4 x 4: 1.82 / 1.85, 4 x 8: 1.79 / 1.87, 16 x 2: 5.64 / 5.95, 16 x 4: 6.21 / 6.68.
constexpr double kStateTileUs = 2.8, kFullTileUs = 4.4, kGroupStateUs = 0.115, kTwoLaunchesUs = 20.0;
double scan_pass_us(double ctas, double tiles_per_group, double tile_us) { return ceil(ctas / 148.0) * tiles_per_group * tile_us; }
int tensor_scan_group(int BH, int slices, int NC, double* model_us = nullptr) {
  const int cpt = tc_stream_tile() / kChunk;
  const int tiles = (NC + cpt - 1) / cpt;
  if (model_us) *model_us = 1e30;
  if (tiles < 2) return NC;
  const double c = (double)slices * BH;
  int best = 2;
  double best_us = 0.0;
  for (int ng = 2; ng <= 32 && ng <= tiles; ++ng) {
    const double tpg = (double)((tiles + ng - 1) / ng);
    const double us = scan_pass_us((ng - 1) * c, tpg, kStateTileUs) + scan_pass_us(ng * c, tpg, kFullTileUs) + ng * c * kGroupStateUs;
    if (ng == 2 || us < best_us) { best = ng; best_us = us; }
  }
  if (model_us) *model_us = best_us + kTwoLaunchesUs;
  const int G = (tiles + best - 1) / best * cpt;
  return G < NC ? G : NC;
}

// inter_chunk = AUTO on the tensor-core kernels: the scan form where its modelled time is below nine tenths of the
// sequential walk's.  The sequential walk is the feature-split kernel where it applies (nine CTAs per head in whole
// waves of 148, about 3.3 us a tile of 128 tokens with the GPU full and 2.6 us with a few heads), else the streaming
// kernel (one CTA per head and value slice, 4.4 us a tile).
bool tensor_scan_pays(int BH, int NC, int split_ctas) {   // split_ctas: CTAs per head of the feature-split kernel, 0 = not used
  const int cpt = tc_stream_tile() / kChunk;
  const int tiles = (NC + cpt - 1) / cpt;
  const int slices = tc_chunked_slices();
  double scan_us;
  tensor_scan_group(BH, slices, NC, &scan_us);
  const double seq_us = split_ctas > 0 ? ceil((double)split_ctas * BH / 148.0) * tiles * (split_ctas * BH >= 74 ? 3.3 : 2.6) + 10.0
                              : scan_pass_us((double)slices * BH, tiles, kFullTileUs);
  return scan_us < 0.9 * seq_us;
}

// How the chunk axis is cut into scan groups, and how many floats one group state takes.
int make_plan(int fn, const Problem& p, const Opts& o, bool tensor, int C, ScanPlan& plan, size_t& state_elems) {
  plan.n_chunks = (p.T + C - 1) / C;
  const int NC = plan.n_chunks;
  const int BH = p.B * p.H;
  if (tensor && p.feature_order == 1) {
    // first-order tensor-core kernel: groups of whole 128-token tiles, reduce-then-scan over the groups whatever
    // the entry point (any grouping of the chunk axis gives the same result up to fp32 re-association)
    state_elems = tc_order1_state_elems();
    const int cpt = tc_order1_tile() / C;                 // chunks per tile: 2 or 1
    int G;
    if (fn == KATA_FN_CHUNKED && o.inter_chunk == KATA_SEQUENTIAL) {
      G = NC;
    } else if (o.scan_group > 0) {
      G = (o.scan_group + cpt - 1) / cpt * cpt;
    } else {
      // One pass per head, or the groups of the single-launch scan (every group walked twice, the second time with
      // its keys and values in L2 only where the groups of all CTAs fit there: up to 1.5x the HBM traffic),
      // whichever the cost model says is faster.  Measured on B200: a CTA alone walks its tiles at about 1.25 us a
      // tile in one pass and 2.15 us a tile for the two passes of a group, a group costs about 12 us on top (two
      // pipeline ramps and the look-back), the kernel streams about 6 GB/ms.  Groups: one per CTA in one wave.
      const double n_tiles = (double)((p.T + tc_order1_tile() - 1) / tc_order1_tile());
      const double hbm_us = (double)BH * n_tiles * 65536.0 / 6.0e6;
      const double one_pass = fmax(hbm_us, ceil(BH / 148.0) * n_tiles * 1.25);
      G = NC;
      const int ng = 148 / BH;
      if (ng >= 2 && n_tiles >= 2 * ng) {
        const double tiles_per_group = ceil(n_tiles / ng);
        const double grouped = fmax(1.5 * hbm_us, tiles_per_group * 2.15) + 12.0;
        if (grouped < one_pass) G = (int)tiles_per_group * cpt;
      }
    }
    if (G > NC) G = NC;
    plan.chunks_per_group = G;
    plan.n_groups = (NC + G - 1) / G;
    // the chained scan over the group states: one hop per anchor (every eighth group) instead of doubling rounds
    plan.rounds = plan.n_groups > 1 ? (plan.n_groups - 2) / 8 + 1 : 0;
    return KATA_OK;
  }
  int slices;
  if (tensor) {
    state_elems = tc_chunked_state_elems();
    slices = tc_chunked_slices();
  } else if (p.feature_order == 1) {
    state_elems = order1_state_elems(p.d_k, p.d_v);
    slices = 1;
  } else {
    state_elems = simt_chunked_state_elems(p.d_k, p.d_v);
    slices = simt_chunked_slices(p.d_k, p.d_v);
  }
  int G;
  if (fn == KATA_FN_CHUNKED) {
    if (o.inter_chunk == KATA_SEQUENTIAL) {
      G = NC;
    } else if (o.scan_group > 0) {
      G = o.scan_group < NC ? o.scan_group : NC;
    } else {
      G = tensor ? tensor_scan_group(BH, slices, NC) : simt_scan_group(BH, slices, NC);
    }
  } else if (tensor && o.s_pre == nullptr && o.scan_group == 0) {
    // tensor-core pipeline without the per-chunk export: the grouping of the scan form of kata_fwd_chunked
    G = tensor_scan_group(BH, slices, NC);
  } else {
    if (o.s_pre != nullptr && o.scan_group > 1) return KATA_ERR_INVALID_ARG;
    if (o.s_pre != nullptr) {
      G = 1;
    } else if (o.scan_group > 0) {
      G = o.scan_group < NC ? o.scan_group : NC;
    } else {
      // the paper's per-chunk pipeline while the two state buffers stay below 2 GiB
      const double cap = 2.0 * 1024 * 1024 * 1024;
      G = 1;
      while (G < NC && 2.0 * BH * ((NC + G - 1) / G) * (double)state_elems * 4.0 > cap) G *= 2;
      if (G > NC) G = NC;
    }
  }
  // the tensor-core kernel works in tiles of 128 tokens: groups of whole tiles
  if (tensor && G < NC) {
    const int cpt = tc_stream_tile() / kChunk;
    G = (G + cpt - 1) / cpt * cpt;
    if (G > NC) G = NC;
  }
  plan.chunks_per_group = G;
  plan.n_groups = (NC + G - 1) / G;
  plan.rounds = plan.n_groups > 2 ? ceil_log2(plan.n_groups - 1) : 0;
  return KATA_OK;
}

size_t inner_workspace(int fn, const ScanPlan& plan, const Problem& p, size_t state_elems) {
  if (fn == KATA_FN_QUADRATIC) return 0;
  if (fn == KATA_FN_CHUNKED && plan.n_groups == 1) return 0;
  // the first-order kernels also keep one flag per group and a counter behind the two state buffers
  const size_t flags = p.feature_order == 1 ? align_up(((size_t)p.B * p.H * plan.n_groups + 1) * sizeof(int)) : 0;
  return 2 * align_up((size_t)p.B * p.H * plan.n_groups * state_elems * sizeof(float)) + flags;
}

size_t elem_bytes(int dtype) { return dtype == KATA_F32 ? 4 : 2; }

struct Staging {
  size_t q, k, v, out, inner, total;
};

Staging staging_layout(const Problem& p, size_t inner_bytes) {
  const size_t eb = elem_bytes(p.dtype);
  const size_t nqk = (size_t)p.B * p.H * p.T * p.d_k * eb;
  const size_t nv = (size_t)p.B * p.H * p.T * p.d_v * eb;
  Staging s;
  s.q = 0;
  s.k = s.q + align_up(nqk);
  s.v = s.k + align_up(nqk);
  s.out = s.v + align_up(nv);
  s.inner = s.out + align_up(nv);
  s.total = s.inner + inner_bytes;
  return s;
}

// Diagnostic override: KATA_CHUNKED_KERNEL=stream in the environment keeps the sequential chunked form on the
// value-sliced streaming kernel (for A/B timing); read once.
bool stream_kernel_forced() {
  static const bool forced = []() {
    const char* e = getenv("KATA_CHUNKED_KERNEL");
    return e != nullptr && strcmp(e, "stream") == 0;
  }();
  return forced;
}

int check_arch() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return KATA_ERR_CUDA;
  }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    cudaGetLastError();
    return KATA_ERR_CUDA;
  }
  return major == 10 ? KATA_OK : KATA_ERR_ARCH;
}

// Validation shared by every entry point; fills the problem, the plan and the workspace need.
struct Prepared {
  Problem p;
  Opts o;
  ScanPlan plan;
  size_t state_elems;
  size_t inner_bytes;
  bool tensor;
  int C;
  bool split;           // sequential chunked form on the feature-split kernel (needs scratch for the links of a head)
  bool pad;             // bf16 rows narrower than 64 are zero-padded to 64 so that the tensor-core kernels apply
  size_t pad_bytes;     // one padded tensor [B*H*T][64] bf16 (q, k, v, out: four of them at the start of the scratch)
};

// Zero-padding the rows of q, k, v to 64 entries changes neither the dot products nor the norms, and the padded
// value columns give output columns that are dropped: the same function, computed by the d = 64 kernels.
__global__ void pad_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t rows, int d) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // one 16-byte chunk of a padded row
  if (idx >= rows * 8) return;
  const size_t row = idx >> 3;
  const int c = (int)(idx & 7);
  uint4 x = make_uint4(0u, 0u, 0u, 0u);
  if (c * 8 < d) x = *reinterpret_cast<const uint4*>(src + row * d + c * 8);
  *reinterpret_cast<uint4*>(dst + row * 64 + c * 8) = x;
}

__global__ void unpad_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t rows, int d) {
  const int cpr = d / 8;                                                  // 16-byte chunks per output row
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * cpr) return;
  const size_t row = idx / cpr;
  const int c = (int)(idx % cpr);
  *reinterpret_cast<uint4*>(dst + row * d + c * 8) = *reinterpret_cast<const uint4*>(src + row * 64 + c * 8);
}

// The problem the kernels see: the caller's, or its copy with rows padded to 64 entries.
Problem kernel_problem(const Prepared& r) {
  Problem pp = r.p;
  if (r.pad) {
    pp.d_k = 64;
    pp.d_v = 64;
  }
  return pp;
}

int prepare(int fn, const void* q, const void* k, const void* v, void* out, int B, int H, int T, int d_k,
            int d_v, int C, const kata_opts* opts, bool need_ptrs, Prepared& r) {
  int st = read_opts(opts, r.o);
  if (st != KATA_OK) return st;
  st = check_shape(fn, B, H, T, d_k, d_v, C);
  if (st != KATA_OK) return st;
  if (need_ptrs && (q == nullptr || k == nullptr || v == nullptr || out == nullptr)) return KATA_ERR_INVALID_ARG;
  // inter_chunk = AUTO stays open only where both forms exist and no state is handed over; decided below
  if (r.o.inter_chunk == KATA_INTER_AUTO &&
      (fn != KATA_FN_CHUNKED || r.o.s_pre != nullptr || r.o.s_init != nullptr || r.o.feature_order != 2))
    r.o.inter_chunk = KATA_SEQUENTIAL;
  // s_pre/z_pre: prefix chunk states of the scan pipeline, or the final state of the sequential chunked forward
  if (r.o.s_pre != nullptr && !(fn == KATA_FN_CHUNK_STATE_SCAN ||
                                (fn == KATA_FN_CHUNKED && r.o.inter_chunk == KATA_SEQUENTIAL))) return KATA_ERR_INVALID_ARG;
  if (r.o.s_pre != nullptr && fn == KATA_FN_CHUNKED && r.o.feature_order != 2) return KATA_ERR_UNSUPPORTED_SHAPE;
  // s_init/z_init: the state before the first token, sequential chunked forward only
  if ((r.o.s_init == nullptr) != (r.o.z_init == nullptr)) return KATA_ERR_INVALID_ARG;
  if (r.o.s_init != nullptr && !(fn == KATA_FN_CHUNKED && r.o.inter_chunk == KATA_SEQUENTIAL)) return KATA_ERR_INVALID_ARG;
  if (r.o.s_init != nullptr && r.o.feature_order != 2) return KATA_ERR_UNSUPPORTED_SHAPE;
  r.p = Problem{q, k, v, out, B, H, T, d_k, d_v, r.o.dtype, r.o.feature_order, r.o.groups};
  // bf16 rows narrower than 64: zero-pad to 64 and use the tensor-core kernels (plain feature, no state hand-off:
  // the state layouts and the feature blocks depend on the true width)
  r.pad = r.o.impl != KATA_IMPL_SIMT && r.o.dtype == KATA_BF16 && (d_k < 64 || d_v < 64) && r.o.groups == 1 &&
          r.o.s_pre == nullptr && r.o.s_init == nullptr;
  r.pad_bytes = 0;
  if (r.pad) {
    r.pad = want_tensor(fn, kernel_problem(r), r.o);
    if (r.pad) r.pad_bytes = align_up((size_t)B * H * T * 64 * 2);
  }
  const Problem kp = kernel_problem(r);
  if (r.o.inter_chunk == KATA_INTER_AUTO) {
    Opts scan = r.o;
    scan.inter_chunk = KATA_SCAN;
    r.o.inter_chunk = KATA_SEQUENTIAL;
    if (C == kChunk && want_tensor(fn, kp, r.o) && want_tensor(fn, kp, scan) && tensor_scan_pays(B * H, (T + C - 1) / C, (r.o.s_init == nullptr && tc_split_supported(kp) && !stream_kernel_forced()) ? tc_split_ctas_per_head(kp) : 0))
      r.o.inter_chunk = KATA_SCAN;
  }
  r.tensor = want_tensor(fn, kp, r.o);
  if (r.o.impl == KATA_IMPL_TENSOR && !r.tensor) return KATA_ERR_UNSUPPORTED_SHAPE;
  r.C = fn == KATA_FN_QUADRATIC ? kChunk : C;
  r.plan = ScanPlan{(T + r.C - 1) / r.C, 0, 1, 0};
  r.state_elems = 0;
  r.split = false;
  r.inner_bytes = (fn == KATA_FN_QUADRATIC && r.tensor) ? tc_quadratic_workspace_bytes(kp) : 0;
  if (fn != KATA_FN_QUADRATIC) {
    if (r.tensor && r.o.s_pre != nullptr && fn == KATA_FN_CHUNK_STATE_SCAN) r.tensor = false;   // per-chunk export: SIMT pipeline
    // C = 128 (the chunk size of the paper's scan benchmark) exists on the first-order tensor-core path only
    if (r.C != kChunk && !(r.tensor && r.p.feature_order == 1)) return KATA_ERR_UNSUPPORTED_SHAPE;
    st = make_plan(fn, kp, r.o, r.tensor, r.C, r.plan, r.state_elems);
    if (st != KATA_OK) return st;
    r.inner_bytes = inner_workspace(fn, r.plan, kp, r.state_elems);
    // one pass over the whole sequence, no state handed in or out: the feature-split kernel
    r.split = fn == KATA_FN_CHUNKED && r.tensor && r.plan.n_groups == 1 && r.o.s_pre == nullptr && r.o.s_init == nullptr &&
              tc_split_supported(kp) && !stream_kernel_forced();
    if (r.split) r.inner_bytes = align_up(tc_split_workspace_bytes(kp));
    // state import and final-state export of the fp32 path go through one internal state per head
    if (fn == KATA_FN_CHUNKED && (r.o.s_pre != nullptr || r.o.s_init != nullptr) && !r.tensor)
      r.inner_bytes = align_up((size_t)B * H * r.state_elems * sizeof(float));
    // tensor-core path, state advanced in place: every value slice of a head reads the normaliser state and one of
    // them writes it, so the kernel reads a copy of z_init
    if (fn == KATA_FN_CHUNKED && r.tensor && r.o.z_init != nullptr && r.o.z_init == r.o.z_pre)
      r.inner_bytes = align_up((size_t)B * H * decode_n_psi(d_k, r.o.state_layout, 2, r.o.groups) * sizeof(float));
  }
  r.inner_bytes += 4 * r.pad_bytes;
  return KATA_OK;
}

int run_device(int fn, Prepared& r, void* ws) {
  LaunchCtx ctx{r.o.stream, 0, KATA_OK};
  Problem P = kernel_problem(r);
  if (r.pad) {
    // [q | k | v | out] padded to 64 columns at the start of the scratch, the kernels' own scratch after them
    unsigned char* w8 = static_cast<unsigned char*>(ws);
    __nv_bfloat16* pq = reinterpret_cast<__nv_bfloat16*>(w8);
    __nv_bfloat16* pk = reinterpret_cast<__nv_bfloat16*>(w8 + r.pad_bytes);
    __nv_bfloat16* pv = reinterpret_cast<__nv_bfloat16*>(w8 + 2 * r.pad_bytes);
    const size_t rows = (size_t)P.B * P.H * P.T;
    const unsigned blocks = (unsigned)((rows * 8 + 255) / 256);
    pad_rows_kernel<<<blocks, 256, 0, r.o.stream>>>(static_cast<const __nv_bfloat16*>(r.p.q), pq, rows, r.p.d_k);
    note_launch(ctx);
    pad_rows_kernel<<<blocks, 256, 0, r.o.stream>>>(static_cast<const __nv_bfloat16*>(r.p.k), pk, rows, r.p.d_k);
    note_launch(ctx);
    pad_rows_kernel<<<blocks, 256, 0, r.o.stream>>>(static_cast<const __nv_bfloat16*>(r.p.v), pv, rows, r.p.d_v);
    note_launch(ctx);
    P.q = pq;
    P.k = pk;
    P.v = pv;
    P.out = w8 + 3 * r.pad_bytes;
    ws = w8 + 4 * r.pad_bytes;
  }
  float* wsf = static_cast<float*>(ws);
  if (fn == KATA_FN_QUADRATIC) {
    if (r.tensor) tc_quadratic(P, ws, r.o.device_status, ctx);
    else simt_quadratic(P, ctx);
  } else {
    const bool use_scan = (fn == KATA_FN_CHUNK_STATE_SCAN) || r.plan.n_groups > 1;
    if (r.tensor && P.feature_order == 1) {
      tc_order1(P, r.plan, use_scan, r.C, wsf, r.o.device_status, ctx);
    } else if (r.split) {
      tc_chunked_split(P, ws, r.o.device_status, ctx);
    } else if (r.tensor) {
      const float* z_init = r.o.z_init;
      if (fn == KATA_FN_CHUNKED && z_init != nullptr && z_init == r.o.z_pre) {
        const size_t nb = (size_t)r.p.B * r.p.H * decode_n_psi(r.p.d_k, r.o.state_layout, 2, r.o.groups) * sizeof(float);
        if (cudaMemcpyAsync(wsf, z_init, nb, cudaMemcpyDeviceToDevice, r.o.stream) != cudaSuccess) {
          cudaGetLastError();
          return KATA_ERR_CUDA;
        }
        z_init = wsf;
      }
      tc_chunked(P, r.plan, use_scan, wsf, r.o.device_status, r.o.s_init, z_init, r.o.s_pre, r.o.z_pre,
                 r.o.state_layout, ctx);
    }
    else if (r.p.feature_order == 1) order1_chunked(P, r.plan, use_scan, wsf, r.o.s_pre, r.o.z_pre, ctx);
    else simt_chunked(P, r.plan, use_scan, wsf, r.o.s_init, r.o.z_init, r.o.s_pre, r.o.z_pre, r.o.state_layout, ctx);
  }
  if (r.pad && ctx.status == KATA_OK) {
    const size_t rows = (size_t)P.B * P.H * P.T;
    const unsigned blocks = (unsigned)((rows * (r.p.d_v / 8) + 255) / 256);
    unpad_rows_kernel<<<blocks, 256, 0, r.o.stream>>>(static_cast<const __nv_bfloat16*>(P.out),
                                                      static_cast<__nv_bfloat16*>(r.p.out), rows, r.p.d_v);
    note_launch(ctx);
  }
  if (ctx.status == KATA_OK) {
    g_last_launches = ctx.launches;
    g_last_impl = r.tensor ? KATA_IMPL_TENSOR : KATA_IMPL_SIMT;
  }
  return ctx.status;
}

// The kernels put the head index on a grid axis that ends at 65535.  Heads are independent and lie one after the other
// in [B,H,T,d] tensors, so the device entries of the forward take more heads than that in slabs of at most 65535, one
// after the other on the caller's stream and in the same scratch (no state pointers: their layouts are per call).
constexpr long long kMaxHeads = 65535;

int entry(int fn, const void* q, const void* k, const void* v, void* out, int B, int H, int T, int d_k,
          int d_v, int C, const kata_opts* opts) {
  if (B >= 1 && H >= 1 && (long long)B * H > kMaxHeads) {
    Opts o;
    int st = read_opts(opts, o);
    if (st != KATA_OK) return st;
    if (T < 1 || d_k < 1 || d_v < 1 || q == nullptr || k == nullptr || v == nullptr || out == nullptr) return KATA_ERR_INVALID_ARG;
    if (o.s_pre != nullptr || o.z_pre != nullptr || o.s_init != nullptr || o.z_init != nullptr) return KATA_ERR_UNSUPPORTED_SHAPE;
    const size_t eb = elem_bytes(o.dtype);
    const long long BH = (long long)B * H;
    int launches = 0;
    for (long long h0 = 0; h0 < BH; h0 += kMaxHeads) {
      const int n = (int)(BH - h0 < kMaxHeads ? BH - h0 : kMaxHeads);
      const size_t offk = (size_t)h0 * T * d_k * eb, offv = (size_t)h0 * T * d_v * eb;
      st = entry(fn, static_cast<const char*>(q) + offk, static_cast<const char*>(k) + offk, static_cast<const char*>(v) + offv,
                 static_cast<char*>(out) + offv, 1, n, T, d_k, d_v, C, opts);
      if (st != KATA_OK) return st;
      launches += g_last_launches;
    }
    g_last_launches = launches;
    return KATA_OK;
  }
  Prepared r;
  int st = prepare(fn, q, k, v, out, B, H, T, d_k, d_v, C, opts, true, r);
  if (st != KATA_OK) return st;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return KATA_ERR_ALIGNMENT;
  if (r.o.s_pre != nullptr && (!aligned16(r.o.s_pre) || !aligned16(r.o.z_pre))) return KATA_ERR_ALIGNMENT;
  if (r.o.s_init != nullptr && (!aligned16(r.o.s_init) || !aligned16(r.o.z_init))) return KATA_ERR_ALIGNMENT;
  if (r.inner_bytes > 0) {
    if (r.o.workspace == nullptr || r.o.workspace_bytes < r.inner_bytes) return KATA_ERR_WORKSPACE_TOO_SMALL;
    if ((reinterpret_cast<uintptr_t>(r.o.workspace) & (kAlign - 1)) != 0) return KATA_ERR_ALIGNMENT;
  }
  st = check_arch();
  if (st != KATA_OK) return st;
  return run_device(fn, r, r.o.workspace);
}

// ---- host buffers, long sequences: copies and kernels overlapped piece by piece ----
// The sequential chunked forward can be fed in pieces of the token axis (the state after a piece is the state before
// the next).  The host-buffer entry uses that on the tensor-core path: while piece i is computed, piece i + 1 is on
// its way to the device and the output of piece i - 1 on its way back, on two internal streams.  The pieces are
// tensors of their own on the device ([B,H,T_piece,d], two sets of buffers); the host tensors are read and written
// with pitched copies.
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, in_done[2] = {nullptr, nullptr}, comp_done[2] = {nullptr, nullptr},
              out_done[2] = {nullptr, nullptr};
};
std::mutex g_pipe_mutex;
HostPipe g_pipe[64];                        // one per device ordinal, created on first use, kept for the process

bool host_pipe_get(HostPipe*& hp) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  HostPipe& h = g_pipe[dev];
  if (!h.ready) {
    bool ok = cudaStreamCreateWithFlags(&h.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&h.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&h.start, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i)
      ok = cudaEventCreateWithFlags(&h.in_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&h.comp_done[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&h.out_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      return false;
    }
    h.ready = true;
  }
  hp = &h;
  return true;
}

struct PipePlan {
  int pieces, piece_T;
  size_t tensor_bytes;       // one piece of q, k, v or out on the device
  size_t s_bytes, z_bytes;   // the state handed from piece to piece (fp32, DIRECT layout)
  size_t inner_bytes;        // scratch of one piece's call
  size_t total;
};

// Pieces of at least 8192 tokens, at most sixteen of them, whole 128-token tiles; bf16 d_k = d_v = 64 tensor-core path of
// the sequential form with no state asked for or given by the caller.
bool host_pipe_plan(int fn, const Prepared& r, const kata_opts* opts, int C, PipePlan& pp) {
  const Problem& p = r.p;
  if (fn != KATA_FN_CHUNKED || !r.tensor || r.pad || r.o.inter_chunk != KATA_SEQUENTIAL || p.feature_order != 2) return false;
  if (r.o.s_pre != nullptr || r.o.s_init != nullptr || p.dtype != KATA_BF16 || p.d_k != 64 || p.d_v != 64) return false;
  if (p.T < 4 * 8192) return false;
  pp.pieces = p.T / 8192 < 16 ? p.T / 8192 : 16;
  pp.piece_T = ((p.T + pp.pieces - 1) / pp.pieces + 127) / 128 * 128;
  pp.pieces = (p.T + pp.piece_T - 1) / pp.piece_T;
  pp.tensor_bytes = align_up((size_t)p.B * p.H * pp.piece_T * 64 * 2);
  const size_t n_psi = (size_t)decode_n_psi(p.d_k, KATA_LAYOUT_DIRECT, 2, p.groups);
  pp.s_bytes = align_up((size_t)p.B * p.H * n_psi * p.d_v * sizeof(float));
  pp.z_bytes = align_up((size_t)p.B * p.H * n_psi * sizeof(float));
  kata_opts po = *opts;
  po.state_layout = KATA_LAYOUT_DIRECT;
  po.s_init = po.s_pre = reinterpret_cast<float*>(kAlign);       // any non-null, aligned value: sizes only
  po.z_init = po.z_pre = reinterpret_cast<float*>(kAlign);
  pp.inner_bytes = align_up(kata_workspace_bytes(KATA_FN_CHUNKED, p.B, p.H, pp.piece_T, p.d_k, p.d_v, C, &po));
  pp.total = 8 * pp.tensor_bytes + pp.s_bytes + pp.z_bytes + pp.inner_bytes;
  return pp.total <= r.o.workspace_bytes;
}

int host_pipelined(const Prepared& r, const PipePlan& pp, const void* q_host, const void* k_host, const void* v_host,
                   void* out_host, int C, const kata_opts* opts) {
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe* hp = nullptr;
  if (!host_pipe_get(hp)) return KATA_ERR_CUDA;
  const Problem& p = r.p;
  cudaStream_t main = r.o.stream;
  char* ws = static_cast<char*>(r.o.workspace);
  auto in_buf = [&](int b, int which) { return ws + (size_t)(b * 3 + which) * pp.tensor_bytes; };
  auto out_buf = [&](int b) { return ws + (size_t)(6 + b) * pp.tensor_bytes; };
  float* S = reinterpret_cast<float*>(ws + 8 * pp.tensor_bytes);
  float* Z = reinterpret_cast<float*>(ws + 8 * pp.tensor_bytes + pp.s_bytes);
  char* inner = ws + 8 * pp.tensor_bytes + pp.s_bytes + pp.z_bytes;
  const size_t row = 64 * 2, host_pitch = (size_t)p.T * row;
  const int heads = p.B * p.H;
  bool ok = cudaEventRecord(hp->start, main) == cudaSuccess &&
            cudaStreamWaitEvent(hp->in, hp->start, 0) == cudaSuccess &&
            cudaStreamWaitEvent(hp->out, hp->start, 0) == cudaSuccess;
  int launches = 0;
  int status = KATA_OK;
  // On every way out the caller's stream is made to wait for whatever is queued on the library's two streams: the
  // caller may reuse its buffers once its own stream is idle, whether the call succeeded or not.
  auto join = [&]() {
    bool j = cudaEventRecord(hp->in_done[0], hp->in) == cudaSuccess && cudaStreamWaitEvent(main, hp->in_done[0], 0) == cudaSuccess;
    j = (cudaEventRecord(hp->out_done[0], hp->out) == cudaSuccess && cudaStreamWaitEvent(main, hp->out_done[0], 0) == cudaSuccess) && j;
    if (!j) {           // last resort: the event calls themselves fail
      cudaGetLastError();
      cudaStreamSynchronize(hp->in);
      cudaStreamSynchronize(hp->out);
      cudaGetLastError();
    }
  };
  for (int i = 0; i < pp.pieces && ok; ++i) {
    const int b = i & 1;
    const int t0 = i * pp.piece_T;
    const int len = p.T - t0 < pp.piece_T ? p.T - t0 : pp.piece_T;
    const size_t width = (size_t)len * row;
    // inputs of piece i: their buffers were last read by the kernels of piece i - 2
    if (i >= 2) ok = cudaStreamWaitEvent(hp->in, hp->comp_done[b], 0) == cudaSuccess;
    const void* src[3] = {q_host, k_host, v_host};
    for (int w = 0; w < 3 && ok; ++w)
      ok = cudaMemcpy2DAsync(in_buf(b, w), width, static_cast<const char*>(src[w]) + (size_t)t0 * row, host_pitch, width,
                             heads, cudaMemcpyHostToDevice, hp->in) == cudaSuccess;
    ok = ok && cudaEventRecord(hp->in_done[b], hp->in) == cudaSuccess &&
         cudaStreamWaitEvent(main, hp->in_done[b], 0) == cudaSuccess;
    // the output buffer of piece i was last drained by the copy of piece i - 2
    if (ok && i >= 2) ok = cudaStreamWaitEvent(main, hp->out_done[b], 0) == cudaSuccess;
    if (!ok) break;
    kata_opts po = *opts;
    po.state_layout = KATA_LAYOUT_DIRECT;
    po.workspace = inner;
    po.workspace_bytes = pp.inner_bytes;
    po.s_init = i > 0 ? S : nullptr;
    po.z_init = i > 0 ? Z : nullptr;
    po.s_pre = i + 1 < pp.pieces ? S : nullptr;
    po.z_pre = i + 1 < pp.pieces ? Z : nullptr;
    const int st = entry(KATA_FN_CHUNKED, in_buf(b, 0), in_buf(b, 1), in_buf(b, 2), out_buf(b), p.B, p.H, len, p.d_k,
                         p.d_v, C, &po);
    if (st != KATA_OK) {
      status = st;
      break;
    }
    launches += g_last_launches;
    ok = cudaEventRecord(hp->comp_done[b], main) == cudaSuccess &&
         cudaStreamWaitEvent(hp->out, hp->comp_done[b], 0) == cudaSuccess &&
         cudaMemcpy2DAsync(static_cast<char*>(out_host) + (size_t)t0 * row, host_pitch, out_buf(b), width, width, heads,
                           cudaMemcpyDeviceToHost, hp->out) == cudaSuccess &&
         cudaEventRecord(hp->out_done[b], hp->out) == cudaSuccess;
  }
  // the caller's stream ends behind the last copies back (the last two pieces cover both event slots)
  ok = ok && status == KATA_OK && cudaStreamWaitEvent(main, hp->out_done[0], 0) == cudaSuccess &&
       cudaStreamWaitEvent(main, hp->out_done[1], 0) == cudaSuccess;
  g_last_launches = launches;
  if (!ok) {
    cudaGetLastError();
    join();
    return status != KATA_OK ? status : KATA_ERR_CUDA;
  }
  return KATA_OK;
}

}  // namespace
}  // namespace kata

using namespace kata;

extern "C" {

int kata_fwd_quadratic(const void* q, const void* k, const void* v, void* out, int B, int H, int T, int d_k,
                       int d_v, int C, const kata_opts* opts) {
  return entry(KATA_FN_QUADRATIC, q, k, v, out, B, H, T, d_k, d_v, C, opts);
}

int kata_fwd_chunked(const void* q, const void* k, const void* v, void* out, int B, int H, int T, int d_k,
                     int d_v, int C, const kata_opts* opts) {
  return entry(KATA_FN_CHUNKED, q, k, v, out, B, H, T, d_k, d_v, C, opts);
}

int kata_chunk_state_scan(const void* q, const void* k, const void* v, void* out, int B, int H, int T,
                          int d_k, int d_v, int C, const kata_opts* opts) {
  return entry(KATA_FN_CHUNK_STATE_SCAN, q, k, v, out, B, H, T, d_k, d_v, C, opts);
}

int kata_decode_step(const void* q, const void* k, const void* v, void* out, float* S, float* Z, int B, int H,
                     int d_k, int d_v, const kata_opts* opts) {
  Opts o;
  int st = read_opts(opts, o);
  if (st != KATA_OK) return st;
  if (B < 1 || H < 1 || d_k < 1 || d_v < 1) return KATA_ERR_INVALID_ARG;
  if ((long long)B * H > 65535) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (!dim_ok(d_k) || !dim_ok(d_v)) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (o.s_pre != nullptr || o.s_init != nullptr || o.z_init != nullptr) return KATA_ERR_INVALID_ARG;
  if (q == nullptr || k == nullptr || v == nullptr || out == nullptr || S == nullptr || Z == nullptr) return KATA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(S) || !aligned16(Z)) return KATA_ERR_ALIGNMENT;
  const int n_psi = decode_n_psi(d_k, o.state_layout, o.feature_order, o.groups);
  const size_t need = align_up(decode_workspace_elems(B * H, n_psi, d_v) * sizeof(float));
  if (o.workspace == nullptr || o.workspace_bytes < need) return KATA_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(o.workspace) & (kAlign - 1)) != 0) return KATA_ERR_ALIGNMENT;
  st = check_arch();
  if (st != KATA_OK) return st;
  LaunchCtx ctx{o.stream, 0, KATA_OK};
  decode_step(q, k, v, out, S, Z, static_cast<float*>(o.workspace), B * H, d_k, d_v, o.dtype, o.state_layout,
              o.feature_order, o.groups, ctx);
  if (ctx.status == KATA_OK) {
    g_last_launches = ctx.launches;
    g_last_impl = KATA_IMPL_SIMT;
  }
  return ctx.status;
}

int kata_bwd_quadratic(const void* q, const void* k, const void* v, const void* dout, void* dq, void* dk, void* dv,
                       int B, int H, int T, int d_k, int d_v, const kata_opts* opts) {
  Opts o;
  int st = read_opts(opts, o);
  if (st != KATA_OK) return st;
  if (B < 1 || H < 1 || T < 1 || d_k < 1 || d_v < 1) return KATA_ERR_INVALID_ARG;
  if ((long long)B * H > 65535) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (!dim_ok(d_k) || !dim_ok(d_v)) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (o.s_pre != nullptr || o.s_init != nullptr || o.z_init != nullptr) return KATA_ERR_INVALID_ARG;
  const Problem p{q, k, v, nullptr, B, H, T, d_k, d_v, o.dtype, o.feature_order, o.groups};
  const bool tensor = bwd_tensor(p, o);
  if (o.impl == KATA_IMPL_TENSOR && !tensor) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (q == nullptr || k == nullptr || v == nullptr || dout == nullptr || dq == nullptr || dk == nullptr || dv == nullptr)
    return KATA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dout) || !aligned16(dq) || !aligned16(dk) ||
      !aligned16(dv))
    return KATA_ERR_ALIGNMENT;
  size_t pad_bytes = 0;
  const size_t need = bwd_workspace(p, o, &pad_bytes);
  if (o.workspace == nullptr || o.workspace_bytes < need) return KATA_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(o.workspace) & (kAlign - 1)) != 0) return KATA_ERR_ALIGNMENT;
  st = check_arch();
  if (st != KATA_OK) return st;
  LaunchCtx ctx{o.stream, 0, KATA_OK};
  if (tensor && pad_bytes > 0) {
    // rows zero-padded to 64 entries: the padded columns of dq, dk, dv come out zero and are dropped
    unsigned char* w8 = static_cast<unsigned char*>(o.workspace);
    auto buf = [&](int i) { return reinterpret_cast<__nv_bfloat16*>(w8 + (size_t)i * pad_bytes); };
    const size_t rows = (size_t)B * H * T;
    const unsigned blocks = (unsigned)((rows * 8 + 255) / 256);
    const void* src[4] = {q, k, v, dout};
    const int width[4] = {d_k, d_k, d_v, d_v};
    for (int i = 0; i < 4; ++i) {
      pad_rows_kernel<<<blocks, 256, 0, o.stream>>>(static_cast<const __nv_bfloat16*>(src[i]), buf(i), rows, width[i]);
      note_launch(ctx);
    }
    Problem pp = p;
    pp.q = buf(0);
    pp.k = buf(1);
    pp.v = buf(2);
    pp.d_k = 64;
    pp.d_v = 64;
    tc_bwd_quadratic(pp, buf(3), buf(4), buf(5), buf(6), w8 + 7 * pad_bytes, o.device_status, ctx);
    void* dst[3] = {dq, dk, dv};
    const int wout[3] = {d_k, d_k, d_v};
    for (int i = 0; i < 3 && ctx.status == KATA_OK; ++i) {
      const unsigned ub = (unsigned)((rows * (wout[i] / 8) + 255) / 256);
      unpad_rows_kernel<<<ub, 256, 0, o.stream>>>(buf(4 + i), static_cast<__nv_bfloat16*>(dst[i]), rows, wout[i]);
      note_launch(ctx);
    }
  } else if (tensor) {
    tc_bwd_quadratic(p, dout, dq, dk, dv, o.workspace, o.device_status, ctx);
  } else {
    simt_bwd_quadratic(p, dout, dq, dk, dv, static_cast<float*>(o.workspace), ctx);
  }
  if (ctx.status == KATA_OK) {
    g_last_launches = ctx.launches;
    g_last_impl = tensor ? KATA_IMPL_TENSOR : KATA_IMPL_SIMT;
  }
  return ctx.status;
}

int kata_fwd_host(int fn, const void* q_host, const void* k_host, const void* v_host, void* out_host, int B,
                  int H, int T, int d_k, int d_v, int C, const kata_opts* opts) {
  Prepared r;
  int st = prepare(fn, q_host, k_host, v_host, out_host, B, H, T, d_k, d_v, C, opts, true, r);
  if (st != KATA_OK) return st;
  if (r.o.s_pre != nullptr && (!aligned16(r.o.s_pre) || !aligned16(r.o.z_pre))) return KATA_ERR_ALIGNMENT;
  if (r.o.s_init != nullptr && (!aligned16(r.o.s_init) || !aligned16(r.o.z_init))) return KATA_ERR_ALIGNMENT;
  const Staging s = staging_layout(r.p, r.inner_bytes);
  if (r.o.workspace == nullptr || r.o.workspace_bytes < s.total) return KATA_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(r.o.workspace) & (kAlign - 1)) != 0) return KATA_ERR_ALIGNMENT;
  st = check_arch();
  if (st != KATA_OK) return st;
  PipePlan pp;
  if (host_pipe_plan(fn, r, opts, C, pp)) return host_pipelined(r, pp, q_host, k_host, v_host, out_host, C, opts);
  char* ws = static_cast<char*>(r.o.workspace);
  const size_t eb = elem_bytes(r.p.dtype);
  const size_t nqk = (size_t)B * H * T * d_k * eb, nv = (size_t)B * H * T * d_v * eb;
  cudaStream_t stream = r.o.stream;
  bool ok = cudaMemcpyAsync(ws + s.q, q_host, nqk, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(ws + s.k, k_host, nqk, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(ws + s.v, v_host, nv, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return KATA_ERR_CUDA;
  }
  r.p.q = ws + s.q;
  r.p.k = ws + s.k;
  r.p.v = ws + s.v;
  r.p.out = ws + s.out;
  st = run_device(fn, r, ws + s.inner);
  if (st != KATA_OK) return st;
  if (cudaMemcpyAsync(out_host, ws + s.out, nv, cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
    cudaGetLastError();
    return KATA_ERR_CUDA;
  }
  return KATA_OK;
}

int kata_bwd_chunked(const void* q, const void* k, const void* v, const void* dout, void* dq, void* dk, void* dv,
                     int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts) {
  Opts o;
  int st = read_opts(opts, o);
  if (st != KATA_OK) return st;
  if (B < 1 || H < 1 || T < 1 || d_k < 1 || d_v < 1) return KATA_ERR_INVALID_ARG;
  if (o.s_pre != nullptr || o.s_init != nullptr || o.z_init != nullptr) return KATA_ERR_INVALID_ARG;
  const Problem p{q, k, v, nullptr, B, H, T, d_k, d_v, o.dtype, o.feature_order, o.groups};
  if (C != kChunk || !simt_bwd_chunked_supported(p) || o.impl == KATA_IMPL_TENSOR) return KATA_ERR_UNSUPPORTED_SHAPE;
  if ((long long)B * H * (d_v / 8) > 2147483647LL) return KATA_ERR_UNSUPPORTED_SHAPE;
  if (q == nullptr || k == nullptr || v == nullptr || dout == nullptr || dq == nullptr || dk == nullptr || dv == nullptr)
    return KATA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dout) || !aligned16(dq) || !aligned16(dk) ||
      !aligned16(dv))
    return KATA_ERR_ALIGNMENT;
  const size_t need = align_up(simt_bwd_chunked_workspace_elems(p) * sizeof(float));
  if (o.workspace == nullptr || o.workspace_bytes < need) return KATA_ERR_WORKSPACE_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(o.workspace) & (kAlign - 1)) != 0) return KATA_ERR_ALIGNMENT;
  st = check_arch();
  if (st != KATA_OK) return st;
  LaunchCtx ctx{o.stream, 0, KATA_OK};
  simt_bwd_chunked(p, dout, dq, dk, dv, static_cast<float*>(o.workspace), ctx);
  if (ctx.status == KATA_OK) {
    g_last_launches = ctx.launches;
    g_last_impl = KATA_IMPL_SIMT;
  }
  return ctx.status;
}

size_t kata_workspace_bytes(int fn, int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts) {
  const bool host_io = (fn & KATA_FN_HOST_IO) != 0;
  fn &= ~KATA_FN_HOST_IO;
  if (fn == KATA_FN_BWD_CHUNKED) {
    Opts o;
    if (host_io || read_opts(opts, o) != KATA_OK || B < 1 || H < 1 || T < 1 || C != kChunk) return 0;
    const Problem p{nullptr, nullptr, nullptr, nullptr, B, H, T, d_k, d_v, o.dtype, o.feature_order, o.groups};
    if (!simt_bwd_chunked_supported(p)) return 0;
    return align_up(simt_bwd_chunked_workspace_elems(p) * sizeof(float));
  }
  if (fn == KATA_FN_BWD_QUADRATIC) {    // C is ignored
    Opts o;
    if (host_io || read_opts(opts, o) != KATA_OK || B < 1 || H < 1 || T < 1 || !dim_ok(d_k) || !dim_ok(d_v)) return 0;
    const Problem p{nullptr, nullptr, nullptr, nullptr, B, H, T, d_k, d_v, o.dtype, o.feature_order, o.groups};
    size_t pad_bytes = 0;
    return bwd_workspace(p, o, &pad_bytes);
  }
  if (fn == KATA_FN_DECODE_STEP) {      // T and C are ignored
    Opts o;
    if (host_io || read_opts(opts, o) != KATA_OK || B < 1 || H < 1 || !dim_ok(d_k) || !dim_ok(d_v)) return 0;
    return align_up(decode_workspace_elems(B * H, decode_n_psi(d_k, o.state_layout, o.feature_order, o.groups), d_v) * sizeof(float));
  }
  if (!host_io && B >= 1 && H >= 1 && (long long)B * H > kMaxHeads) {
    // the device entries work in slabs of heads: the scratch of the largest slab and of the last one
    const long long BH = (long long)B * H, last = BH % kMaxHeads;
    const size_t a = kata_workspace_bytes(fn, 1, (int)kMaxHeads, T, d_k, d_v, C, opts);
    const size_t b = last > 0 ? kata_workspace_bytes(fn, 1, (int)last, T, d_k, d_v, C, opts) : 0;
    return a > b ? a : b;
  }
  Prepared r;
  if (prepare(fn, nullptr, nullptr, nullptr, nullptr, B, H, T, d_k, d_v, C, opts, false, r) != KATA_OK) return 0;
  if (!host_io) return r.inner_bytes;
  return staging_layout(r.p, r.inner_bytes).total;
}

int kata_scan_plan(int fn, int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts, int* n_groups,
                   int* chunks_per_group, int* scan_rounds) {
  if (B >= 1 && H >= 1 && (long long)B * H > kMaxHeads) { B = 1; H = (int)kMaxHeads; }   // the plan of a full slab of heads
  Prepared r;
  const int st = prepare(fn & ~KATA_FN_HOST_IO, nullptr, nullptr, nullptr, nullptr, B, H, T, d_k, d_v, C, opts,
                         false, r);
  if (st != KATA_OK) return st;
  if (n_groups) *n_groups = r.plan.n_groups;
  if (chunks_per_group) *chunks_per_group = r.plan.chunks_per_group;
  if (scan_rounds) *scan_rounds = r.plan.rounds;
  return KATA_OK;
}

int kata_host_plan(int fn, int B, int H, int T, int d_k, int d_v, int C, const kata_opts* opts, int* pieces,
                   int* piece_tokens) {
  Prepared r;
  fn &= ~KATA_FN_HOST_IO;
  const int st = prepare(fn, nullptr, nullptr, nullptr, nullptr, B, H, T, d_k, d_v, C, opts, false, r);
  if (st != KATA_OK) return st;
  // as if the caller had passed the workspace the host entry asks for
  r.o.workspace_bytes = staging_layout(r.p, r.inner_bytes).total;
  PipePlan pp;
  const bool piecewise = host_pipe_plan(fn, r, opts, C, pp);
  if (pieces) *pieces = piecewise ? pp.pieces : 1;
  if (piece_tokens) *piece_tokens = piecewise ? pp.piece_T : T;
  return KATA_OK;
}

int kata_last_launch_count(void) { return g_last_launches; }

int kata_last_impl(void) { return g_last_impl; }

const char* kata_status_string(int status) {
  switch (status) {
    case KATA_OK: return "ok";
    case KATA_ERR_INVALID_ARG: return "invalid argument";
    case KATA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case KATA_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
    case KATA_ERR_WORKSPACE_TOO_SMALL: return "workspace missing or too small";
    case KATA_ERR_ARCH: return "device is not compute capability 10.x (B200)";
    case KATA_ERR_CUDA: return "CUDA runtime error";
    case KATA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int kata_version(void) { return KATA_VERSION; }

}  // extern "C"
