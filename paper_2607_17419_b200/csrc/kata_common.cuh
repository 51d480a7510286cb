// Shared device/host helpers of the KATA kernels (element-type access, status plumbing).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/kata.h"

namespace kata {

constexpr int kChunk = 64;  // chunk size C of the chunked and scan forms

// ---- element access: global element -> fp32 and back (round-to-nearest-even) -------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// 1/||x||^2-style scale with the zero-row reading: a zero row has a zero feature.
__device__ __forceinline__ float inv_or_zero(float s) { return s > 0.f ? 1.f / s : 0.f; }
__device__ __forceinline__ float rsqrt_or_zero(float s) { return s > 0.f ? rsqrtf(s) : 0.f; }

// ---- launch bookkeeping (host) --------------------------------------------------------------
struct LaunchCtx {
  cudaStream_t stream;
  int launches;
  int status;
};

inline void note_launch(LaunchCtx& ctx) {
  ctx.launches++;
  if (ctx.status == KATA_OK && cudaPeekAtLastError() != cudaSuccess) {
    cudaGetLastError();
    ctx.status = KATA_ERR_CUDA;
  }
}

struct Problem {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  int B, H, T, d_k, d_v;
  int dtype;
  int feature_order;
  int groups;            // blocks of the blockwise PSD map (1 = full lift)
};

// Scan/group plan of the chunked forms.
struct ScanPlan {
  int n_chunks;          // N_C = ceil(T / C)
  int chunks_per_group;  // G
  int n_groups;          // ceil(N_C / G)
  int rounds;            // ceil(log2 n_groups)
};

// SIMT kernels (fp32 arithmetic; any supported shape and element type)
void simt_quadratic(const Problem& p, LaunchCtx& ctx);
size_t simt_chunked_state_elems(int d_k, int d_v);  // floats of internal state per (b,h,group)
int simt_chunked_slices(int d_k, int d_v);          // CTAs per (b,h,group)
// Inclusive Hillis-Steele scan over the first g_used of n_groups group states x[BH][n_groups][E]
// (E a multiple of 4), ping-ponging between bufA (input) and bufB; returns the buffer holding the result.
const float* scan_group_states(float* bufA, float* bufB, int BH, int n_groups, int g_used, size_t E,
                               LaunchCtx& ctx);
void simt_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, const float* s_init,
                  const float* z_init, float* s_pre, float* z_pre, int state_layout, LaunchCtx& ctx);

// Backward of the quadratic form (fp32 arithmetic; any supported shape and element type)
size_t simt_bwd_workspace_elems(int BH, int T);
void simt_bwd_quadratic(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* stats, LaunchCtx& ctx);
bool simt_bwd_chunked_supported(const Problem& p);
size_t simt_bwd_chunked_workspace_elems(const Problem& p);
void simt_bwd_chunked(const Problem& p, const void* dout, void* dq, void* dk, void* dv, float* ws, LaunchCtx& ctx);

// Backward of the quadratic form on the tensor cores (bf16, d_k = d_v = 64, full rank-one feature)
size_t tc_bwd_workspace_bytes(const Problem& p);
void tc_bwd_quadratic(const Problem& p, const void* dout, void* dq, void* dk, void* dv, void* workspace, int* device_status,
                      LaunchCtx& ctx);

// feature_order = 1: rows of q,k are the features (plain normalised linear attention, state d_k x d_v)
size_t order1_state_elems(int d_k, int d_v);
void order1_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, float* s_pre,
                    float* z_pre, LaunchCtx& ctx);

// Decode step (fp32 state in the exported layout; any supported shape and element type)
int decode_n_psi(int d_k, int layout, int order, int groups);
int decode_slabs(int n_psi);
size_t decode_workspace_elems(int BH, int n_psi, int d_v);
void decode_step(const void* q, const void* k, const void* v, void* out, float* S, float* Z, float* part, int BH,
                 int d_k, int d_v, int dtype, int layout, int order, int groups, LaunchCtx& ctx);

// Tensor-core kernels (tcgen05/TMEM; bf16, d_k = d_v = 64)
bool tc_supported(const Problem& p, int fn);
size_t tc_quadratic_workspace_bytes(const Problem& p);
void tc_quadratic(const Problem& p, void* workspace, int* device_status, LaunchCtx& ctx);
void tc_chunked_stream(const Problem& p, int* device_status, LaunchCtx& ctx);
// Sequential chunked form with the feature axis of the state split over the CTAs of a head (kata_tc_split.cu)
bool tc_split_supported(const Problem& p);
size_t tc_split_workspace_bytes(const Problem& p);
int tc_split_ctas_per_head(const Problem& p);
void tc_chunked_split(const Problem& p, void* workspace, int* device_status, LaunchCtx& ctx);
// State hand-off and groups of tiles for the second build of the streaming kernel (zero-initialise, then set).
struct StreamIO {
  const float* s_init;         // state before the first token in the public layout (null: zero)
  const float* z_init;
  float* s_final;              // state after the last token in the public layout (null: not exported)
  float* z_final;
  int layout;                  // KATA_LAYOUT_DIRECT / KATA_LAYOUT_PACKED
  const float* init_compact;   // [BH][n_groups][state]: group g starts from slot g - 1 (null: zero)
  float* final_compact;        // [BH][n_groups][state]: what a group leaves behind (null: not kept)
  int write_out;               // 0: state only
  int tiles_per_group;         // used when n_groups > 0
  int n_groups;                // 0: the whole sequence is one group
  int launch_groups;           // groups launched (0: n_groups)
};
void tc_chunked_stream_export(const Problem& p, int* device_status, const StreamIO& io, LaunchCtx& ctx);    // public state I/O
void tc_chunked_stream_restart(const Problem& p, int* device_status, const StreamIO& io, LaunchCtx& ctx);   // groups from init_compact
void tc_chunked_stream_state(const Problem& p, int* device_status, const StreamIO& io, LaunchCtx& ctx);     // groups to final_compact
size_t tc_stream_state_elems();
int tc_stream_slices();
int tc_stream_tile();
size_t tc_chunked_state_elems();
int tc_chunked_slices();
void tc_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, int* device_status,
                const float* s_init, const float* z_init, float* s_final, float* z_final, int state_layout,
                LaunchCtx& ctx);

// First-order feature on the tensor cores (bf16, d_k = d_v = 64): groups of whole 128-token tiles
size_t tc_order1_state_elems();
int tc_order1_tile();
void tc_order1(const Problem& p, const ScanPlan& plan, bool use_scan, int C, float* ws, int* device_status,
               LaunchCtx& ctx);

}  // namespace kata
