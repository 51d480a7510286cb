// kata_chunk_state_scan_static: the chunk-state / scan / chunk-output pipeline for callers that cannot
// allocate device memory.  The scan scratch (group states and the ping-pong buffer of the log-depth
// scan) lives in a file-scope device array of fixed size instead of a caller-provided workspace.
// See include/kata.h for the contract.
#include <mutex>

#include <cuda_runtime.h>

#include "../../include/kata.h"

namespace {

// The scratch itself.  Every GPU context that loads this library holds these bytes until it exits.
static __device__ __align__(256) unsigned char g_static_scratch[KATA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// The array's name is only a host-side handle; kernels need its device address, which differs per
// device.  Looked up once per device, with that device current.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return KATA_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return KATA_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return KATA_OK;
}

}  // namespace

extern "C" int kata_chunk_state_scan_static(const void* q, const void* k, const void* v, void* out, int B, int H,
                                            int T, int d_k, int d_v, int C, const kata_opts* opts) {
  if (opts == nullptr || opts->struct_size != sizeof(kata_opts)) return KATA_ERR_INVALID_ARG;
  if (opts->s_pre != nullptr || opts->z_pre != nullptr) return KATA_ERR_INVALID_ARG;   // no state export here
  kata_opts o = *opts;
  o.workspace = nullptr;
  o.workspace_bytes = 0;
  // Group size: the caller's, or the smallest power of two whose scratch fits the static array.
  size_t need = 0;
  if (o.scan_group > 0) {
    need = kata_workspace_bytes(KATA_FN_CHUNK_STATE_SCAN, B, H, T, d_k, d_v, C, &o);
  } else {
    const int n_chunks = (T > 0 && C > 0) ? (T + C - 1) / C : 1;
    for (int g = 1;; g *= 2) {
      o.scan_group = g;
      need = kata_workspace_bytes(KATA_FN_CHUNK_STATE_SCAN, B, H, T, d_k, d_v, C, &o);
      if (need <= (size_t)KATA_STATIC_SCRATCH_BYTES || g >= n_chunks) break;
    }
  }
  // Validation first, with the codes of kata_chunk_state_scan: arguments it rejects (and the few it accepts without
  // scratch) give need == 0 and go straight to it, before the array or the device is looked at.
  if (need == 0) return kata_chunk_state_scan(q, k, v, out, B, H, T, d_k, d_v, C, &o);
  if (need > (size_t)KATA_STATIC_SCRATCH_BYTES) return KATA_ERR_WORKSPACE_TOO_SMALL;
  {
    int dev = -1, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
      cudaGetLastError();
      return KATA_ERR_CUDA;
    }
    if (major != 10) return KATA_ERR_ARCH;
  }
  void* scratch = nullptr;
  const int st = scratch_for_current_device(&scratch);
  if (st != KATA_OK) return st;
  o.workspace = scratch;
  o.workspace_bytes = KATA_STATIC_SCRATCH_BYTES;
  return kata_chunk_state_scan(q, k, v, out, B, H, T, d_k, d_v, C, &o);
}
