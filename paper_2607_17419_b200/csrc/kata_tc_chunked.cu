// Chunked (linear-state) KATA forward on the tensor cores, bf16, d_k = d_v = 64: which launches make up each form.
// The kernel is the token-major streaming kernel (kata_tc_stream.cu); the scan forms run it over groups of
// 128-token tiles as reduce -> scan -> restart:
//   pass 1  every group but the last computes the state it adds (state-only mode: keys and values only)
//   pass 2  inclusive scan over the group states (scan_round_kernel, fp32 adds)
//   pass 3  every group starts from the prefix before it and writes its outputs
#include "kata_common.cuh"

namespace kata {

size_t tc_chunked_state_elems() { return tc_stream_state_elems(); }
int tc_chunked_slices() { return tc_stream_slices(); }

void tc_chunked(const Problem& p, const ScanPlan& plan, bool use_scan, float* ws, int* device_status,
                const float* s_init, const float* z_init, float* s_final, float* z_final, int state_layout,
                LaunchCtx& ctx) {
  if (!use_scan || plan.n_groups <= 1) {   // whole sequence in one pass
    if (s_final != nullptr || s_init != nullptr) {
      StreamIO io{};
      io.s_init = s_init;
      io.z_init = z_init;
      io.s_final = s_final;
      io.z_final = z_final;
      io.layout = state_layout;
      io.write_out = 1;
      tc_chunked_stream_export(p, device_status, io, ctx);
    } else {
      tc_chunked_stream(p, device_status, ctx);
    }
    return;
  }
  const int BH = p.B * p.H;
  const int NG = plan.n_groups;
  const size_t E = tc_chunked_state_elems();
  float* bufA = ws;
  float* bufB = ws + (size_t)BH * NG * E;
  StreamIO io{};
  io.layout = state_layout;
  io.n_groups = NG;
  io.tiles_per_group = plan.chunks_per_group * kChunk / tc_stream_tile();
  // pass 1: the states the groups add (the last group's is never needed)
  io.final_compact = bufA;
  io.write_out = 0;
  io.launch_groups = NG - 1;
  tc_chunked_stream_state(p, device_status, io, ctx);
  // pass 2
  const float* incl = scan_group_states(bufA, bufB, BH, NG, NG - 1, E, ctx);
  // pass 3
  io.init_compact = incl;
  io.final_compact = nullptr;
  io.write_out = 1;
  io.launch_groups = NG;
  tc_chunked_stream_restart(p, device_status, io, ctx);
}

}  // namespace kata
