// Tensor-core (tcgen05/TMEM) kernels: placeholder until the first version lands.
#include "kata_common.cuh"

namespace kata {
bool tc_supported(const Problem&) { return false; }
void tc_quadratic(const Problem&, int*, LaunchCtx& ctx) { ctx.status = KATA_ERR_UNSUPPORTED_SHAPE; }
size_t tc_chunked_state_elems() { return 0; }
int tc_chunked_slices() { return 1; }
void tc_chunked(const Problem&, const ScanPlan&, bool, float*, int*, LaunchCtx& ctx) {
  ctx.status = KATA_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace kata
