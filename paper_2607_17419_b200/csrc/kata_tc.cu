// Which problems the tensor-core (tcgen05/TMEM) kernels cover.
#include "kata_common.cuh"

namespace kata {

bool tc_supported(const Problem& p, int fn) {
  if (p.dtype != KATA_BF16 || p.d_k != 64 || p.d_v != 64) return false;
  const bool forward = fn == KATA_FN_QUADRATIC || fn == KATA_FN_CHUNKED || fn == KATA_FN_CHUNK_STATE_SCAN;
  // first-order feature: the chunked and scan forms (the quadratic form stays on the fp32 kernel)
  if (p.feature_order == 1) return forward && fn != KATA_FN_QUADRATIC;
  // rank-one lift, whole or blockwise (g = 2, 4: the same kernels with the state blocks of the feature groups only)
  return p.feature_order == 2 && forward && (p.groups == 1 || p.groups == 2 || p.groups == 4);
}

}  // namespace kata
