// Tensor-core attention path for work items that carry several query rows.
#include "apar_internal.h"

namespace apar {

cudaError_t launch_attention_mma(const AttnArgs& a, int item_begin, int n_items, cudaStream_t st) {
  return launch_attention_vec(a, item_begin, n_items, false, st);
}

}  // namespace apar
