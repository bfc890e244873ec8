// Tensor-core attention entry points.  Placeholder until the kernel lands.
#include "common.cuh"

namespace nz {
bool attention_tc_supported(const AttnArgs&) { return false; }
void launch_attention_tc(const AttnArgs&, cudaStream_t) {}
}  // namespace nz
