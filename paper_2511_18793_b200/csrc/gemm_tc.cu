// Tensor-core GEMM entry points (tcgen05 path).  Placeholder until the kernel lands: nothing is supported, so
// every GEMM takes the CUDA-core path.
#include "common.cuh"

namespace nz {
bool gemm_tc_supported(const GemmArgs&) { return false; }
void launch_gemm_tc(const GemmArgs&, cudaStream_t) {}
}  // namespace nz
