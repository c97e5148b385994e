// Tensor-core GEMM (tcgen05 / TMEM / TMA). Placeholder until the kernel lands: reports itself
// unavailable so that the planner routes every GEMM to the SIMT kernel.
#include "fluid.h"
#include "kernels.h"

namespace fluid {

bool tc_kernel_available() { return false; }

int encode_tensor_map(TensorMapStorage*, const void*, const TmaOperand&) { return -1; }

cudaError_t launch_gemm_tc(const GemmParams&, const GemmTcHost&, uint32_t*, cudaStream_t) {
  return cudaErrorNotSupported;
}

int sm_count() { return 148; }

}  // namespace fluid
