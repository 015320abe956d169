// tcgen05 tensor-core kernel of the W4A4 linear (placeholder until the kernel lands).
#include "linear.cuh"

namespace sqap {
bool tcgen05_supports(const LinearArgs&) { return false; }
sqap_status launch_linear_tcgen05(const LinearArgs&, cudaStream_t) { return SQAP_ERR_UNSUPPORTED; }
}  // namespace sqap
