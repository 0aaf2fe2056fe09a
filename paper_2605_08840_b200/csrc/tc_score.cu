// Tensor-core score kernels (placeholder until the tcgen05 kernels land).
#include "restkv_common.cuh"
namespace restkv {
bool tc_supported(const Problem&) { return false; }
cudaError_t tc_init(void** state) { *state = nullptr; return cudaSuccess; }
cudaError_t launch_tc_pass1(void*, const Problem&, const Workspace&, const void*, const void*, const void*,
                            unsigned int*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_tc_pass2(void*, const Problem&, const Workspace&, const void*, const void*, const void*, float,
                            unsigned int*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace restkv
