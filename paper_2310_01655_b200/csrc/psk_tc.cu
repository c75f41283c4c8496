// Tensor-core path (placeholder until the tcgen05 kernels land): reports "unsupported",
// so PSK_PATH_AUTO uses the CUDA-core kernels and PSK_PATH_TENSOR_CORES is refused.
#include "psk_internal.cuh"

namespace psk {
bool tc_supported(const Dims&) { return false; }
size_t tc_workspace_bytes(const Dims&, bool) { return 0; }
cudaError_t tc_fwd(const Dims&, const void*, const void*, const void*, const void*, const void*, void*, float*,
                   char*, cudaStream_t, int*) { return cudaErrorNotSupported; }
cudaError_t tc_bwd(const Dims&, const void*, const void*, const void*, const void*, const void*, const void*,
                   const float*, const void*, void*, void*, void*, char*, cudaStream_t, int*) {
    return cudaErrorNotSupported;
}
}  // namespace psk
