// Placeholder translation unit for the tcgen05 forward kernels.
#include "common.cuh"
namespace wersa {
bool tc_supported(const wersa_config&) { return false; }
cudaError_t launch_tc_prepare_w(const Plan&, const Ws&, const void*, cudaStream_t, int*) { return cudaErrorNotSupported; }
cudaError_t launch_tc_kside(const Plan&, const Ws&, const void*, const void*, cudaStream_t, int*) { return cudaErrorNotSupported; }
cudaError_t launch_tc_qside(const Plan&, const Ws&, const void*, const float*, void*, cudaStream_t, int*) { return cudaErrorNotSupported; }
}  // namespace wersa
