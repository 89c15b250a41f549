#include "tc_kernels.cuh"

namespace vgg {

bool tc_conv3x3_supported(ConvShape) { return false; }
cudaError_t tc_conv3x3(const bf16*, const bf16*, const float*, const bf16*, bf16*, ConvShape, bool,
                       int*, cudaStream_t) { return cudaErrorNotSupported; }
bool tc_wgrad_supported(ConvShape) { return false; }
size_t tc_wgrad_scratch_elems(ConvShape) { return 0; }
int tc_wgrad_launches(ConvShape) { return 0; }
cudaError_t tc_conv3x3_wgrad(const bf16*, const bf16*, float*, float*, float*, ConvShape, int*,
                             cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace vgg
