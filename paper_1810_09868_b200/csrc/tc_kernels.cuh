// Tensor-core (tcgen05 + TMEM + TMA) kernels of the VGG19 pass, bf16 operands
// with fp32 accumulation.  Each *_supported() predicate says whether the
// kernel takes a shape; the scheduler falls back to the CUDA-core kernels for
// the rest (3 input channels, images too small to fill a tile).
#pragma once

#include "common.cuh"

namespace vgg {

// out = [relu](conv3x3(in, wt) + bias) [* (mask > 0)] as an implicit GEMM:
// M = N*H*W output pixels, N = Cout, K = 9*Cin.  in/out NHWC bf16,
// wt [Cout][3][3][Cin] bf16, bias fp32 or null, mask NHWC bf16 (same shape as
// out) or null.  dev_error: device word that receives a DeviceError code if a
// bounded wait runs out.
bool tc_conv3x3_supported(ConvShape s);
cudaError_t tc_conv3x3(const bf16* in, const bf16* wt, const float* bias, const bf16* mask,
                       bf16* out, ConvShape s, bool relu, int* dev_error, cudaStream_t st);

// Filter and bias gradient of the same convolution (M = Cout, N = 9*Cin,
// K = pixels).
bool tc_wgrad_supported(ConvShape s);
size_t tc_wgrad_scratch_elems(ConvShape s);
int tc_wgrad_launches(ConvShape s);
cudaError_t tc_conv3x3_wgrad(const bf16* x, const bf16* dz, float* dW, float* db, float* partial,
                             ConvShape s, int* dev_error, cudaStream_t st);

}  // namespace vgg
