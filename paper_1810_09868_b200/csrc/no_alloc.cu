// Filter and bias gradient of one 3x3 convolution for callers that must not
// allocate device memory: the split-K scratch the kernel needs lives in a
// fixed array inside this library instead of a caller-provided workspace.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/vgg19_b200.h"
#include "common.cuh"

namespace {

// Scratch shared by every call of vgg19_conv_wgrad_static() on a device.
// In host code this name is only a handle for the symbol; the address that
// kernels may dereference is looked up per device with cudaGetSymbolAddress.
static __device__ __align__(256) float g_static_scratch[VGG19_STATIC_SCRATCH_BYTES / sizeof(float)];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices];     // written once per device, under g_lookup_once
std::once_flag g_lookup_once[kMaxDevices];

}  // namespace

extern "C" int vgg19_conv_wgrad_static(const void* x, const void* dz, int32_t batch, int32_t height, int32_t width,
                                       int32_t cin, int32_t cout, int32_t dtype, float* dw, float* db,
                                       size_t* needed_bytes, void* stream) {
  if (needed_bytes) *needed_bytes = 0;
  if (!x || !dz || !dw || !db || batch < 1 || height < 1 || width < 1 || cin < 1 || cout < 1 ||
      (dtype != VGG19_FP32 && dtype != VGG19_BF16) || (long)batch * height * width >= (1L << 31))
    return VGG19_ERR_ARG;
  vgg::ConvShape s{batch, height, width, cin, cout};
  const size_t need = vgg::simt_wgrad_scratch_elems(s) * sizeof(float);
  if (needed_bytes) *needed_bytes = need;
  if (need > VGG19_STATIC_SCRATCH_BYTES) return VGG19_ERR_WORKSPACE;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VGG19_ERR_CUDA;
  // First call on this device: resolve the array's device address (the device is current).  One host
  // thread does the lookup, any others calling at the same moment wait for it.  With lazy module
  // loading (the CUDA default) this lookup is also what makes the driver place the array on the device.
  std::call_once(g_lookup_once[dev], [dev] {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch) == cudaSuccess) g_scratch_ptr[dev] = p;
  });
  if (!g_scratch_ptr[dev]) return VGG19_ERR_CUDA;
  // Nothing in the scratch has to start at zero: every partial sum the second
  // pass reads is written by the first pass of the same call.
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = dtype == VGG19_BF16
                      ? vgg::simt_conv3x3_wgrad<vgg::bf16>(static_cast<const vgg::bf16*>(x),
                                                           static_cast<const vgg::bf16*>(dz), dw, db,
                                                           g_scratch_ptr[dev], s, st)
                      : vgg::simt_conv3x3_wgrad<float>(static_cast<const float*>(x), static_cast<const float*>(dz),
                                                       dw, db, g_scratch_ptr[dev], s, st);
  return e == cudaSuccess ? VGG19_OK : VGG19_ERR_CUDA;
}
