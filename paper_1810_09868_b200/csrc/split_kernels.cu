// fp32 tensors as pairs of fp16 terms, for the fp32 configuration's tensor-core path.
//
// A value v is carried as hi = fp16(v) and lo = fp16(v - hi): v - hi is exact in fp32, and hi + lo keeps
// 22 bits of v's mantissa (two bf16 terms would keep 16 at the same cost of three products).  The price is
// fp16's range: values beyond 65504 are reported (kDevSplitRange); where the lo term falls among fp16's subnormal
// numbers (|v| below about 0.25) the pair keeps an absolute 2^-25 rather than 22 bits - nothing beside activations of
// order one, but weights around 1e-2 would lose five bits, which is why they are scaled by a power of two before
// they are split.
// A row of C values (a pixel's channels, a dense layer's row) is stored as [hi_0 .. hi_{C-1} | lo_0 .. lo_{C-1}]:
// 4 C bytes, the size of the fp32 row, so a buffer planned for fp32 holds either form.  The kernels here move
// tensors between the two forms, pool the split form, and build the filter copies [w_hi | w_lo | w_hi] whose
// K blocks pair with [x_hi | x_hi | x_lo] in the convolution and GEMM kernels (three fp16 products per fp32
// product; x_lo * w_lo, 2^-22 of the product, is left out).
#include <cuda_fp16.h>

#include "common.cuh"

namespace vgg {
namespace {

constexpr int kBlock = 1024;       // threads; each takes four consecutive values
constexpr int kSpan = 4 * kBlock;  // values a block converts: whole rows when C divides it
constexpr float kHalfMax = 65504.f;

__device__ __forceinline__ void split4(float4 v, uint2* hi, uint2* lo) {
  __half2 h0 = __floats2half2_rn(v.x, v.y), h1 = __floats2half2_rn(v.z, v.w);
  __half2 l0 = __floats2half2_rn(v.x - __low2float(h0), v.y - __high2float(h0));
  __half2 l1 = __floats2half2_rn(v.z - __low2float(h1), v.w - __high2float(h1));
  *hi = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
  *lo = make_uint2(*reinterpret_cast<uint32_t*>(&l0), *reinterpret_cast<uint32_t*>(&l1));
}

__device__ __forceinline__ float4 merge4(uint2 hi, uint2 lo) {
  const __half2 h0 = *reinterpret_cast<__half2*>(&hi.x), h1 = *reinterpret_cast<__half2*>(&hi.y);
  const __half2 l0 = *reinterpret_cast<__half2*>(&lo.x), l1 = *reinterpret_cast<__half2*>(&lo.y);
  return make_float4(__low2float(h0) + __low2float(l0), __high2float(h0) + __high2float(l0),
                     __low2float(h1) + __low2float(l1), __high2float(h1) + __high2float(l1));
}

// rows of C fp32 -> rows of [hi | lo].  A block reads the 4096 values of its whole rows before it writes
// any, so dst may be src (the two forms of a row occupy the same bytes).
__global__ void __launch_bounds__(kBlock) split_rows_kernel(const float* src, half16* dst, long total, int C, int* dev_error) {
  const long e = (long)blockIdx.x * kSpan + 4L * threadIdx.x;
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (e < total) v = *reinterpret_cast<const float4*>(src + e);
  __syncthreads();
  if (e >= total) return;
  if (fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))) > kHalfMax && dev_error)
    atomicCAS(dev_error, 0, (int)kDevSplitRange);
  const long r = e / C;
  const int c = (int)(e - r * C);
  uint2 hi, lo;
  split4(v, &hi, &lo);
  *reinterpret_cast<uint2*>(dst + r * 2 * C + c) = hi;
  *reinterpret_cast<uint2*>(dst + r * 2 * C + C + c) = lo;
}

// the reverse, also in place
__global__ void __launch_bounds__(kBlock) merge_rows_kernel(const half16* src, float* dst, long total, int C) {
  const long e = (long)blockIdx.x * kSpan + 4L * threadIdx.x;
  uint2 hi = make_uint2(0, 0), lo = make_uint2(0, 0);
  if (e < total) {
    const long r = e / C;
    const int c = (int)(e - r * C);
    hi = *reinterpret_cast<const uint2*>(src + r * 2 * C + c);
    lo = *reinterpret_cast<const uint2*>(src + r * 2 * C + C + c);
  }
  __syncthreads();
  if (e < total) *reinterpret_cast<float4*>(dst + e) = merge4(hi, lo);
}

// 2x2 max pooling of a split tensor [N][H][W][2C]: the maximum of hi + lo (exact in fp32), split again.
// The output pixel (n, p) starts at n * img_stride + p * pix_stride, its lo terms lo_off further on: per pixel
// [hi | lo] like the input (pix_stride 2C, lo_off C), or per image [all hi | all lo] (pix_stride C,
// lo_off (H/2)(W/2)C), the row form a dense layer reads.
__global__ void maxpool_split_kernel(const half16* __restrict__ x, half16* __restrict__ y, int N, int H, int W, int C,
                                     long img_stride, int pix_stride, long lo_off) {
  const int Ho = H / 2, Wo = W / 2, C4 = C / 4;
  const long t = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (long)N * Ho * Wo * C4) return;
  const int c = (int)(t % C4) * 4;
  long q = t / C4;
  const int wo = (int)(q % Wo); q /= Wo;
  const int ho = (int)(q % Ho);
  const int n = (int)(q / Ho);
  float4 m = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const half16* px = x + (((long)n * H + 2 * ho + (i >> 1)) * W + 2 * wo + (i & 1)) * 2 * C + c;
    const float4 v = merge4(*reinterpret_cast<const uint2*>(px), *reinterpret_cast<const uint2*>(px + C));
    if (i == 0) m = v;
    else { m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w); }
  }
  uint2 hi, lo;
  split4(m, &hi, &lo);
  half16* out = y + (long)n * img_stride + ((long)ho * Wo + wo) * pix_stride + c;
  *reinterpret_cast<uint2*>(out) = hi;
  *reinterpret_cast<uint2*>(out + lo_off) = lo;
}

// rows of K fp32 weights -> rows of [hi | lo | hi] of the weights times kSplitWeightScale
__global__ void split_weights_kernel(const float* __restrict__ w, half16* __restrict__ out, long rows, int K) {
  const long e = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (e >= rows * K) return;
  const long r = e / K;
  const int k = (int)(e - r * K);
  float4 v = *reinterpret_cast<const float4*>(w + e);
  v.x *= kSplitWeightScale; v.y *= kSplitWeightScale; v.z *= kSplitWeightScale; v.w *= kSplitWeightScale;
  uint2 hi, lo;
  split4(v, &hi, &lo);
  half16* o = out + r * 3 * K + k;
  *reinterpret_cast<uint2*>(o) = hi;
  *reinterpret_cast<uint2*>(o + K) = lo;
  *reinterpret_cast<uint2*>(o + 2 * K) = hi;
}

}  // namespace

bool split_rows_supported(int C) { return C >= 4 && C <= kSpan && kSpan % C == 0; }

cudaError_t split_rows(const float* src, half16* dst, long rows, int C, int* dev_error, cudaStream_t st) {
  if (!split_rows_supported(C)) return cudaErrorInvalidValue;
  const long total = rows * C;
  split_rows_kernel<<<(unsigned)((total + kSpan - 1) / kSpan), kBlock, 0, st>>>(src, dst, total, C, dev_error);
  return cudaGetLastError();
}

cudaError_t merge_rows(const half16* src, float* dst, long rows, int C, cudaStream_t st) {
  if (!split_rows_supported(C)) return cudaErrorInvalidValue;
  const long total = rows * C;
  merge_rows_kernel<<<(unsigned)((total + kSpan - 1) / kSpan), kBlock, 0, st>>>(src, dst, total, C);
  return cudaGetLastError();
}

cudaError_t maxpool_split(const half16* x, half16* y, int N, int H, int W, int C, bool rows_per_image, cudaStream_t st) {
  if (C % 4 != 0 || H % 2 != 0 || W % 2 != 0) return cudaErrorInvalidValue;
  const long hw = (long)(H / 2) * (W / 2);
  const long total = (long)N * hw * (C / 4);
  maxpool_split_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(x, y, N, H, W, C, hw * 2 * C,
                                                                        rows_per_image ? C : 2 * C,
                                                                        rows_per_image ? hw * C : C);
  return cudaGetLastError();
}

cudaError_t split_weights(const float* w, half16* out, long rows, int K, cudaStream_t st) {
  if (K % 4 != 0) return cudaErrorInvalidValue;
  const long total = rows * K / 4;
  split_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w, out, rows, K);
  return cudaGetLastError();
}

}  // namespace vgg
