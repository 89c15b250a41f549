// Shared declarations of the VGG19 device library: status codes, small
// device helpers, and the host-side launch functions each .cu file exports
// to the pass scheduler in vgg19_api.cu.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace vgg {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// Device-side error word (one per network).  A kernel whose bounded wait ran
// out stores a nonzero code here and returns; the host reads it at
// vgg19_sync_status().
enum DeviceError : int {
  kDevOk = 0,
  kDevTimeoutTmaFull = 1,   // consumer waited too long for a TMA stage
  kDevTimeoutStageFree = 2, // producer waited too long for a free stage
  kDevTimeoutAccum = 3,     // epilogue waited too long for the accumulator
  kDevTimeoutTmemFree = 4,  // MMA issuer waited too long for a drained accumulator
  kDevTimeoutTest = 5,      // the self-test kernel's wait on a barrier nobody arrives on
  kDevBadLabel = 64,        // a label outside [0, classes): not a timeout, reported as a bad argument
  kDevSplitRange = 65,      // fp32 configuration on tensor cores: an activation beyond fp16's range
};

// ---- CUDA-core kernels (simt_kernels.cu) ---------------------------------
// T is the storage type of activations and weights (float or bf16); every
// sum is accumulated in fp32.

struct ConvShape {
  int N, H, W, Cin, Cout;
};

// out = [relu](conv3x3(in, wt) + bias) [* (mask > 0)], NHWC, wt [Cout][3][3][Cin].
template <typename T>
cudaError_t simt_conv3x3(const T* in, const T* wt, const float* bias, const T* mask, T* out,
                         ConvShape s, bool relu, cudaStream_t st);

// dW[k][r][s][c] = sum_p dz[p][k] x[p+(r-1,s-1)][c]; db[k] = sum_p dz[p][k].
// partial: fp32 scratch of simt_wgrad_scratch_elems() elements.
size_t simt_wgrad_scratch_elems(ConvShape s);
template <typename T>
cudaError_t simt_conv3x3_wgrad(const T* x, const T* dz, float* dW, float* db, float* partial,
                               ConvShape s, cudaStream_t st);

// db[c] = sum_p dz[p][c]; partial: fp32 scratch of at least 1024 * C elements.
template <typename T>
cudaError_t simt_bias_grad(const T* dz, float* db, float* partial, long P, int C, cudaStream_t st);
// db[o] = sum_m dY[m][o]
template <typename T>
cudaError_t simt_dense_db(const T* dY, float* db, int M, int Out, cudaStream_t st);

// y = max over 2x2 windows (stride 2) of x, NHWC.  code (or null), one byte per element of y: where the
// window's maximum sits, 0..3 in the order (0,0), (0,1), (1,0), (1,1), the first one on ties; 4 when the
// maximum is not positive (the ReLU that produced x passes no gradient to this window).
template <typename T>
cudaError_t simt_maxpool_fwd(const T* x, T* y, int N, int H, int W, int C, cudaStream_t st, uint8_t* code = nullptr);

// Pool scatter from the stored codes: dy[n][2i + a][2j + b][c] = dp[n][i][j][c] where code = 2a + b,
// 0 elsewhere (and everywhere for code 4): select-and-scatter fused with the ReLU mask below it,
// without reading the activation again.  H, W are the full-resolution sizes.
template <typename T>
cudaError_t simt_pool_scatter(const uint8_t* code, const T* dp, T* dy, int N, int H, int W, int C, cudaStream_t st);

// dy[pos] = dp[window] where pos is the window's first maximum of y and
// y[pos] > 0, else 0 (pool scatter fused with the ReLU mask of the layer that
// produced y).
template <typename T>
cudaError_t simt_maxpool_bwd_relu(const T* y, const T* dp, T* dy, int N, int H, int W, int C,
                                  cudaStream_t st);

// C[m][n] = epilogue(sum_k A[m][k] * B[n][k]); A [M][K] and B [N][K] row-major.
// Epilogue: + bias[n], ReLU, * (mask[m][n] > 0); written as T (out_t) and/or fp32 (out_f).
template <typename T>
cudaError_t simt_dense_nt(const T* A, const T* B, const float* bias, const T* mask, T* out_t,
                          float* out_f, int M, int N, int K, bool relu, cudaStream_t st);

// dX[m][i] = (sum_o dY[m][o] * W[o][i]) * (mask[m][i] > 0)      (W [Out][In] row-major)
template <typename T>
cudaError_t simt_dense_dx(const T* dY, const T* W, const T* mask, T* dX, int M, int In, int Out,
                          cudaStream_t st);

// dW[o][i] = sum_m dY[m][o] * X[m][i];  db[o] = sum_m dY[m][o]   (fp32 out)
template <typename T>
cudaError_t simt_dense_dw(const T* dY, const T* X, float* dW, float* db, int M, int In, int Out,
                          cudaStream_t st);

// Row-wise softmax of fp32 logits (probs may be null), and for the backward
// pass the per-row loss and dlogits = (p - onehot(label)) / rows, stored as T.
// A label outside [0, classes) is never dereferenced: the row's loss becomes NaN and kDevBadLabel is
// recorded in dev_error (when given).
template <typename T>
cudaError_t softmax_xent(const float* logits, const int32_t* labels, float* probs, T* dlogits,
                         float* row_loss, float* loss, int rows, int classes, cudaStream_t st,
                         int* dev_error = nullptr);

// fp32 -> T copy (weights), and the dgrad filter: wt_t[c][r][s][k] = w[k][2-r][2-s][c].
template <typename T>
cudaError_t convert_f32(const float* src, T* dst, size_t n, cudaStream_t st);
// Where the filters of layers 2..16 sit: in the flat fp32 parameter buffer (w_off) and in the three
// bf16 copy buffers (copy_off, the same in each); first[l] = number of 32 x 32 tiles (per tap, of the
// [Cout][Cin] matrix) before layer l, total = all tiles.  Cin and Cout are multiples of 32.
struct FilterCopyTable {
  int layers;
  long total;
  long first[16];
  long w_off[16];
  long copy_off[16];
  int Cin[16], Cout[16];
};
// Rebuilds, from the fp32 master, the rotated filters of the input gradients ([Cin][3][3][Cout], rotated
// by 180 degrees), the tap-major filters [9][Cout][Cin] and the rotated tap-major filters [9][Cin][Cout]
// of every layer in the table, all bf16, in one launch.
cudaError_t refresh_filter_copies(const float* params, bf16* dgrad_w, bf16* tap_fwd, bf16* tap_bwd,
                                  const FilterCopyTable& tab, cudaStream_t st);

// params -= lr * grads (fp32 master, in place); params_t (the storage-type copy, or null when T is
// float and the master is the copy) receives the rounded result in the same pass.  With lr_dev the
// rate is read from that device scalar instead of `lr` (a recorded graph keeps working when it changes).
template <typename T>
cudaError_t sgd_update(float* params, const float* grads, T* params_t, float lr, size_t n, cudaStream_t st,
                       const float* lr_dev = nullptr);
cudaError_t set_scalar(float* dst, float v, cudaStream_t st);
template <typename T>
cudaError_t make_dgrad_filter(const float* w, T* wt_t, int Cin, int Cout, cudaStream_t st);

// fp32 tensors as pairs of fp16 terms (split_kernels.cu): a row of C values as [hi | lo], hi = fp16(v),
// lo = fp16(v - hi), the same bytes as the fp32 row (the 16-bit words are passed as `half16`).  split_rows /
// merge_rows convert between the forms (dst may be src); C must divide 4096; a value beyond fp16's range sets
// kDevSplitRange in *dev_error.  maxpool_split pools [N][H][W][2C]; with rows_per_image the output is one row
// [all hi | all lo] per image, the form a dense layer reads.  split_weights turns rows of K weights, scaled
// by kSplitWeightScale, into rows [hi | lo | hi] of 3K.
typedef unsigned short half16;
// Weights are split after scaling by this power of two (exact), so that the lo terms of weights around 1e-2
// stay above fp16's smallest normal number; the kernels that multiply by them scale their sums back.
constexpr float kSplitWeightScale = 64.f;
bool split_rows_supported(int C);
cudaError_t split_rows(const float* src, half16* dst, long rows, int C, int* dev_error, cudaStream_t st);
cudaError_t merge_rows(const half16* src, float* dst, long rows, int C, cudaStream_t st);
cudaError_t maxpool_split(const half16* x, half16* y, int N, int H, int W, int C, bool rows_per_image, cudaStream_t st);
cudaError_t split_weights(const float* w, half16* out, long rows, int K, cudaStream_t st);

}  // namespace vgg
