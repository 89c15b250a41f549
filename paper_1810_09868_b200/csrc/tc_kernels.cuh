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

// fp32 convolution as three fp16 products per product: in [N][H][W][2 Cin] and out [N][H][W][2 Cout] hold each
// pixel's channels as [hi | lo] fp16 terms, wt_split [Cout][9][3 Cin] each tap's filter row as [hi | lo | hi] of
// the weights times kSplitWeightScale; s names the logical channels (shapes as tc_conv3x3_supported).
cudaError_t tc_conv3x3_split(const half16* in, const half16* wt_split, const float* bias, half16* out, ConvShape s,
                             bool relu, int* dev_error, cudaStream_t st);

// The same convolution on CTA pairs (tc_conv_pair.cu): a cluster of two CTAs per 256-pixel x 256-channel
// tile, each staging half of the filter slice.  Cout must be a multiple of 256.
// partial (or null): fp32 scratch of tc_conv3x3_pair_scratch_elems() elements.  With it, when the tile count
// leaves a last round less than half full, the tiles of that round are cut along K over all the
// pairs and a second kernel adds the pieces (in a fixed order) and applies the epilogue.
// launches (or null) receives the number of kernels launched (1 or 2).
bool tc_conv3x3_pair_supported(ConvShape s);
size_t tc_conv3x3_pair_scratch_elems(ConvShape s);
cudaError_t tc_conv3x3_pair(const bf16* in, const bf16* wt, const float* bias, const bf16* mask,
                            bf16* out, ConvShape s, bool relu, int* dev_error, cudaStream_t st,
                            float* partial = nullptr, int* launches = nullptr, bf16* pooled = nullptr);

// The same convolution with the input patch (plus halo) kept in shared memory
// for all nine taps (tc_conv_halo.cu): the large-image, few-channel layers.
bool tc_conv3x3_halo_supported(ConvShape s);
bool tc_conv3x3_halo_supported_unpooled(ConvShape s);  // shapes it takes when no pooled output is asked for
// The filter comes tap-major, [9][Cout][Cin] (tc_make_tap_major builds it from the fp32 [Cout][3][3][Cin]
// master; for_dgrad gives the rotated, channel-swapped filter of the input gradient, [9][Cin][Cout]).
// `pooled` (or null) also receives the 2x2 max-pool of the result; `out` may then be null.
cudaError_t tc_make_tap_major(const float* w, bf16* out, int Cin, int Cout, bool for_dgrad, cudaStream_t st);
// pairs: work as CTA pairs (two tiles at a time, each CTA staging half of the filter's output channels)
// when the tile count is even.
// code (with pooled, or null): the arg-max code of every pooling window, as simt_maxpool_fwd writes it.
// scatter_code + scatter_out (input gradient of a layer that reads a pooled tensor; out, pooled and mask
// null): the result is not stored at its own resolution but scattered through the pool into
// scatter_out [N][2H][2W][Cout], each value to the window position its code names (none for code 4) and
// zeros to the other three: select-and-scatter and the ReLU mask below it, fused into this epilogue.
cudaError_t tc_conv3x3_halo(const bf16* in, const bf16* wt_tap_major, const float* bias, const bf16* mask, bf16* out,
                            bf16* pooled, ConvShape s, bool relu, int* dev_error, cudaStream_t st, bool pairs = true,
                            uint8_t* code = nullptr, const uint8_t* scatter_code = nullptr, bf16* scatter_out = nullptr);

// The same convolution for 64 output channels (tc_conv_rowshift.cu): the three taps of a filter row
// share one 128 x 192 x 16 MMA, and the epilogue adds the three column-shifted partial sums.  Same
// arguments as tc_conv3x3_halo; W must be a multiple of 14 and H of 8.
bool tc_conv3x3_rowshift_supported(ConvShape s);
cudaError_t tc_conv3x3_rowshift(const bf16* in, const bf16* wt_tap_major, const float* bias, const bf16* mask, bf16* out,
                                bf16* pooled, ConvShape s, bool relu, int* dev_error, cudaStream_t st,
                                uint8_t* code = nullptr, const uint8_t* scatter_code = nullptr, bf16* scatter_out = nullptr);

// Filter gradient of the same convolution as a GEMM with M = Cout, N = 9*Cin,
// K = pixels (both operands read transposed, x through the im2col window):
// dW fp32 [Cout][3][3][Cin]; db fp32 [Cout] = column sums of dz from the same GEMM (a block of
// ones as a second B operand), or null.  partial: fp32 scratch of tc_wgrad_scratch_elems().
// pairs: let CTA pairs (256 output channels per tile, each CTA staging half of the x tile) take the
// shapes that allow it; the scratch size and launch count are asked for with the same value.
bool tc_wgrad_supported(ConvShape s);
size_t tc_wgrad_scratch_elems(ConvShape s, bool pairs = true);
int tc_wgrad_launches(ConvShape s, bool with_db, bool pairs = true);
cudaError_t tc_conv3x3_wgrad(const bf16* x, const bf16* dz, float* dW, float* db, float* partial, ConvShape s,
                             int* dev_error, cudaStream_t st, bool pairs = true);

// The same filter gradient for layers with few channels (at most four 64 x 64 channel blocks), from
// tiled patches of x and dz instead of im2col boxes (tc_wgrad_patch.cu); always two launches.
bool tc_wgrad_patch_supported(ConvShape s);
size_t tc_wgrad_patch_scratch_elems(ConvShape s);
cudaError_t tc_conv3x3_wgrad_patch(const bf16* x, const bf16* dz, float* dW, float* db, float* partial, ConvShape s,
                                   int* dev_error, cudaStream_t st);

// Dense layers on the same GEMM kernel.  X [M][In], W [Out][In], dY [M][Out].
bool tc_dense_supported(int M, int In, int Out);
size_t tc_dense_scratch_elems(int M, int In, int Out);
cudaError_t tc_dense_forward(const bf16* X, const bf16* W, const float* bias, bf16* out_h, float* out_f,
                             float* partial, int M, int In, int Out, bool relu, int* dev_error, cudaStream_t st);
cudaError_t tc_dense_dx(const bf16* dY, const bf16* W, const bf16* mask, bf16* dX, float* partial, int M, int In,
                        int Out, int* dev_error, cudaStream_t st);
// fp32 dense layer from split operands: X [M][2 In] = [hi | lo] rows of fp16 terms, Ws [Out][3 In] = [hi | lo | hi]
// rows of the weights times kSplitWeightScale (In a multiple of 64); fp32 output.
// partial: tc_dense_split_scratch_elems(M, In, Out) elements (K is cut into many short splits).
size_t tc_dense_split_scratch_elems(int M, int In, int Out);
cudaError_t tc_dense_forward_split(const half16* X, const half16* Ws, const float* bias, float* out_f, float* partial,
                                   int M, int In, int Out, bool relu, int* dev_error, cudaStream_t st);
// With sgd_copy and sgd_lr (a device scalar) the gradient is not stored: dW then points at the layer's fp32
// master weights, which become w - lr * gradient in the GEMM's epilogue, and sgd_copy (their bf16 copy)
// receives the rounded result - the parameter update of a training step folded into the filter-gradient GEMM.
cudaError_t tc_dense_dw(const bf16* dY, const bf16* X, float* dW, int M, int In, int Out, int* dev_error,
                        cudaStream_t st, bf16* sgd_copy = nullptr, const float* sgd_lr = nullptr);

// First layer (3 input channels, 64 output channels) on tensor cores, through an
// 8-channel zero-padded copy x8 [N][H][W][8] of the image and a padded filter
// w8 [64][10 taps][8] (tc_conv_first.cu).  dW fp32 [64][3][3][3].
bool tc_first_conv_supported(ConvShape s);
cudaError_t tc_pad_to8(const bf16* x, bf16* x8, long pixels, cudaStream_t st);
cudaError_t tc_make_first_filter(const float* w, bf16* w8, cudaStream_t st);
cudaError_t tc_first_conv(const bf16* x8, const bf16* w8, const float* bias, bf16* out, ConvShape s, bool relu,
                          int* dev_error, cudaStream_t st);
size_t tc_first_wgrad_scratch_elems(ConvShape s);
// x8 must come from tc_pad_to8 (its constant channel yields db, fp32 [64], when db is not null).
cudaError_t tc_first_wgrad(const bf16* x8, const bf16* dz, float* dW, float* db, float* partial, ConvShape s, int* dev_error,
                           cudaStream_t st);

// conv1_1 and conv1_2 (3 -> 64 -> 64 channels, bias and ReLU each) as one kernel that never writes conv1_1's
// output (tc_conv_fused12.cu).  x8 from tc_pad_to8, w8 from tc_make_first_filter, wt2_tap_major the second
// layer's tap-major filter; out (or null) the second layer's output, pooled (or null) its 2x2 max-pool.
// s describes the first layer (Cin 3, Cout 64); W must be a multiple of 14 and H of 8.
bool tc_conv12_fused_supported(ConvShape s);
cudaError_t tc_conv12_fused(const bf16* x8, const bf16* w8, const float* bias1, const bf16* wt2_tap_major, const float* bias2,
                            bf16* out, bf16* pooled, ConvShape s, int* dev_error, cudaStream_t st);

// Self-test of the bounded-wait plumbing: one CTA of 32 threads initialises an mbarrier in shared
// memory on which nothing ever arrives and waits for it with a limit of `limit_cycles` SM cycles; the
// wait runs out, kDevTimeoutTest lands in dev_error and the kernel returns normally.  No TMA, no
// tensor memory, nothing in flight when it gives up.
cudaError_t tc_wait_selftest(int* dev_error, long long limit_cycles, cudaStream_t st);

}  // namespace vgg
