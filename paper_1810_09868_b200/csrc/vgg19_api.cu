// C-ABI of the VGG19 device library: the static layer table, the workspace
// plan, the order in which kernels are enqueued for a forward or a
// forward+backward pass, and the CUDA-graph cache that turns a pass into one
// launch (the counterpart of the paper's single offloaded executable,
// section 7.2).
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/vgg19_b200.h"
#include "../../seeded_inputs/seeded_inputs.h"
#include "common.cuh"
#include "tc_kernels.cuh"

using namespace vgg;

namespace {

constexpr int kConvLayers = 16, kFcLayers = 3, kLayers = 19, kClasses = 1000;
const int kConvOut[kConvLayers] = {64, 64, 128, 128, 256, 256, 256, 256,
                                   512, 512, 512, 512, 512, 512, 512, 512};
const bool kPoolAfter[kConvLayers] = {false, true, false, true, false, false, false, true,
                                      false, false, false, true, false, false, false, true};

struct ConvLayer {
  int H, W, Cin, Cout;  // input spatial size = output spatial size
  bool pool_after;
  size_t w_off, b_off;  // element offsets in the flat parameter buffer
  size_t dgrad_off;     // element offset of the rotated filter in the dgrad filter buffer
};
struct FcLayer {
  int In, Out;
  bool relu;
  size_t w_off, b_off;
};

std::string g_create_error;

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

struct GraphEntry {
  int mode, batch;
  const void *p[6];
  cudaGraphExec_t exec;
  int n_kernels;
};

}  // namespace

struct vgg19 {
  vgg19_config cfg;
  size_t elt;  // bytes per activation element
  ConvLayer conv[kConvLayers];
  int pool_idx[kConvLayers];  // which of the five pools follows layer l, or -1
  FcLayer fc[kFcLayers];
  size_t n_params, n_dgrad;
  float *params = nullptr;   // fp32 master, device
  void *params_t = nullptr;  // copy in the storage dtype (aliases params in fp32 mode)
  void *dgrad_w = nullptr;   // rotated filters for layers 2..16, storage dtype
  bf16 *tap_fwd = nullptr;   // tap-major [9][Cout][Cin] filters of layers 2..16 (halo kernel), at dgrad_off
  bf16 *tap_bwd = nullptr;   // tap-major rotated filters [9][Cin][Cout] of the same layers
  bf16 *w8 = nullptr;        // first-layer filter padded to [64][10][8] (bf16 tensor-core path)
  half16 *split_w = nullptr; // fp32 configuration on tensor cores: rows [hi | lo | hi] (fp16 terms) of every weight matrix, at 3 * w_off
  int *dev_error = nullptr;
  void *ws = nullptr;
  size_t ws_bytes = 0;
  std::vector<GraphEntry> graphs;
  int launches[3] = {0, 0, 0};
  cudaEvent_t dense_grads_event = nullptr;  // caller's; recorded once the dense layers' gradients are final
  std::string err;
  bool use_tc = false;
  bool use_pair = false;  // two-CTA kernels where a layer's shape takes them
  bool use_split = false; // fp32 forward-only passes on tensor cores, three fp16 products per product
  // vgg19_forward_host_async: two staging slots, a stream of the library's own for the uploads, and per
  // slot an event for "images uploaded" and one for "the pass that used the slot has finished"
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_uploaded[2] = {nullptr, nullptr}, ev_consumed[2] = {nullptr, nullptr};
  bool slot_used[2] = {false, false};
  unsigned next_slot = 0;
  int async_batch = 0;        // batch of the last vgg19_forward_host_async call (0: none yet)
  bool other_pass = false;    // a pass went through another entry point since that call
  cudaEvent_t ev_order = nullptr;
};

namespace {

int fail(vgg19 *n, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (n) n->err = buf; else g_create_error = buf;
  return code;
}

#define CUDA_TRY(n, expr)                                                                   \
  do {                                                                                      \
    cudaError_t e_ = (expr);                                                                \
    if (e_ != cudaSuccess)                                                                  \
      return fail((n), VGG19_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e_), \
                  __FILE__, __LINE__);                                                      \
  } while (0)

// ---- workspace plan ---------------------------------------------------------
// All offsets in bytes from the workspace base, each 256-byte aligned.
struct Plan {
  size_t act[kConvLayers];  // y_l = relu(conv_l + b): [B][H][W][Cout]
  size_t pooled[5];         // outputs of the five pools
  size_t code[5];           // backward: one byte per pooled element, where its window's maximum sits
  size_t a1, a2;            // dense activations [B][4096]
  size_t logits, probs;     // fp32 [B][1000] (used when the caller passes none)
  size_t dl, dz2, dz1, dflat;  // backward: dlogits, dense pre-activation grads, d(flatten)
  size_t dza, dzb, dxlow;   // conv backward ping-pong and the pooled-resolution dx
  size_t partial;           // fp32 split-K partials
  size_t x8;                // image copied to 8 channels (bf16 tensor-core path of layer 1)
  bool valid = true;
  size_t row_loss, loss;
  size_t grads, lr;         // training step: the gradient buffer and the learning rate (a device scalar)
  size_t total;
  size_t io_images, io_labels, io_logits, io_probs, io_grads, io_loss, io_total;
};

Plan make_plan(const vgg19 *n, int B, int mode) {
  Plan p{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  int pi = 0;
  size_t max_act = 0, max_low = 0, max_partial = 0, conv_fwd_partial = 0;
  for (int l = 0; l < kConvLayers; ++l) {
    const ConvLayer &c = n->conv[l];
    size_t a = (size_t)B * c.H * c.W * c.Cout;
    p.act[l] = take(a * n->elt);
    if (a > max_act) max_act = a;
    if (c.pool_after) {
      p.pooled[pi++] = take(a / 4 * n->elt);
      if (a / 4 > max_low) max_low = a / 4;
    }
    ConvShape s{B, c.H, c.W, c.Cin, c.Cout};
    size_t pe = simt_wgrad_scratch_elems(s);
    size_t te = tc_wgrad_scratch_elems(s, n->use_pair);
    if (te > pe) pe = te;
    if (n->use_tc && tc_wgrad_patch_scratch_elems(s) > pe) pe = tc_wgrad_patch_scratch_elems(s);
    if (pe > max_partial) max_partial = pe;
    // tail-split scratch of the two-CTA convolution (forward, and input gradient with the channels swapped)
    if (n->use_pair) {
      size_t fe = tc_conv3x3_pair_scratch_elems(s), de = tc_conv3x3_pair_scratch_elems(ConvShape{B, c.H, c.W, c.Cout, c.Cin});
      if (fe > conv_fwd_partial) conv_fwd_partial = fe;
      if (fe > max_partial) max_partial = fe;
      if (de > max_partial) max_partial = de;
    }
  }
  p.x8 = take(n->use_tc ? (size_t)B * n->cfg.height * n->cfg.width * 16 : 0);
  {
    const ConvLayer &c = n->conv[0];
    size_t e = n->use_tc ? tc_first_wgrad_scratch_elems(ConvShape{B, c.H, c.W, c.Cin, c.Cout}) : 0;
    if (e > max_partial) max_partial = e;
  }
  p.a1 = take((size_t)B * 4096 * n->elt);
  p.a2 = take((size_t)B * 4096 * n->elt);
  p.logits = take((size_t)B * kClasses * 4);
  p.probs = take((size_t)B * kClasses * 4);
  size_t dense_partial = 0;
  for (int i = 0; i < kFcLayers; ++i) {
    size_t e = tc_dense_scratch_elems(B, n->fc[i].In, n->fc[i].Out);
    if (n->use_split && tc_dense_split_scratch_elems(B, n->fc[i].In, n->fc[i].Out) > e)
      e = tc_dense_split_scratch_elems(B, n->fc[i].In, n->fc[i].Out);
    if (e > dense_partial) dense_partial = e;
  }
  if (1024 * 512 > max_partial) max_partial = 1024 * 512;  // bias-gradient column sums
  if (conv_fwd_partial > dense_partial) dense_partial = conv_fwd_partial;
  if (mode == VGG19_MODE_FORWARD) p.partial = take(dense_partial * 4);
  if (dense_partial > max_partial) max_partial = dense_partial;
  const bool train = mode == VGG19_MODE_TRAIN;
  if (train) mode = VGG19_MODE_BACKWARD;
  if (mode == VGG19_MODE_BACKWARD) {
    for (int l = 0, k = 0; l < kConvLayers; ++l)
      if (n->conv[l].pool_after) p.code[k++] = take((size_t)B * (n->conv[l].H / 2) * (n->conv[l].W / 2) * n->conv[l].Cout);
    p.dl = take((size_t)B * kClasses * n->elt);
    p.dz2 = take((size_t)B * 4096 * n->elt);
    p.dz1 = take((size_t)B * 4096 * n->elt);
    p.dflat = take((size_t)B * n->fc[0].In * n->elt);
    p.dza = take(max_act * n->elt);
    p.dzb = take(max_act * n->elt);
    p.dxlow = take(max_low * n->elt);
    p.partial = take(max_partial * 4);
    p.row_loss = take((size_t)B * 4);
    p.loss = take(256);
  }
  if (train) {
    p.grads = take(n->n_params * 4);
    p.lr = take(256);
  }
  p.total = off;
  size_t io = off;
  auto take_io = [&](size_t bytes) { size_t o = io; io += align_up(bytes); return o; };
  p.io_images = take_io((size_t)B * n->cfg.height * n->cfg.width * 3 * n->elt);
  p.io_logits = take_io((size_t)B * kClasses * 4);
  p.io_probs = take_io((size_t)B * kClasses * 4);
  if (mode == VGG19_MODE_BACKWARD) {
    p.io_labels = take_io((size_t)B * 4);
    p.io_grads = take_io(n->n_params * 4);
    p.io_loss = take_io(256);
  }
  p.io_total = io - off;
  return p;
}

// ---- enqueueing a pass ------------------------------------------------------

struct PassArgs {
  const void *images;
  const int32_t *labels;
  float *logits, *probs, *grads, *loss;
  int batch;
  int steps = 1;  // training mode: batches taken in turn by one recorded graph
};

template <typename T>
struct Pass {
  vgg19 *n;
  Plan p;
  cudaStream_t st;
  int launches = 0;
  cudaError_t err = cudaSuccess;
  bool keep_activations = true;  // false in a forward-only pass: nothing will read a pre-pool output again
  // Whether a forward convolution may cut the tiles of its last round along K.  That changes the fp32
  // summation order of the images in those tiles with the batch size, so a training pass, whose ReLU and
  // pooling decisions should not depend on what else is in the batch, keeps it off for its forward half.
  bool forward_tail_split = true;
  const void *x8_of = nullptr;  // the image whose 8-channel copy this pass has already made
  // fp32 configuration, forward only: activations travel as [hi | lo] fp16 terms (the same bytes as fp32) and
  // layers 2..16 and the dense layers run on tensor cores with three fp16 products per product
  bool split = false;
  // Training step on one GPU: the learning rate (device scalar).  Where a filter-gradient kernel can
  // apply the update itself (the dense layers' GEMM: 86 % of the parameters at 224x224) the gradient is
  // never stored; `folded` tells the caller which parameter ranges are already updated.
  const float *fold_lr = nullptr;
  bool folded[kFcLayers] = {false, false, false};

  T *buf(size_t off) const { return reinterpret_cast<T *>(static_cast<char *>(n->ws) + off); }
  float *fbuf(size_t off) const { return reinterpret_cast<float *>(static_cast<char *>(n->ws) + off); }
  const T *wt(size_t off) const { return static_cast<const T *>(n->params_t) + off; }
  void ok(cudaError_t e, int k) { if (err == cudaSuccess) err = e; launches += k; }

  bool tc_conv_ok(const ConvShape &s) const { return n->use_tc && tc_conv3x3_supported(s); }
  bool pair_ok(const ConvShape &s) const { return n->use_pair && tc_conv3x3_pair_supported(s); }
  // layer 1 on tensor cores needs the 8-channel image copy, i.e. a planned workspace
  bool first_tc_ok(int l, const ConvShape &s) const {
    return l == 0 && n->use_tc && p.valid && tc_first_conv_supported(s);
  }

  // whether layer l's forward kernel can leave out the full-resolution output and write only the pooled one
  bool pools_in_epilogue(int l, int B) const {
    const ConvLayer &c = n->conv[l];
    ConvShape s{B, c.H, c.W, c.Cin, c.Cout};
    if (!n->use_tc || first_tc_ok(l, s) || l == 0) return false;
    return tc_conv3x3_rowshift_supported(s) || tc_conv3x3_halo_supported(s) || (pair_ok(s) && c.H % 2 == 0 && c.W % 2 == 0);
  }

  // y = relu(conv(x) + b), optionally pooled.  With need_y false the full-resolution output may be
  // left unwritten when the pool is fused into the convolution's epilogue.
  // code (with pooled, or null): receives the arg-max code of every pooling window for the backward pass.
  void conv_forward(int l, const T *x, int B, T *y, T *pooled, bool need_y = true, uint8_t *code = nullptr) {
    const ConvLayer &c = n->conv[l];
    ConvShape s{B, c.H, c.W, c.Cin, c.Cout};
    if (split) {
      // layer 1 (3 input channels) stays on the CUDA cores in fp32 and its output is split in place; the others
      // read and write split tensors.  The last pool writes one [all hi | all lo] row per image for dense 1.
      if (l == 0) {
        ok(simt_conv3x3<T>(x, wt(c.w_off), n->params + c.b_off, nullptr, y, s, true, st), 1);
        ok(split_rows((const float *)y, (half16 *)y, (long)B * c.H * c.W, c.Cout, n->dev_error, st), 1);
      } else {
        ok(tc_conv3x3_split((const half16 *)x, n->split_w + 3 * c.w_off, n->params + c.b_off, (half16 *)y, s, true,
                            n->dev_error, st), 1);
      }
      if (pooled) ok(maxpool_split((const half16 *)y, (half16 *)pooled, B, c.H, c.W, c.Cout, l == kConvLayers - 1, st), 1);
      return;
    }
    if (first_tc_ok(l, s)) {
      ok(tc_pad_to8((const bf16 *)x, (bf16 *)buf(p.x8), (long)B * c.H * c.W, st), 1);
      x8_of = x;
      ok(tc_first_conv((const bf16 *)buf(p.x8), n->w8, n->params + c.b_off, (bf16 *)y, s, true, n->dev_error, st), 1);
    } else if (n->use_tc && tc_conv3x3_rowshift_supported(s)) {
      ok(tc_conv3x3_rowshift((const bf16 *)x, n->tap_fwd + c.dgrad_off, n->params + c.b_off, nullptr,
                             (need_y || !pooled) ? (bf16 *)y : nullptr, (bf16 *)pooled, s, true, n->dev_error, st,
                             pooled ? code : nullptr), 1);
      return;
    } else if (n->use_tc && tc_conv3x3_halo_supported(s)) {
      ok(tc_conv3x3_halo((const bf16 *)x, n->tap_fwd + c.dgrad_off, n->params + c.b_off, nullptr,
                         (need_y || !pooled) ? (bf16 *)y : nullptr, (bf16 *)pooled, s, true, n->dev_error, st, n->use_pair,
                         pooled ? code : nullptr), 1);
      return;
    } else if (pair_ok(s)) {
      // a block-ending layer whose own output nobody reads again pools in its epilogue
      const bool pool_only = pooled && !need_y && !code && c.H % 2 == 0 && c.W % 2 == 0;
      int k = 1;
      ok(tc_conv3x3_pair((const bf16 *)x, (const bf16 *)wt(c.w_off), n->params + c.b_off, nullptr,
                         (bf16 *)y, s, true, n->dev_error, st, p.valid && forward_tail_split ? fbuf(p.partial) : nullptr, &k,
                         pool_only ? (bf16 *)pooled : nullptr), 0);
      launches += k + (pool_only ? 1 : 0);
      if (pool_only) return;
    } else if (tc_conv_ok(s))
      ok(tc_conv3x3((const bf16 *)x, (const bf16 *)wt(c.w_off), n->params + c.b_off, nullptr,
                    (bf16 *)y, s, true, n->dev_error, st), 1);
    else
      ok(simt_conv3x3<T>(x, wt(c.w_off), n->params + c.b_off, nullptr, y, s, true, st), 1);
    if (pooled) ok(simt_maxpool_fwd<T>(y, pooled, B, c.H, c.W, c.Cout, st, code), 1);
  }

  // dW, db from (x, dz); dx = dgrad(dz) [* (mask > 0)] unless dx is null.  With code and dx_full (the
  // layer's input is a pooled tensor): dx_full [B][2H][2W][Cin] = dgrad(dz) scattered through the pool by
  // the stored arg-max codes, in the input-gradient kernel's own epilogue where that kernel can, else
  // by way of dx (then scratch for the pooled-resolution gradient) and a scatter kernel.
  void conv_backward(int l, const T *x, const T *dz, int B, float *dW, float *db, T *dx,
                     const T *mask, const uint8_t *code = nullptr, T *dx_full = nullptr) {
    const ConvLayer &c = n->conv[l];
    ConvShape s{B, c.H, c.W, c.Cin, c.Cout};
    if (!dW) {
      // input gradient only (per-layer entry point)
    } else if (first_tc_ok(l, s)) {
      if (x8_of != x) ok(tc_pad_to8((const bf16 *)x, (bf16 *)buf(p.x8), (long)B * c.H * c.W, st), 1);  // the forward half's copy serves
      ok(tc_first_wgrad((const bf16 *)buf(p.x8), (const bf16 *)dz, dW, db, fbuf(p.partial), s, n->dev_error, st), 2);
    } else if (n->use_tc && tc_wgrad_patch_supported(s)) {
      ok(tc_conv3x3_wgrad_patch((const bf16 *)x, (const bf16 *)dz, dW, db, fbuf(p.partial), s, n->dev_error, st), 2);
    } else if (n->use_tc && tc_wgrad_supported(s)) {
      ok(tc_conv3x3_wgrad((const bf16 *)x, (const bf16 *)dz, dW, db, fbuf(p.partial), s, n->dev_error, st, n->use_pair),
         tc_wgrad_launches(s, db != nullptr, n->use_pair));
    } else
      ok(simt_conv3x3_wgrad<T>(x, dz, dW, db, fbuf(p.partial), s, st), 4);
    if (dx) {
      ConvShape t{B, c.H, c.W, c.Cout, c.Cin};  // a 3x3 correlation from Cout to Cin channels
      const T *wr = static_cast<const T *>(n->dgrad_w) + c.dgrad_off;
      if (code && n->use_tc && tc_conv3x3_rowshift_supported(t)) {
        ok(tc_conv3x3_rowshift((const bf16 *)dz, n->tap_bwd + c.dgrad_off, nullptr, nullptr, nullptr, nullptr, t, false,
                               n->dev_error, st, nullptr, code, (bf16 *)dx_full), 1);
        return;
      } else if (code && n->use_tc && tc_conv3x3_halo_supported_unpooled(t)) {
        ok(tc_conv3x3_halo((const bf16 *)dz, n->tap_bwd + c.dgrad_off, nullptr, nullptr, nullptr, nullptr, t, false,
                           n->dev_error, st, n->use_pair, nullptr, code, (bf16 *)dx_full), 1);
        return;
      }
      if (n->use_tc && tc_conv3x3_rowshift_supported(t))
        ok(tc_conv3x3_rowshift((const bf16 *)dz, n->tap_bwd + c.dgrad_off, nullptr, (const bf16 *)mask, (bf16 *)dx, nullptr,
                               t, false, n->dev_error, st), 1);
      else if (n->use_tc && tc_conv3x3_halo_supported_unpooled(t))
        ok(tc_conv3x3_halo((const bf16 *)dz, n->tap_bwd + c.dgrad_off, nullptr, (const bf16 *)mask, (bf16 *)dx, nullptr, t,
                           false, n->dev_error, st, n->use_pair), 1);
      else if (pair_ok(t)) {
        int k = 1;
        ok(tc_conv3x3_pair((const bf16 *)dz, (const bf16 *)wr, nullptr, (const bf16 *)mask, (bf16 *)dx,
                           t, false, n->dev_error, st, p.valid ? fbuf(p.partial) : nullptr, &k), 0);
        launches += k;
      } else if (tc_conv_ok(t))
        ok(tc_conv3x3((const bf16 *)dz, (const bf16 *)wr, nullptr, (const bf16 *)mask, (bf16 *)dx,
                      t, false, n->dev_error, st), 1);
      else
        ok(simt_conv3x3<T>(dz, wr, nullptr, mask, dx, t, false, st), 1);
      if (code) ok(simt_pool_scatter<T>(code, dx, dx_full, B, 2 * c.H, 2 * c.W, c.Cin, st), 1);
    }
  }

  bool tc_dense_ok(int B, const FcLayer &f) const { return n->use_tc && tc_dense_supported(B, f.In, f.Out); }

  void dense_forward(const FcLayer &f, const T *x, int B, T *out_t, float *out_f) {
    if (split) {
      // fp32 result into the output buffer, then split in place for the next layer (the logits stay fp32)
      float *o = out_f ? out_f : (float *)out_t;
      ok(tc_dense_forward_split((const half16 *)x, n->split_w + 3 * f.w_off, n->params + f.b_off, o, fbuf(p.partial), B,
                                f.In, f.Out, f.relu, n->dev_error, st), 2);
      if (!out_f) ok(split_rows(o, (half16 *)out_t, B, f.Out, n->dev_error, st), 1);
      return;
    }
    if (tc_dense_ok(B, f))
      ok(tc_dense_forward((const bf16 *)x, (const bf16 *)wt(f.w_off), n->params + f.b_off, (bf16 *)out_t, out_f,
                          fbuf(p.partial), B, f.In, f.Out, f.relu, n->dev_error, st), 2);
    else
      ok(simt_dense_nt<T>(x, wt(f.w_off), n->params + f.b_off, nullptr, out_t, out_f, B, f.Out, f.In, f.relu, st), 1);
  }

  // dW, db from (x, dy); dx = (dy W) [* (mask > 0)]
  void dense_backward(const FcLayer &f, const T *x, const T *dy, int B, float *dW, float *db, T *dx, const T *mask) {
    if (tc_dense_ok(B, f)) {
      ok(simt_dense_db<T>(dy, db, B, f.Out, st), 1);
      // the input gradient reads the weights: it comes before a filter gradient that updates them in place
      ok(tc_dense_dx((const bf16 *)dy, (const bf16 *)wt(f.w_off), (const bf16 *)mask, (bf16 *)dx, fbuf(p.partial), B,
                     f.In, f.Out, n->dev_error, st), 2);
      if (fold_lr && f.In % 32 == 0) {
        ok(tc_dense_dw((const bf16 *)dy, (const bf16 *)x, n->params + f.w_off, B, f.In, f.Out, n->dev_error, st,
                       (bf16 *)n->params_t + f.w_off, fold_lr), 1);
        folded[&f - n->fc] = true;
      } else {
        ok(tc_dense_dw((const bf16 *)dy, (const bf16 *)x, dW, B, f.In, f.Out, n->dev_error, st), 1);
      }
    } else {
      ok(simt_dense_dw<T>(dy, x, dW, db, B, f.In, f.Out, st), 2);
      ok(simt_dense_dx<T>(dy, wt(f.w_off), mask, dx, B, f.In, f.Out, st), 1);
    }
  }

  // conv1_1 -> conv1_2 as one kernel (neither layer's full-resolution output is stored): forward-only passes
  bool first_block_fused_ok(int B) const {
    const ConvLayer &c0 = n->conv[0], &c1 = n->conv[1];
    return n->use_tc && p.valid && c1.Cin == 64 && c1.Cout == 64 &&
           tc_conv12_fused_supported(ConvShape{B, c0.H, c0.W, c0.Cin, c0.Cout});
  }
  void first_block_fused(const T *x, int B, T *y2, T *pooled) {
    const ConvLayer &c0 = n->conv[0], &c1 = n->conv[1];
    ok(tc_pad_to8((const bf16 *)x, (bf16 *)buf(p.x8), (long)B * c0.H * c0.W, st), 1);
    x8_of = x;
    ok(tc_conv12_fused((const bf16 *)buf(p.x8), n->w8, n->params + c0.b_off, n->tap_fwd + c1.dgrad_off, n->params + c1.b_off,
                       (bf16 *)y2, (bf16 *)pooled, ConvShape{B, c0.H, c0.W, c0.Cin, c0.Cout}, n->dev_error, st), 1);
  }

  void forward(const PassArgs &a) {
    const int B = a.batch;
    const T *x = static_cast<const T *>(a.images);
    int pi = 0;
    int first = 0;
    // (opt-in: at batch 100 the fused kernel measures 0.55 ms against 0.51 ms for the two kernels it replaces)
    if (!keep_activations && !a.grads && (n->cfg.flags & VGG19_FLAG_FIRST_FUSION) && n->conv[1].pool_after &&
        first_block_fused_ok(B)) {
      first_block_fused(x, B, nullptr, buf(p.pooled[0]));
      x = buf(p.pooled[0]);
      pi = 1; first = 2;
    }
    for (int l = first; l < kConvLayers; ++l) {
      T *y = buf(p.act[l]);
      T *pooled = n->conv[l].pool_after ? buf(p.pooled[pi]) : nullptr;
      // a pass that will run backward stores, with each pooled tensor, where every window's maximum sat
      uint8_t *code = pooled && a.grads ? reinterpret_cast<uint8_t *>(static_cast<char *>(n->ws) + p.code[pi]) : nullptr;
      if (pooled) ++pi;
      conv_forward(l, x, B, y, pooled, keep_activations, code);
      x = pooled ? pooled : y;
    }
    float *logits = a.logits ? a.logits : fbuf(p.logits);
    const FcLayer *f = n->fc;
    dense_forward(f[0], x, B, buf(p.a1), nullptr);
    dense_forward(f[1], buf(p.a1), B, buf(p.a2), nullptr);
    dense_forward(f[2], buf(p.a2), B, nullptr, logits);
    if (a.probs && !a.grads)
      ok(softmax_xent<T>(logits, nullptr, a.probs, nullptr, nullptr, nullptr, B, kClasses, st), 1);
  }

  void backward(const PassArgs &a) {
    const int B = a.batch;
    forward(a);
    float *logits = a.logits ? a.logits : fbuf(p.logits);
    float *loss = a.loss ? a.loss : fbuf(p.loss);
    float *g = a.grads;
    const FcLayer *f = n->fc;
    ok(softmax_xent<T>(logits, a.labels, a.probs, buf(p.dl), fbuf(p.row_loss), loss, B, kClasses,
                       st, n->dev_error), 2);
    const T *flat = buf(p.pooled[4]);
    // dense 3, 2, 1: filter gradient, then input gradient masked by the ReLU below
    dense_backward(f[2], buf(p.a2), buf(p.dl), B, g + f[2].w_off, g + f[2].b_off, buf(p.dz2), buf(p.a2));
    dense_backward(f[1], buf(p.a1), buf(p.dz2), B, g + f[1].w_off, g + f[1].b_off, buf(p.dz1), buf(p.a1));
    dense_backward(f[0], flat, buf(p.dz1), B, g + f[0].w_off, g + f[0].b_off, buf(p.dflat), nullptr);
    if (n->dense_grads_event && err == cudaSuccess) {
      // the dense layers' gradients (the tail of the flat buffer, 86 % of it at 224x224) are final here:
      // a caller's exchange of them can run beside the convolution layers' backward pass.  Inside a
      // capture the record becomes a node of the graph that signals the caller's (external) event.
      cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
      cudaStreamIsCapturing(st, &cs);
      err = cudaEventRecordWithFlags(n->dense_grads_event, st,
                                     cs == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault);
    }
    // convolutions 16..1.  `dz` is the gradient at layer l's pre-activation.
    T *dz = buf(p.dza), *other = buf(p.dzb);
    auto code_of = [&](int pool) { return reinterpret_cast<const uint8_t *>(static_cast<char *>(n->ws) + p.code[pool]); };
    {
      const ConvLayer &c = n->conv[15];
      ok(simt_pool_scatter<T>(code_of(4), buf(p.dflat), dz, B, c.H, c.W, c.Cout, st), 1);
    }
    for (int l = kConvLayers - 1; l >= 0; --l) {
      const ConvLayer &c = n->conv[l];
      const bool in_is_pool = l > 0 && n->conv[l - 1].pool_after;
      const T *x = l == 0 ? static_cast<const T *>(a.images)
                          : (in_is_pool ? buf(p.pooled[n->pool_idx[l - 1]]) : buf(p.act[l - 1]));
      float *dW = g + c.w_off, *db = g + c.b_off;
      if (l == 0) {
        conv_backward(l, x, dz, B, dW, db, nullptr, nullptr);
      } else if (in_is_pool) {
        conv_backward(l, x, dz, B, dW, db, buf(p.dxlow), nullptr, code_of(n->pool_idx[l - 1]), other);
      } else {
        conv_backward(l, x, dz, B, dW, db, other, buf(p.act[l - 1]));
      }
      T *t = dz; dz = other; other = t;
    }
  }
};

int check_batch(vgg19 *n, int batch, int mode, size_t extra) {
  if (batch < 1 || batch > n->cfg.batch_max)
    return fail(n, VGG19_ERR_ARG, "batch %d outside [1, %d]", batch, n->cfg.batch_max);
  Plan p = make_plan(n, batch, mode);
  if (!n->ws) return fail(n, VGG19_ERR_WORKSPACE, "no workspace bound");
  if (n->ws_bytes < p.total + extra)
    return fail(n, VGG19_ERR_WORKSPACE, "workspace has %zu bytes, this call needs %zu", n->ws_bytes,
                p.total + extra);
  return VGG19_OK;
}

int refresh_filter_copies(vgg19 *n, cudaStream_t st);

template <typename T>
int enqueue(vgg19 *n, int mode, const PassArgs &a, cudaStream_t st, int *launches) {
  Pass<T> pass{n, make_plan(n, a.batch, mode), st};
  if (mode == VGG19_MODE_FORWARD) {
    pass.keep_activations = false;
    pass.split = n->use_split;
    pass.forward(a);
  } else if (mode == VGG19_MODE_BACKWARD) {
    pass.forward_tail_split = false;
    pass.backward(a);
  } else {
    // training steps: a.steps times [forward + backward on the next batch, parameter update], the
    // gradient staying in the workspace; images / labels / loss advance by one batch per step
    pass.forward_tail_split = false;
    const size_t img_stride = (size_t)a.batch * n->cfg.height * n->cfg.width * 3 * n->elt;
    for (int k = 0; k < a.steps && pass.err == cudaSuccess; ++k) {
      PassArgs b = a;
      b.images = static_cast<const char *>(a.images) + (size_t)k * img_stride;
      b.labels = a.labels + (size_t)k * a.batch;
      b.loss = a.loss ? a.loss + k : nullptr;
      b.grads = pass.fbuf(pass.p.grads);
      const float *lr = pass.fbuf(pass.p.lr);
      pass.fold_lr = lr;
      pass.backward(b);
      // update what the gradient kernels have not updated themselves: maximal runs of the flat buffer
      T *copy = n->cfg.dtype == VGG19_BF16 ? (T *)n->params_t : (T *)nullptr;
      size_t run0 = 0;
      for (int i = 0; i <= kFcLayers; ++i) {
        const size_t skip0 = i < kFcLayers ? n->fc[i].w_off : n->n_params;
        const bool skip = i < kFcLayers && pass.folded[i];
        if (i < kFcLayers && !skip) continue;
        if (skip0 > run0)
          pass.ok(sgd_update<T>(n->params + run0, b.grads + run0, copy ? copy + run0 : copy, 0.f, skip0 - run0, st, lr), 1);
        if (skip) run0 = n->fc[i].b_off;  // the layer's bias follows its weights
      }
      int rc = refresh_filter_copies(n, st);
      if (rc != VGG19_OK) return rc;
      pass.launches += n->use_tc ? 2 : 0;
    }
  }
  if (launches) *launches = pass.launches;
  n->launches[mode] = pass.launches;
  if (pass.err != cudaSuccess)
    return fail(n, VGG19_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(pass.err));
  return VGG19_OK;
}

int enqueue_any(vgg19 *n, int mode, const PassArgs &a, cudaStream_t st, int *launches) {
  return n->cfg.dtype == VGG19_BF16 ? enqueue<bf16>(n, mode, a, st, launches)
                                    : enqueue<float>(n, mode, a, st, launches);
}

// Run the pass: replay its CUDA graph when there is one for these pointers,
// else record it first.  The legacy default stream cannot be captured, so work
// given to it is enqueued directly.
int run_pass(vgg19 *n, int mode, const PassArgs &a, cudaStream_t st) {
  n->other_pass = true;  // vgg19_forward_host_async clears this again for its own passes
  if ((n->cfg.flags & VGG19_FLAG_NO_GRAPH) || st == nullptr || st == cudaStreamLegacy)
    return enqueue_any(n, mode, a, st, nullptr);
  const void *key[6] = {a.images, a.labels, a.logits, a.probs, mode == VGG19_MODE_TRAIN ? (const void *)(intptr_t)a.steps : a.grads,
                        a.loss};
  for (auto &g : n->graphs)
    if (g.mode == mode && g.batch == a.batch && !memcmp(g.p, key, sizeof key)) {
      CUDA_TRY(n, cudaGraphLaunch(g.exec, st));
      return VGG19_OK;
    }
  cudaGraph_t graph = nullptr;
  CUDA_TRY(n, cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
  int launches = 0;
  int rc = enqueue_any(n, mode, a, st, &launches);
  cudaError_t ce = cudaStreamEndCapture(st, &graph);
  if (rc != VGG19_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
  CUDA_TRY(n, ce);
  GraphEntry e{};
  size_t n_nodes = 0;
  if (cudaGraphGetNodes(graph, nullptr, &n_nodes) == cudaSuccess && n_nodes > 0) {
    // kernel launches of the captured pass (it also holds a few memset and event-record nodes)
    std::vector<cudaGraphNode_t> nodes(n_nodes);
    int kernels = 0;
    if (cudaGraphGetNodes(graph, nodes.data(), &n_nodes) == cudaSuccess)
      for (size_t i = 0; i < n_nodes; ++i) {
        cudaGraphNodeType t;
        if (cudaGraphNodeGetType(nodes[i], &t) == cudaSuccess && t == cudaGraphNodeTypeKernel) ++kernels;
      }
    if (kernels > 0) { launches = kernels; n->launches[mode] = launches; }
  }
  e.mode = mode; e.batch = a.batch; memcpy(e.p, key, sizeof key); e.n_kernels = launches;
  cudaError_t ie = cudaGraphInstantiate(&e.exec, graph, 0);
  cudaGraphDestroy(graph);
  CUDA_TRY(n, ie);
  if (n->graphs.size() >= 8) { cudaGraphExecDestroy(n->graphs.front().exec); n->graphs.erase(n->graphs.begin()); }
  n->graphs.push_back(e);
  CUDA_TRY(n, cudaGraphLaunch(e.exec, st));
  return VGG19_OK;
}

void drop_graphs(vgg19 *n) {
  for (auto &g : n->graphs) cudaGraphExecDestroy(g.exec);
  n->graphs.clear();
}

// The filter copies the kernels read besides the storage-type parameters (rotated filters of the input
// gradients, tap-major filters, the padded first-layer filter), rebuilt from the fp32 master on `st`.
int refresh_filter_copies(vgg19 *n, cudaStream_t st) {
  const bool h = n->cfg.dtype == VGG19_BF16;
  if (n->split_w) {
    for (int l = 1; l < kConvLayers; ++l) {
      const ConvLayer &c = n->conv[l];
      CUDA_TRY(n, split_weights(n->params + c.w_off, n->split_w + 3 * c.w_off, 9L * c.Cout, c.Cin, st));
    }
    for (int i = 0; i < kFcLayers; ++i) {
      const FcLayer &f = n->fc[i];
      CUDA_TRY(n, split_weights(n->params + f.w_off, n->split_w + 3 * f.w_off, f.Out, f.In, st));
    }
  }
  if (h && n->tap_fwd && n->tap_bwd) {
    // tensor-core configuration: all three bf16 copies of layers 2..16 in one launch
    FilterCopyTable tab{};
    tab.layers = kConvLayers - 1;
    long first = 0;
    for (int l = 1; l < kConvLayers; ++l) {
      const ConvLayer &c = n->conv[l];
      tab.first[l - 1] = first;
      tab.w_off[l - 1] = (long)c.w_off;
      tab.copy_off[l - 1] = (long)c.dgrad_off;
      tab.Cin[l - 1] = c.Cin; tab.Cout[l - 1] = c.Cout;
      first += 9L * (c.Cin / 32) * (c.Cout / 32);
    }
    tab.total = first;
    CUDA_TRY(n, vgg::refresh_filter_copies(n->params, (bf16 *)n->dgrad_w, n->tap_fwd, n->tap_bwd, tab, st));
    if (n->w8) CUDA_TRY(n, tc_make_first_filter(n->params + n->conv[0].w_off, n->w8, st));
    return VGG19_OK;
  }
  for (int l = 1; l < kConvLayers; ++l) {
    const ConvLayer &c = n->conv[l];
    if (h)
      CUDA_TRY(n, make_dgrad_filter<bf16>(n->params + c.w_off, (bf16 *)n->dgrad_w + c.dgrad_off, c.Cin, c.Cout, st));
    else
      CUDA_TRY(n, make_dgrad_filter<float>(n->params + c.w_off, (float *)n->dgrad_w + c.dgrad_off, c.Cin, c.Cout, st));
  }
  if (n->w8) CUDA_TRY(n, tc_make_first_filter(n->params + n->conv[0].w_off, n->w8, st));
  if (n->tap_fwd)
    for (int l = 1; l < kConvLayers; ++l) {
      const ConvLayer &c = n->conv[l];
      CUDA_TRY(n, tc_make_tap_major(n->params + c.w_off, n->tap_fwd + c.dgrad_off, c.Cin, c.Cout, false, st));
      CUDA_TRY(n, tc_make_tap_major(n->params + c.w_off, n->tap_bwd + c.dgrad_off, c.Cin, c.Cout, true, st));
    }
  return VGG19_OK;
}

int upload_params(vgg19 *n, const float *host) {
  CUDA_TRY(n, cudaMemcpy(n->params, host, n->n_params * 4, cudaMemcpyHostToDevice));
  if (n->cfg.dtype == VGG19_BF16) CUDA_TRY(n, convert_f32<bf16>(n->params, (bf16 *)n->params_t, n->n_params, 0));
  int rc = refresh_filter_copies(n, 0);
  if (rc != VGG19_OK) return rc;
  CUDA_TRY(n, cudaDeviceSynchronize());
  return VGG19_OK;
}

int create_common(const vgg19_config *cfg, vgg19 **out) {
  if (!cfg || !out) return fail(nullptr, VGG19_ERR_ARG, "null argument");
  *out = nullptr;
  if (cfg->dtype != VGG19_FP32 && cfg->dtype != VGG19_BF16)
    return fail(nullptr, VGG19_ERR_ARG, "dtype %d is neither VGG19_FP32 nor VGG19_BF16", cfg->dtype);
  if (cfg->height < 32 || cfg->width < 32 || cfg->height % 32 || cfg->width % 32)
    return fail(nullptr, VGG19_ERR_SHAPE, "height %d / width %d must be positive multiples of 32",
                cfg->height, cfg->width);
  if (cfg->batch_max < 1) return fail(nullptr, VGG19_ERR_ARG, "batch_max %d < 1", cfg->batch_max);
  if ((cfg->flags & VGG19_FLAG_SPLIT_F16) && cfg->dtype != VGG19_FP32)
    return fail(nullptr, VGG19_ERR_ARG, "VGG19_FLAG_SPLIT_F16 applies to the fp32 configuration only");
  int dev = 0;
  cudaDeviceProp prop;
  CUDA_TRY(nullptr, cudaGetDevice(&dev));
  CUDA_TRY(nullptr, cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10)
    return fail(nullptr, VGG19_ERR_UNSUPPORTED_ARCH, "device is sm_%d%d; this library is built for sm_100a only",
                prop.major, prop.minor);
  vgg19 *n = new (std::nothrow) vgg19();
  if (!n) return fail(nullptr, VGG19_ERR_ARG, "out of host memory");
  n->cfg = *cfg;
  n->elt = cfg->dtype == VGG19_BF16 ? 2 : 4;
  n->use_tc = cfg->dtype == VGG19_BF16 && !(cfg->flags & VGG19_FLAG_NO_TENSOR_CORES);
  n->use_pair = n->use_tc && !(cfg->flags & VGG19_FLAG_NO_CTA_PAIRS);
  n->use_split = cfg->dtype == VGG19_FP32 && (cfg->flags & VGG19_FLAG_SPLIT_F16) != 0;
  size_t off = 0, doff = 0;
  int h = cfg->height, w = cfg->width, cin = 3, n_pool = 0;
  for (int l = 0; l < kConvLayers; ++l) {
    ConvLayer &c = n->conv[l];
    n->pool_idx[l] = kPoolAfter[l] ? n_pool++ : -1;
    c.H = h; c.W = w; c.Cin = cin; c.Cout = kConvOut[l]; c.pool_after = kPoolAfter[l];
    c.w_off = off; off += (size_t)c.Cout * 9 * c.Cin;
    c.b_off = off; off += c.Cout;
    c.dgrad_off = doff;
    if (l > 0) doff += (size_t)c.Cout * 9 * c.Cin;
    cin = c.Cout;
    if (c.pool_after) { h /= 2; w /= 2; }
  }
  const int fc_dims[4] = {512 * h * w, 4096, 4096, kClasses};
  for (int i = 0; i < kFcLayers; ++i) {
    FcLayer &f = n->fc[i];
    f.In = fc_dims[i]; f.Out = fc_dims[i + 1]; f.relu = i < 2;
    f.w_off = off; off += (size_t)f.In * f.Out;
    f.b_off = off; off += f.Out;
  }
  n->n_params = off;
  n->n_dgrad = doff;
  cudaError_t e = cudaMalloc(&n->params, n->n_params * 4);
  if (e == cudaSuccess) {
    if (cfg->dtype == VGG19_BF16) e = cudaMalloc(&n->params_t, n->n_params * 2);
    else n->params_t = n->params;
  }
  if (e == cudaSuccess) e = cudaMalloc(&n->dgrad_w, n->n_dgrad * n->elt);
  if (e == cudaSuccess && n->use_tc) e = cudaMalloc(&n->w8, 64 * 80 * sizeof(bf16));
  if (e == cudaSuccess && n->use_tc) e = cudaMalloc(&n->tap_fwd, n->n_dgrad * sizeof(bf16));
  if (e == cudaSuccess && n->use_tc) e = cudaMalloc(&n->tap_bwd, n->n_dgrad * sizeof(bf16));
  if (e == cudaSuccess && n->use_split) e = cudaMalloc(&n->split_w, 3 * n->n_params * sizeof(half16));
  if (e == cudaSuccess) e = cudaMalloc(&n->dev_error, 256);
  if (e == cudaSuccess) e = cudaMemset(n->dev_error, 0, 256);
  if (e != cudaSuccess) {
    int rc = fail(nullptr, VGG19_ERR_CUDA, "allocating parameters failed: %s", cudaGetErrorString(e));
    vgg19_destroy(n);
    return rc;
  }
  *out = n;
  return VGG19_OK;
}

}  // namespace

extern "C" {

int vgg19_create_from_params(const vgg19_config *cfg, const float *host_params, vgg19_t **out) {
  if (!host_params) return fail(nullptr, VGG19_ERR_ARG, "null host_params");
  int rc = create_common(cfg, out);
  if (rc != VGG19_OK) return rc;
  rc = upload_params(*out, host_params);
  if (rc != VGG19_OK) { g_create_error = (*out)->err; vgg19_destroy(*out); *out = nullptr; }
  return rc;
}

int vgg19_create(const vgg19_config *cfg, uint64_t seed, vgg19_t **out) {
  int rc = create_common(cfg, out);
  if (rc != VGG19_OK) return rc;
  std::vector<float> host;
  try { host.resize((*out)->n_params); } catch (...) {
    vgg19_destroy(*out); *out = nullptr;
    return fail(nullptr, VGG19_ERR_ARG, "out of host memory");
  }
  seeded_vgg19_params(host.data(), cfg->height, cfg->width, seed, 0.0, 0);
  rc = upload_params(*out, host.data());
  if (rc != VGG19_OK) { g_create_error = (*out)->err; vgg19_destroy(*out); *out = nullptr; }
  return rc;
}

void vgg19_destroy(vgg19_t *n) {
  if (!n) return;
  drop_graphs(n);
  if (n->params_t && n->params_t != (void *)n->params) cudaFree(n->params_t);
  if (n->params) cudaFree(n->params);
  if (n->dgrad_w) cudaFree(n->dgrad_w);
  if (n->w8) cudaFree(n->w8);
  if (n->split_w) cudaFree(n->split_w);
  if (n->tap_fwd) cudaFree(n->tap_fwd);
  if (n->tap_bwd) cudaFree(n->tap_bwd);
  if (n->dev_error) cudaFree(n->dev_error);
  if (n->copy_stream) cudaStreamDestroy(n->copy_stream);
  for (int i = 0; i < 2; ++i) {
    if (n->ev_uploaded[i]) cudaEventDestroy(n->ev_uploaded[i]);
    if (n->ev_consumed[i]) cudaEventDestroy(n->ev_consumed[i]);
  }
  if (n->ev_order) cudaEventDestroy(n->ev_order);
  delete n;
}

int vgg19_param_count(const vgg19_t *n, int32_t *n_tensors, size_t *n_elems) {
  if (!n) return VGG19_ERR_ARG;
  if (n_tensors) *n_tensors = 2 * kLayers;
  if (n_elems) *n_elems = n->n_params;
  return VGG19_OK;
}

int vgg19_param_info(const vgg19_t *n, int32_t i, size_t *offset, int32_t *rank, int64_t dims[4]) {
  if (!n || i < 0 || i >= 2 * kLayers) return VGG19_ERR_ARG;
  int l = i / 2;
  bool bias = i & 1;
  int64_t d[4] = {0, 0, 0, 0};
  int r;
  size_t off;
  if (l < kConvLayers) {
    const ConvLayer &c = n->conv[l];
    if (bias) { r = 1; d[0] = c.Cout; off = c.b_off; }
    else { r = 4; d[0] = c.Cout; d[1] = 3; d[2] = 3; d[3] = c.Cin; off = c.w_off; }
  } else {
    const FcLayer &f = n->fc[l - kConvLayers];
    if (bias) { r = 1; d[0] = f.Out; off = f.b_off; }
    else { r = 2; d[0] = f.Out; d[1] = f.In; off = f.w_off; }
  }
  if (offset) *offset = off;
  if (rank) *rank = r;
  if (dims) memcpy(dims, d, sizeof d);
  return VGG19_OK;
}

int vgg19_get_params(const vgg19_t *n, float *host) {
  if (!n || !host) return VGG19_ERR_ARG;
  return cudaMemcpy(host, n->params, n->n_params * 4, cudaMemcpyDeviceToHost) == cudaSuccess
             ? VGG19_OK : VGG19_ERR_CUDA;
}

int vgg19_set_params(vgg19_t *n, const float *host) {
  if (!n || !host) return VGG19_ERR_ARG;
  CUDA_TRY(n, cudaDeviceSynchronize());
  return upload_params(n, host);
}

int vgg19_sgd_step(vgg19_t *n, const float *grads, float lr, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!grads || !(lr == lr)) return fail(n, VGG19_ERR_ARG, "null gradient or NaN learning rate");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the parameter buffers keep their addresses, so recorded graphs stay valid
  if (n->cfg.dtype == VGG19_BF16)
    CUDA_TRY(n, sgd_update<bf16>(n->params, grads, (bf16 *)n->params_t, lr, n->n_params, st));
  else
    CUDA_TRY(n, sgd_update<float>(n->params, grads, (float *)nullptr, lr, n->n_params, st));
  return refresh_filter_copies(n, st);
}

int vgg19_train_steps(vgg19_t *n, const void *images, const int32_t *labels, int32_t batch, int32_t steps, float lr,
                      float *losses, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!images || !labels || steps < 1 || steps > 64 || !(lr == lr))
    return fail(n, VGG19_ERR_ARG, "null images / labels, steps outside [1, 64] or NaN learning rate");
  int rc = check_batch(n, batch, VGG19_MODE_TRAIN, 0);
  if (rc != VGG19_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Plan p = make_plan(n, batch, VGG19_MODE_TRAIN);
  // the rate is a device scalar the recorded update kernels read, so one graph serves every rate
  CUDA_TRY(n, set_scalar(reinterpret_cast<float *>(static_cast<char *>(n->ws) + p.lr), lr, st));
  PassArgs a{images, labels, nullptr, nullptr, nullptr, losses, batch, steps};
  return run_pass(n, VGG19_MODE_TRAIN, a, st);
}

int vgg19_train_step(vgg19_t *n, const void *images, const int32_t *labels, int32_t batch, float lr, float *loss,
                     void *stream) {
  return vgg19_train_steps(n, images, labels, batch, 1, lr, loss, stream);
}

int vgg19_set_dense_grads_event(vgg19_t *n, void *cuda_event) {
  if (!n) return VGG19_ERR_ARG;
  drop_graphs(n);  // recorded passes signal the event they were recorded with
  n->dense_grads_event = static_cast<cudaEvent_t>(cuda_event);
  return VGG19_OK;
}

size_t vgg19_workspace_bytes(const vgg19_t *n, int32_t batch, int32_t mode) {
  if (!n || batch < 1 || batch > n->cfg.batch_max || mode < 0 || mode > 2) return 0;
  return make_plan(n, batch, mode).total;
}

size_t vgg19_io_bytes(const vgg19_t *n, int32_t batch, int32_t mode) {
  if (!n || batch < 1 || batch > n->cfg.batch_max || (mode != 0 && mode != 1)) return 0;
  // the forward staging area is doubled: vgg19_forward_host_async alternates between two slots
  const Plan p = make_plan(n, batch, mode);
  return mode == VGG19_MODE_FORWARD ? 2 * p.io_total : p.io_total;
}

int vgg19_bind_workspace(vgg19_t *n, void *ws, size_t bytes) {
  if (!n) return VGG19_ERR_ARG;
  if (ws && (reinterpret_cast<uintptr_t>(ws) & 255))
    return fail(n, VGG19_ERR_ARG, "workspace must be 256-byte aligned");
  drop_graphs(n);
  n->ws = ws;
  n->ws_bytes = ws ? bytes : 0;
  return VGG19_OK;
}

int vgg19_forward(vgg19_t *n, const void *images, int32_t batch, float *logits, float *probs,
                  void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!images || !logits) return fail(n, VGG19_ERR_ARG, "images and logits must not be null");
  int rc = check_batch(n, batch, VGG19_MODE_FORWARD, 0);
  if (rc != VGG19_OK) return rc;
  PassArgs a{images, nullptr, logits, probs, nullptr, nullptr, batch};
  return run_pass(n, VGG19_MODE_FORWARD, a, static_cast<cudaStream_t>(stream));
}

int vgg19_backward(vgg19_t *n, const void *images, const int32_t *labels, int32_t batch,
                   float *grads, float *loss, float *logits, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!images || !labels || !grads)
    return fail(n, VGG19_ERR_ARG, "images, labels and grads must not be null");
  int rc = check_batch(n, batch, VGG19_MODE_BACKWARD, 0);
  if (rc != VGG19_OK) return rc;
  PassArgs a{images, labels, logits, nullptr, grads, loss, batch};
  return run_pass(n, VGG19_MODE_BACKWARD, a, static_cast<cudaStream_t>(stream));
}

int vgg19_forward_host(vgg19_t *n, const void *host_images, int32_t batch, float *host_logits,
                       float *host_probs, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!host_images) return fail(n, VGG19_ERR_ARG, "host_images must not be null");
  int rc = check_batch(n, batch, VGG19_MODE_FORWARD, 0);
  if (rc != VGG19_OK) return rc;
  Plan p = make_plan(n, batch, VGG19_MODE_FORWARD);
  rc = check_batch(n, batch, VGG19_MODE_FORWARD, p.io_total);
  if (rc != VGG19_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char *base = static_cast<char *>(n->ws);
  size_t img_bytes = (size_t)batch * n->cfg.height * n->cfg.width * 3 * n->elt;
  CUDA_TRY(n, cudaMemcpyAsync(base + p.io_images, host_images, img_bytes, cudaMemcpyHostToDevice, st));
  float *logits = reinterpret_cast<float *>(base + p.io_logits);
  float *probs = host_probs ? reinterpret_cast<float *>(base + p.io_probs) : nullptr;
  PassArgs a{base + p.io_images, nullptr, logits, probs, nullptr, nullptr, batch};
  rc = run_pass(n, VGG19_MODE_FORWARD, a, st);
  if (rc != VGG19_OK) return rc;
  size_t out_bytes = (size_t)batch * kClasses * 4;
  if (host_logits) CUDA_TRY(n, cudaMemcpyAsync(host_logits, logits, out_bytes, cudaMemcpyDeviceToHost, st));
  if (host_probs) CUDA_TRY(n, cudaMemcpyAsync(host_probs, probs, out_bytes, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(n, cudaStreamSynchronize(st));
  return VGG19_OK;
}

int vgg19_forward_host_async(vgg19_t *n, const void *host_images, int32_t batch, float *host_logits,
                             float *host_probs, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!host_images) return fail(n, VGG19_ERR_ARG, "host_images must not be null");
  int rc = check_batch(n, batch, VGG19_MODE_FORWARD, 0);
  if (rc != VGG19_OK) return rc;
  Plan p = make_plan(n, batch, VGG19_MODE_FORWARD);
  rc = check_batch(n, batch, VGG19_MODE_FORWARD, 2 * p.io_total);
  if (rc != VGG19_OK) return rc;
  if (!n->copy_stream) {
    CUDA_TRY(n, cudaStreamCreateWithFlags(&n->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      CUDA_TRY(n, cudaEventCreateWithFlags(&n->ev_uploaded[i], cudaEventDisableTiming));
      CUDA_TRY(n, cudaEventCreateWithFlags(&n->ev_consumed[i], cudaEventDisableTiming));
    }
    CUDA_TRY(n, cudaEventCreateWithFlags(&n->ev_order, cudaEventDisableTiming));
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The staging slots sit behind the work area of a pass at THIS batch.  A pass enqueued earlier at
  // another batch (or through another entry point) has a work area of another size, which may cover
  // this call's slots: the early upload would then overwrite activations that pass is still using.
  // In that case the upload waits for everything enqueued on `stream` so far instead of for the
  // slot's last reader only.
  if (n->async_batch != batch || n->other_pass) {
    CUDA_TRY(n, cudaEventRecord(n->ev_order, st));
    CUDA_TRY(n, cudaStreamWaitEvent(n->copy_stream, n->ev_order, 0));
  }
  const unsigned slot = n->next_slot++ & 1u;
  char *base = static_cast<char *>(n->ws) + (size_t)slot * p.io_total;
  size_t img_bytes = (size_t)batch * n->cfg.height * n->cfg.width * 3 * n->elt;
  // upload on the library's stream, as soon as the pass that last read this slot is done: it overlaps
  // whatever `stream` is still computing
  if (n->slot_used[slot]) CUDA_TRY(n, cudaStreamWaitEvent(n->copy_stream, n->ev_consumed[slot], 0));
  CUDA_TRY(n, cudaMemcpyAsync(base + p.io_images, host_images, img_bytes, cudaMemcpyHostToDevice, n->copy_stream));
  CUDA_TRY(n, cudaEventRecord(n->ev_uploaded[slot], n->copy_stream));
  CUDA_TRY(n, cudaStreamWaitEvent(st, n->ev_uploaded[slot], 0));
  float *logits = reinterpret_cast<float *>(base + p.io_logits);
  float *probs = host_probs ? reinterpret_cast<float *>(base + p.io_probs) : nullptr;
  PassArgs a{base + p.io_images, nullptr, logits, probs, nullptr, nullptr, batch};
  rc = run_pass(n, VGG19_MODE_FORWARD, a, st);
  if (rc != VGG19_OK) return rc;
  size_t out_bytes = (size_t)batch * kClasses * 4;
  if (host_logits) CUDA_TRY(n, cudaMemcpyAsync(host_logits, logits, out_bytes, cudaMemcpyDeviceToHost, st));
  if (host_probs) CUDA_TRY(n, cudaMemcpyAsync(host_probs, probs, out_bytes, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(n, cudaEventRecord(n->ev_consumed[slot], st));
  n->slot_used[slot] = true;
  n->async_batch = batch;
  n->other_pass = false;
  return VGG19_OK;
}

int vgg19_backward_host(vgg19_t *n, const void *host_images, const int32_t *host_labels,
                        int32_t batch, float *host_grads, float *host_loss, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!host_images || !host_labels) return fail(n, VGG19_ERR_ARG, "host_images and host_labels must not be null");
  int rc = check_batch(n, batch, VGG19_MODE_BACKWARD, 0);
  if (rc != VGG19_OK) return rc;
  Plan p = make_plan(n, batch, VGG19_MODE_BACKWARD);
  rc = check_batch(n, batch, VGG19_MODE_BACKWARD, p.io_total);
  if (rc != VGG19_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char *base = static_cast<char *>(n->ws);
  size_t img_bytes = (size_t)batch * n->cfg.height * n->cfg.width * 3 * n->elt;
  CUDA_TRY(n, cudaMemcpyAsync(base + p.io_images, host_images, img_bytes, cudaMemcpyHostToDevice, st));
  CUDA_TRY(n, cudaMemcpyAsync(base + p.io_labels, host_labels, (size_t)batch * 4, cudaMemcpyHostToDevice, st));
  float *grads = reinterpret_cast<float *>(base + p.io_grads);
  float *loss = reinterpret_cast<float *>(base + p.io_loss);
  PassArgs a{base + p.io_images, reinterpret_cast<const int32_t *>(base + p.io_labels), nullptr,
             nullptr, grads, loss, batch};
  rc = run_pass(n, VGG19_MODE_BACKWARD, a, st);
  if (rc != VGG19_OK) return rc;
  if (host_grads) CUDA_TRY(n, cudaMemcpyAsync(host_grads, grads, n->n_params * 4, cudaMemcpyDeviceToHost, st));
  if (host_loss) CUDA_TRY(n, cudaMemcpyAsync(host_loss, loss, 4, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(n, cudaStreamSynchronize(st));
  return VGG19_OK;
}

int vgg19_conv_layer_forward(vgg19_t *n, int32_t layer, const void *x, int32_t batch, void *y,
                             void *pooled, void *stream) {
  return vgg19_conv_layer_forward_ex(n, layer, x, batch, y, pooled, nullptr, stream);
}

int vgg19_conv_layer_forward_ex(vgg19_t *n, int32_t layer, const void *x, int32_t batch, void *y, void *pooled,
                                uint8_t *pool_code, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (layer < 1 || layer > kConvLayers || !x || (!y && !pooled) || batch < 1 || (pool_code && (!pooled || !y)))
    return fail(n, VGG19_ERR_ARG, "bad layer (%d), batch (%d) or null tensor", layer, batch);
  if (pooled && !n->conv[layer - 1].pool_after) {
    // pooling after any layer is well defined; only the fused schedule is per-layer
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  n->other_pass = true;
  cudaError_t e;
  Plan plan{};
  plan.valid = false;  // without a bound workspace the layer runs on kernels that need no scratch
  if (n->ws && batch <= n->cfg.batch_max) {
    Plan full = make_plan(n, batch, VGG19_MODE_FORWARD);
    if (n->ws_bytes >= full.total) plan = full;
  }
  if (n->cfg.dtype == VGG19_BF16) {
    Pass<bf16> ps{n, plan, st};
    if (!y && !ps.pools_in_epilogue(layer - 1, batch))
      return fail(n, VGG19_ERR_ARG, "layer %d at this size has no pooled-only kernel: y must not be null", layer);
    ps.conv_forward(layer - 1, (const bf16 *)x, batch, (bf16 *)y, (bf16 *)pooled, y != nullptr, pool_code);
    e = ps.err;
  } else if (n->use_split && layer > 1) {
    // fp32 tensors in and out; between them the layer runs on its split form: x is split into the workspace slot
    // a whole pass would read it from, y and pooled receive split tensors and are merged in place
    const ConvLayer &c = n->conv[layer - 1];
    if (!y || pool_code) return fail(n, VGG19_ERR_ARG, "the fp32 configuration has no pooled-only kernel and stores no pool codes here");
    if (!plan.valid) return fail(n, VGG19_ERR_WORKSPACE, "this layer needs the forward workspace bound");
    if (!split_rows_supported(c.Cin) || !split_rows_supported(c.Cout))
      return fail(n, VGG19_ERR_SHAPE, "channel counts %d -> %d do not divide 4096", c.Cin, c.Cout);
    Pass<float> ps{n, plan, st};
    ps.split = true;
    const bool in_is_pool = n->conv[layer - 2].pool_after;
    half16 *xs = (half16 *)ps.buf(in_is_pool ? plan.pooled[n->pool_idx[layer - 2]] : plan.act[layer - 2]);
    ps.ok(split_rows((const float *)x, xs, (long)batch * c.H * c.W, c.Cin, n->dev_error, st), 1);
    ps.conv_forward(layer - 1, (const float *)xs, batch, (float *)y, nullptr);
    if (pooled) {
      ps.ok(maxpool_split((const half16 *)y, (half16 *)pooled, batch, c.H, c.W, c.Cout, false, st), 1);
      ps.ok(merge_rows((const half16 *)pooled, (float *)pooled, (long)batch * (c.H / 2) * (c.W / 2), c.Cout, st), 1);
    }
    ps.ok(merge_rows((const half16 *)y, (float *)y, (long)batch * c.H * c.W, c.Cout, st), 1);
    e = ps.err;
  } else {
    Pass<float> ps{n, plan, st};
    if (!y) return fail(n, VGG19_ERR_ARG, "the fp32 configuration has no pooled-only kernel: y must not be null");
    ps.conv_forward(layer - 1, (const float *)x, batch, (float *)y, (float *)pooled, y != nullptr, pool_code);
    e = ps.err;
  }
  if (e != cudaSuccess) return fail(n, VGG19_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return VGG19_OK;
}

int vgg19_first_block_forward(vgg19_t *n, const void *images, int32_t batch, void *y2, void *pooled, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!images || (!y2 && !pooled)) return fail(n, VGG19_ERR_ARG, "null images, or neither output asked for");
  int rc = check_batch(n, batch, VGG19_MODE_FORWARD, 0);
  if (rc != VGG19_OK) return rc;
  if (n->cfg.dtype != VGG19_BF16) return fail(n, VGG19_ERR_ARG, "the fused first block exists for the bf16 configuration only");
  n->other_pass = true;
  Pass<bf16> ps{n, make_plan(n, batch, VGG19_MODE_FORWARD), static_cast<cudaStream_t>(stream)};
  if (!ps.first_block_fused_ok(batch))
    return fail(n, VGG19_ERR_SHAPE, "no fused first block at %dx%d (width a multiple of 14, height of 8)", n->cfg.height,
                n->cfg.width);
  ps.first_block_fused((const bf16 *)images, batch, (bf16 *)y2, (bf16 *)pooled);
  if (ps.err != cudaSuccess) return fail(n, VGG19_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(ps.err));
  return VGG19_OK;
}

int vgg19_conv_layer_backward_ex(vgg19_t *n, int32_t layer, const void *x, const void *dz, int32_t batch,
                                 float *dw, float *db, void *dx, const void *relu_mask, const uint8_t *pool_code,
                                 void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (layer < 1 || layer > kConvLayers || !dz || batch < 1 || (!dw != !db) || (dw && !x) || (!dw && !dx))
    return fail(n, VGG19_ERR_ARG, "bad layer (%d), batch (%d) or null tensor", layer, batch);
  if (dx && layer == 1) return fail(n, VGG19_ERR_ARG, "layer 1 has no input gradient");
  if (relu_mask && !dx) return fail(n, VGG19_ERR_ARG, "relu_mask without dx");
  if (pool_code && (!dx || relu_mask)) return fail(n, VGG19_ERR_ARG, "pool_code needs dx and excludes relu_mask");
  int rc = check_batch(n, batch, VGG19_MODE_BACKWARD, 0);
  if (rc != VGG19_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  n->other_pass = true;
  Plan p = make_plan(n, batch, VGG19_MODE_BACKWARD);
  cudaError_t e;
  if (n->cfg.dtype == VGG19_BF16) {
    Pass<bf16> ps{n, p, st};
    if (pool_code)
      ps.conv_backward(layer - 1, (const bf16 *)x, (const bf16 *)dz, batch, dw, db, ps.buf(p.dxlow), nullptr, pool_code, (bf16 *)dx);
    else
      ps.conv_backward(layer - 1, (const bf16 *)x, (const bf16 *)dz, batch, dw, db, (bf16 *)dx, (const bf16 *)relu_mask);
    e = ps.err;
  } else {
    Pass<float> ps{n, p, st};
    if (pool_code)
      ps.conv_backward(layer - 1, (const float *)x, (const float *)dz, batch, dw, db, ps.buf(p.dxlow), nullptr, pool_code, (float *)dx);
    else
      ps.conv_backward(layer - 1, (const float *)x, (const float *)dz, batch, dw, db, (float *)dx, (const float *)relu_mask);
    e = ps.err;
  }
  if (e != cudaSuccess) return fail(n, VGG19_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return VGG19_OK;
}

int vgg19_conv_layer_backward(vgg19_t *n, int32_t layer, const void *x, const void *dz,
                              int32_t batch, float *dw, float *db, void *dx, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (!x || !dw || !db) return fail(n, VGG19_ERR_ARG, "bad layer (%d), batch (%d) or null tensor", layer, batch);
  return vgg19_conv_layer_backward_ex(n, layer, x, dz, batch, dw, db, dx, nullptr, nullptr, stream);
}

int vgg19_dense_layer_forward(vgg19_t *n, int32_t layer, const void *x, int32_t batch, void *y, float *y_f32,
                              void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (layer < 1 || layer > kFcLayers || !x || (!y && !y_f32))
    return fail(n, VGG19_ERR_ARG, "bad dense layer (%d) or null tensor", layer);
  int rc = check_batch(n, batch, VGG19_MODE_FORWARD, 0);
  if (rc != VGG19_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  n->other_pass = true;
  Plan p = make_plan(n, batch, VGG19_MODE_FORWARD);
  cudaError_t e;
  if (n->cfg.dtype == VGG19_BF16) {
    Pass<bf16> ps{n, p, st};
    ps.dense_forward(n->fc[layer - 1], (const bf16 *)x, batch, (bf16 *)y, y_f32);
    e = ps.err;
  } else {
    Pass<float> ps{n, p, st};
    ps.dense_forward(n->fc[layer - 1], (const float *)x, batch, (float *)y, y_f32);
    e = ps.err;
  }
  if (e != cudaSuccess) return fail(n, VGG19_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return VGG19_OK;
}

int vgg19_dense_layer_backward(vgg19_t *n, int32_t layer, const void *x, const void *dy, int32_t batch, float *dw,
                               float *db, void *dx, const void *relu_mask, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  if (layer < 1 || layer > kFcLayers || !x || !dy || !dw || !db || (relu_mask && !dx))
    return fail(n, VGG19_ERR_ARG, "bad dense layer (%d) or null tensor", layer);
  int rc = check_batch(n, batch, VGG19_MODE_BACKWARD, 0);
  if (rc != VGG19_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  n->other_pass = true;
  Plan p = make_plan(n, batch, VGG19_MODE_BACKWARD);
  cudaError_t e;
  if (n->cfg.dtype == VGG19_BF16) {
    Pass<bf16> ps{n, p, st};
    ps.dense_backward(n->fc[layer - 1], (const bf16 *)x, (const bf16 *)dy, batch, dw, db,
                      dx ? (bf16 *)dx : ps.buf(p.dflat), (const bf16 *)relu_mask);
    e = ps.err;
  } else {
    Pass<float> ps{n, p, st};
    ps.dense_backward(n->fc[layer - 1], (const float *)x, (const float *)dy, batch, dw, db,
                      dx ? (float *)dx : ps.buf(p.dflat), (const float *)relu_mask);
    e = ps.err;
  }
  if (e != cudaSuccess) return fail(n, VGG19_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
  return VGG19_OK;
}

int vgg19_saved_tensor(const vgg19_t *n, int32_t batch, int32_t mode, int32_t index,
                       size_t *offset_bytes, int64_t dims[4]) {
  if (!n || !offset_bytes || !dims || batch < 1 || batch > n->cfg.batch_max || mode < 0 || mode > 2 ||
      index < 0 || index > 22)
    return VGG19_ERR_ARG;
  Plan p = make_plan(n, batch, mode);
  if (index < kConvLayers) {
    const ConvLayer &c = n->conv[index];
    *offset_bytes = p.act[index];
    dims[0] = batch; dims[1] = c.H; dims[2] = c.W; dims[3] = c.Cout;
  } else if (index < kConvLayers + 5) {
    int l = 0;
    while (n->pool_idx[l] != index - kConvLayers) ++l;
    const ConvLayer &c = n->conv[l];
    *offset_bytes = p.pooled[index - kConvLayers];
    dims[0] = batch; dims[1] = c.H / 2; dims[2] = c.W / 2; dims[3] = c.Cout;
  } else {
    *offset_bytes = index == 21 ? p.a1 : p.a2;
    dims[0] = batch; dims[1] = 4096; dims[2] = 1; dims[3] = 1;
  }
  return VGG19_OK;
}

int vgg19_sync_status(vgg19_t *n, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  CUDA_TRY(n, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  int code = 0;
  CUDA_TRY(n, cudaMemcpy(&code, n->dev_error, sizeof code, cudaMemcpyDeviceToHost));
  if (code != 0) {
    cudaMemset(n->dev_error, 0, 256);
    if (code == kDevBadLabel)
      return fail(n, VGG19_ERR_ARG, "a label outside [0, %d) reached the loss (its row's loss is NaN)", kClasses);
    if (code == kDevSplitRange)
      return fail(n, VGG19_ERR_RANGE, "an activation beyond fp16's range (65504) met the split-fp16 path");
    return fail(n, VGG19_ERR_DEVICE_TIMEOUT, "a device-side wait ran out (code %d)", code);
  }
  return VGG19_OK;
}

int vgg19_selftest_wait_timeout(vgg19_t *n, void *stream) {
  if (!n) return VGG19_ERR_ARG;
  // a millisecond or two of SM clock: long enough to be a real wait, short enough for a test
  CUDA_TRY(n, tc_wait_selftest(n->dev_error, 2000000ll, static_cast<cudaStream_t>(stream)));
  return VGG19_OK;
}

int vgg19_launch_count(const vgg19_t *n, int32_t mode, int32_t *n_kernels) {
  if (!n || !n_kernels || mode < 0 || mode > 2) return VGG19_ERR_ARG;
  *n_kernels = n->launches[mode];
  return VGG19_OK;
}

int vgg19_describe(const vgg19_t *n, char *out, size_t cap) {
  if (!n) return VGG19_ERR_ARG;
  std::string s;
  char line[256];
  snprintf(line, sizeof line, "vgg19 %dx%dx3 dtype=%s batch_max=%d params=%zu\n", n->cfg.height,
           n->cfg.width, n->cfg.dtype == VGG19_BF16 ? "bf16" : "fp32", n->cfg.batch_max, n->n_params);
  s += line;
  for (int l = 0; l < kConvLayers; ++l) {
    const ConvLayer &c = n->conv[l];
    ConvShape sh{n->cfg.batch_max, c.H, c.W, c.Cin, c.Cout};
    ConvShape sd{n->cfg.batch_max, c.H, c.W, c.Cout, c.Cin};
    // the kernel each pass picks for this layer, in the order the scheduler tries them
    const char *fwd = n->use_split ? (l == 0 ? "simt" : "tcgen05:im2col-split-fp16 (forward-only passes; else simt)")
                      : !n->use_tc ? "simt"
                      : l == 0 ? (tc_first_conv_supported(sh) ? "tcgen05:first-layer" : "simt")
                      : tc_conv3x3_rowshift_supported(sh) ? "tcgen05:row-shift"
                      : tc_conv3x3_halo_supported(sh) ? (n->use_pair && c.Cout == 128 ? "tcgen05:halo-pair" : "tcgen05:halo")
                      : n->use_pair && tc_conv3x3_pair_supported(sh) ? "tcgen05:pair"
                      : tc_conv3x3_supported(sh) ? "tcgen05:im2col" : "simt";
    const char *dgrad = l == 0 ? "none"
                        : !n->use_tc ? "simt"
                        : tc_conv3x3_rowshift_supported(sd) ? "tcgen05:row-shift"
                        : tc_conv3x3_halo_supported_unpooled(sd) ? (n->use_pair && c.Cin == 128 ? "tcgen05:halo-pair" : "tcgen05:halo")
                        : n->use_pair && tc_conv3x3_pair_supported(sd) ? "tcgen05:pair"
                        : tc_conv3x3_supported(sd) ? "tcgen05:im2col" : "simt";
    const char *wgrad = !n->use_tc ? "simt"
                        : l == 0 ? (tc_first_conv_supported(sh) ? "tcgen05:gemm-8ch" : "simt")
                        : tc_wgrad_patch_supported(sh) ? "tcgen05:patch"
                        : tc_wgrad_supported(sh) ? (n->use_pair && c.Cin % 128 == 0 && c.Cout % 256 == 0 ? "tcgen05:gemm-pair" : "tcgen05:gemm")
                        : "simt";
    snprintf(line, sizeof line, "conv%-2d %3dx%-3d %3d->%-3d +bias +relu%s  fwd=%s dgrad=%s wgrad=%s\n",
             l + 1, c.H, c.W, c.Cin, c.Cout, c.pool_after ? " +maxpool2x2" : "", fwd, dgrad, wgrad);
    s += line;
  }
  for (int i = 0; i < kFcLayers; ++i) {
    const FcLayer &f = n->fc[i];
    snprintf(line, sizeof line, "dense%d %5d->%-4d +bias%s%s\n", i + 1, f.In, f.Out, f.relu ? " +relu" : "",
             n->use_split ? "  fwd=tcgen05:gemm-split-fp16 (forward-only passes; else simt)" : "");
    s += line;
  }
  s += "softmax 1000\n";
  snprintf(line, sizeof line, "counts: convolution=16 reduce-window=5 dot=3 relu=18 softmax=1 rng=0\n");
  s += line;
  if (out && cap) {
    size_t k = s.size() < cap - 1 ? s.size() : cap - 1;
    memcpy(out, s.data(), k);
    out[k] = 0;
  }
  return (int)s.size();
}

const char *vgg19_last_error(const vgg19_t *n) { return n ? n->err.c_str() : g_create_error.c_str(); }

}  // extern "C"
