/*
 * vgg19_b200 - the VGG19 forward and backward pass as one device program for
 * NVIDIA B200 (sm_100a).
 *
 * The computation is the one the paper offloads as a single executable
 * (section 7.2 "VGG19 forward pass", section 7.3 "VGG19 backward pass"):
 * 16 convolutions 3x3 / pad 1 / stride 1 with bias and ReLU, five 2x2
 * max-pools, three dense layers (section 7.1, dense(W,x,b) = W*x .+ b),
 * softmax (section 7.1), and the gradient of a scalar loss with respect to
 * every parameter.  The loss is the mean cross-entropy of the softmax output
 * against integer labels.
 *
 * Conventions
 *  - Every function returns VGG19_OK (0) or a negative vgg19_status.  No C++
 *    exception crosses this boundary.  vgg19_last_error() gives text.
 *  - "device" pointers are CUDA device pointers of the current device, owned
 *    by the caller, and must stay valid until the work enqueued on the stream
 *    has finished.  "host" pointers are ordinary host memory.
 *  - Work is enqueued on the given cudaStream_t (passed as void*; NULL = the
 *    legacy default stream) and returns without waiting for it.
 *  - Layouts: images and activations are NHWC (channel fastest); a conv weight
 *    is [Cout][3][3][Cin]; a dense weight is [out][in] with `in` enumerating
 *    the flattened (h, w, c) activation, c fastest; a bias is [out].
 *  - The flat parameter / gradient buffer holds, for layer 1..19 in network
 *    order, the weight then the bias, as fp32.
 */
#ifndef VGG19_B200_H_
#define VGG19_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vgg19 vgg19_t;

typedef enum {
  VGG19_OK = 0,
  VGG19_ERR_ARG = -1,             /* null pointer, bad enum, batch out of range */
  VGG19_ERR_SHAPE = -2,           /* height/width not a positive multiple of 32 */
  VGG19_ERR_WORKSPACE = -3,       /* no workspace bound, or too small */
  VGG19_ERR_CUDA = -4,            /* a CUDA runtime/driver call failed */
  VGG19_ERR_DEVICE_TIMEOUT = -5,  /* a bounded device-side wait ran out */
  VGG19_ERR_UNSUPPORTED_ARCH = -6,/* the device is not compute capability 10.x */
  VGG19_ERR_RANGE = -7            /* VGG19_FLAG_SPLIT_F16: an activation beyond fp16's range (reported by vgg19_sync_status) */
} vgg19_status;

typedef enum {
  VGG19_FP32 = 0, /* fp32 storage and fp32 FMA arithmetic throughout */
  VGG19_BF16 = 1  /* bf16 activations/weights, fp32 accumulation, fp32 gradients */
} vgg19_dtype;

enum {
  VGG19_FLAG_NO_GRAPH = 1,        /* enqueue kernels directly instead of replaying a CUDA graph */
  VGG19_FLAG_NO_TENSOR_CORES = 2, /* bf16 only: use the CUDA-core kernels for every layer */
  VGG19_FLAG_NO_CTA_PAIRS = 4,    /* one CTA per tile everywhere: no two-CTA (cta_group::2) kernels */
  VGG19_FLAG_FIRST_FUSION = 8,    /* forward-only passes run conv1_1 and conv1_2 as one kernel (vgg19_first_block_forward) */
  /* fp32 only: forward-only passes (vgg19_forward*, vgg19_conv_layer_forward*) run layers 2..16 and the dense
   * layers on tensor cores, every fp32 value carried as two fp16 terms (hi = fp16(v), lo = fp16(v - hi)) and
   * every product formed as hi*hi + hi*lo + lo*hi in an fp32 accumulator: 22 of fp32's 24 mantissa bits per
   * operand (an absolute 3e-8 for activations below 0.25).  Activations must stay within fp16's range (65504): one beyond it makes vgg19_sync_status
   * return VGG19_ERR_RANGE.  Backward and training passes keep the CUDA-core kernels.  The paper runs its
   * fp32 network (section 7.2) on CPU and GPU back ends and has no counterpart of this. */
  VGG19_FLAG_SPLIT_F16 = 16
};

typedef enum {
  VGG19_MODE_FORWARD = 0,  /* vgg19_forward */
  VGG19_MODE_BACKWARD = 1, /* vgg19_backward */
  VGG19_MODE_TRAIN = 2     /* vgg19_train_step(s): the backward workspace plus a gradient buffer */
} vgg19_mode;

typedef struct {
  int32_t height;    /* input height, multiple of 32 */
  int32_t width;     /* input width, multiple of 32 */
  int32_t batch_max; /* largest batch any later call will use */
  int32_t dtype;     /* vgg19_dtype */
  uint32_t flags;    /* VGG19_FLAG_* */
} vgg19_config;

/* Build a network whose parameters are the seeded He-normal set (weights
 * N(0, 2/fan_in), biases 0) drawn on the host from `seed` and uploaded.  The
 * library owns the parameters.  (The paper itself used trained weights,
 * section 7.2; a seeded random set stands in for them.) */
int vgg19_create(const vgg19_config *cfg, uint64_t seed, vgg19_t **out);

/* Same, from a caller-supplied flat fp32 HOST buffer of vgg19_param_count()
 * elements in the order given above.  The buffer is copied. */
int vgg19_create_from_params(const vgg19_config *cfg, const float *host_params, vgg19_t **out);

/* Frees everything the library allocated (parameters, graphs).  Never frees
 * the workspace.  NULL is allowed. */
void vgg19_destroy(vgg19_t *net);

/* Number of parameter tensors (38) and of fp32 elements in the flat buffer. */
int vgg19_param_count(const vgg19_t *net, int32_t *n_tensors, size_t *n_elems);

/* Tensor i (0..37): element offset in the flat buffer, rank and dims
 * ([Cout,3,3,Cin], [out,in] or [out]). */
int vgg19_param_info(const vgg19_t *net, int32_t i, size_t *offset, int32_t *rank, int64_t dims[4]);

/* Copy the fp32 master parameters to / from a HOST buffer (synchronous). */
int vgg19_get_params(const vgg19_t *net, float *host_params);
int vgg19_set_params(vgg19_t *net, const float *host_params);

/* Bytes of device scratch a call in `mode` at `batch` needs (saved
 * activations, gradients in flight, split-K partials).  0 on bad arguments. */
size_t vgg19_workspace_bytes(const vgg19_t *net, int32_t batch, int32_t mode);

/* Hand the library a DEVICE buffer (256-byte aligned) to use as scratch.  The
 * caller keeps ownership and must keep it alive while calls are in flight. */
int vgg19_bind_workspace(vgg19_t *net, void *device_workspace, size_t bytes);

/* Forward pass (section 7.2).  images: device, [batch][H][W][3], fp32 or bf16
 * per the config, already normalised.  logits: device fp32 [batch][1000], the
 * input of the softmax.  probs: device fp32 [batch][1000] = softmax(logits)
 * (section 7.1), or NULL to skip it.  The first call for a given (batch,
 * pointers) records the whole pass into one CUDA graph; later calls replay
 * it - the counterpart of the paper's single offloaded executable. */
int vgg19_forward(vgg19_t *net, const void *images, int32_t batch, float *logits, float *probs,
                  void *stream);

/* Forward + loss + backward (section 7.3) as one graph.  labels: device int32
 * [batch] in [0,1000).  grads: device fp32, vgg19_param_count() elements,
 * fully overwritten with d(loss)/d(parameter), loss = mean cross-entropy.
 * loss: device fp32 scalar or NULL.  logits: device fp32 [batch][1000] or
 * NULL.  batch: number of images in this call, at most the config's batch_max. */
int vgg19_backward(vgg19_t *net, const void *images, const int32_t *labels, int32_t batch,
                   float *grads, float *loss, float *logits, void *stream);

/* One step of plain gradient descent, parameter <- parameter - lr * gradient, on the
 * fp32 master copy, with the bf16 copy and every filter copy the kernels read
 * (rotated, tap-major, padded) rebuilt on the same stream.  The paper fuses "the
 * training loop" with the two passes into one executable (introduction and
 * conclusion) without naming the optimiser; plain SGD is the reading taken.
 * grads: device fp32, vgg19_param_count() elements, in parameter order (what
 * vgg19_backward wrote).  Asynchronous on `stream`; passes enqueued later on the
 * same stream see the new parameters.  Graphs recorded earlier stay valid. */
int vgg19_sgd_step(vgg19_t *net, const float *grads, float lr, void *stream);

/* The training step as ONE device program: forward + loss + backward on a
 * batch and the gradient-descent update of every parameter (fp32 master, bf16
 * copy, the rotated / tap-major / padded filter copies), recorded as a single
 * CUDA graph - the paper's claim for its own system is that the forward pass,
 * the backward pass and the training loop fuse into one executable
 * (introduction and conclusion).  The gradient never leaves the workspace,
 * which must hold vgg19_workspace_bytes(net, batch, VGG19_MODE_TRAIN).
 * images / labels: device, as for vgg19_backward.  loss: device fp32 scalar
 * (the loss BEFORE the update) or NULL.  lr may change from call to call
 * without a new recording (the update kernels read it from device memory).
 * For one GPU only: with several, the gradients must be averaged between the
 * two halves - use vgg19_backward, the exchange, vgg19_sgd_step. */
int vgg19_train_step(vgg19_t *net, const void *images, const int32_t *labels, int32_t batch, float lr,
                     float *loss, void *stream);

/* `steps` (1..64) training steps on `steps` resident batches as one graph:
 * images [steps][batch][H][W][3], labels [steps][batch], losses (or NULL)
 * device fp32 [steps]; step k trains on batch k with the parameters step k-1
 * left.  The counterpart of compiling the training LOOP, not just its body. */
int vgg19_train_steps(vgg19_t *net, const void *images, const int32_t *labels, int32_t batch, int32_t steps,
                      float lr, float *losses, void *stream);

/* Overlap point for data-parallel training.  In the flat gradient buffer the
 * three dense layers come last (from the offset vgg19_param_info(net, 32)
 * reports; 123.6 M of the 143.7 M elements at 224x224) and the backward pass
 * finishes them first, before any convolution layer's gradient.  With an
 * event set here (a cudaEvent_t the caller owns; NULL clears it), every later
 * vgg19_backward records it on its stream at that point - inside the recorded
 * graph too - so that a caller can start the all-reduce of the dense
 * gradients on another stream (cudaStreamWaitEvent) while the convolution
 * layers' backward pass, most of the pass's time, still runs, and exchange the
 * convolution gradients when the pass ends.  The paper lists distributed
 * primitives as future work (section 8); the exchange itself stays with the
 * caller.  Setting or clearing the event discards recorded graphs. */
int vgg19_set_dense_grads_event(vgg19_t *net, void *cuda_event);

/* HOST-buffer convenience wrappers: copy images (and labels) to the device,
 * run the pass, copy the results back and wait for the stream.  The bound
 * workspace must hold vgg19_workspace_bytes(net, batch, mode) +
 * vgg19_io_bytes(net, batch, mode) bytes; the staging area is its tail.
 * Host buffers should be page-locked for full copy bandwidth.  Any result
 * pointer may be NULL to skip that copy. */
size_t vgg19_io_bytes(const vgg19_t *net, int32_t batch, int32_t mode);
int vgg19_forward_host(vgg19_t *net, const void *host_images, int32_t batch, float *host_logits,
                       float *host_probs, void *stream);
int vgg19_backward_host(vgg19_t *net, const void *host_images, const int32_t *host_labels,
                        int32_t batch, float *host_grads, float *host_loss, void *stream);

/* vgg19_forward_host without the wait: the upload runs on a stream of the
 * library's own into one of two staging slots (taken in turn), the pass and the
 * download of its results are enqueued on `stream`, and the call returns.  A
 * caller that enqueues batch after batch gets the upload of the next batch
 * overlapped with the pass of the current one - how a serving loop would feed
 * the executable of section 7.2.  host_images must stay untouched, and the
 * results are not in host_logits / host_probs, until `stream` has been waited
 * for (vgg19_sync_status); with more than two calls in flight the library orders
 * the reuse of a slot itself; a call whose batch differs from the previous
 * call's, or that follows a pass made through another entry point, uploads
 * only after the work already enqueued on `stream` (the staging slots move
 * with the batch).  Keep all calls in flight on one handle on one stream.
 * stream must not be the legacy default stream.
 * Needs the same workspace as vgg19_forward_host (vgg19_io_bytes counts both slots). */
int vgg19_forward_host_async(vgg19_t *net, const void *host_images, int32_t batch, float *host_logits,
                             float *host_probs, void *stream);

/* Single convolution layer (3x3, pad 1, stride 1) + bias + ReLU, optionally
 * followed by the 2x2 max-pool, on caller-supplied device tensors in the
 * config's dtype; the per-layer building block of section 7.2, exposed for
 * per-layer parity and timing.  layer in 1..16 selects shape and weights;
 * x: [batch][h][w][Cin]; y: [batch][h][w][Cout]; pooled (or NULL):
 * [batch][h/2][w/2][Cout].  On a network created with VGG19_FLAG_SPLIT_F16
 * layers 2..16 run on the split-fp16 tensor-core kernel: x, y and pooled are
 * fp32 as always (y and pooled also serve as scratch for their two-term
 * forms), and the forward workspace must be bound (VGG19_ERR_WORKSPACE). */
int vgg19_conv_layer_forward(vgg19_t *net, int32_t layer, const void *x, int32_t batch,
                             void *y, void *pooled, void *stream);

/* The same, also recording what the backward pass needs to know about the
 * max-pool (the appendix table's `select-and-scatter`): pool_code (with pooled;
 * or NULL), device uint8 [batch][h/2][w/2][Cout], receives for every window
 * where its maximum sits - 0..3 for (0,0), (0,1), (1,0), (1,1), the first one
 * on ties - or 4 when that maximum is not positive, i.e. when the ReLU before
 * the pool passes no gradient to the window.  y may be NULL (with pooled, and
 * without pool_code) where the layer's kernel pools in its own epilogue, as a
 * forward-only pass runs the block-ending layers: the full-resolution output
 * is then never written; VGG19_ERR_ARG where it cannot. */
int vgg19_conv_layer_forward_ex(vgg19_t *net, int32_t layer, const void *x, int32_t batch, void *y, void *pooled,
                                uint8_t *pool_code, void *stream);

/* The first block, conv1_1 -> conv1_2 (-> max-pool), as ONE kernel that never
 * writes conv1_1's activation (the paper's point about the forward pass is
 * that the whole of it fuses into one executable, section 7.2; here the two
 * layers whose intermediate is the largest tensor of the network share a
 * kernel: the second layer's input patches are computed on the fly from image
 * patches).  Same result, bit for bit, as the two layers run one after the
 * other.  A forward-only pass runs layers 1 and 2 this way when the network
 * was created with VGG19_FLAG_FIRST_FUSION (off by default: on a B200 at batch
 * 100 the one kernel takes 0.55 ms, the two it replaces 0.51 ms).  bf16 only,
 * width a multiple of 14, height of 8; else VGG19_ERR_SHAPE.  images: device
 * [batch][H][W][3] bf16; y2 (or NULL): conv1_2's output [batch][H][W][64];
 * pooled (or NULL): its 2x2 max-pool.  Needs the forward workspace. */
int vgg19_first_block_forward(vgg19_t *net, const void *images, int32_t batch, void *y2, void *pooled, void *stream);

/* Gradients of that layer given dz = d(loss)/d(pre-activation) already
 * masked by the ReLU: dw fp32 [Cout][3][3][Cin], db fp32 [Cout], and (unless
 * NULL) dx in the config's dtype [batch][h][w][Cin] (section 7.3). */
int vgg19_conv_layer_backward(vgg19_t *net, int32_t layer, const void *x, const void *dz,
                              int32_t batch, float *dw, float *db, void *dx, void *stream);

/* The same with the two halves separable and the ReLU of the layer below
 * folded in, as the whole pass runs them (section 7.3: the `select`s that
 * follow each input-gradient convolution).  dw and db may both be NULL (input
 * gradient only; x is then unused and may be NULL), or dx may be NULL (filter
 * and bias gradient only).  relu_mask (or NULL): [batch][h][w][Cin] in the
 * config's dtype, the stored output of the layer below; dx is set to zero
 * wherever relu_mask is not positive.  pool_code (or NULL; excludes
 * relu_mask): for a layer whose input is a pooled tensor, the codes
 * vgg19_conv_layer_forward_ex recorded for that pool, [batch][h][w][Cin]; dx
 * is then the gradient at the output of the layer BELOW the pool,
 * [batch][2h][2w][Cin]: every value of the input gradient goes to the window
 * position its code names (nowhere for code 4), zeros elsewhere - pool scatter
 * and ReLU mask in one, done in the input-gradient kernel's epilogue where the
 * layer's shape allows. */
int vgg19_conv_layer_backward_ex(vgg19_t *net, int32_t layer, const void *x, const void *dz, int32_t batch,
                                 float *dw, float *db, void *dx, const void *relu_mask, const uint8_t *pool_code,
                                 void *stream);

/* Where a pass at `batch` in `mode` leaves the activations it stores, as a
 * byte offset into the bound workspace, so that a caller can inspect the
 * forward state a backward pass differentiated (the ReLU masks and pool
 * arg-maxima of section 7.3 are decided on exactly these stored values).
 * index 0..15: output of conv layer index+1 after bias and ReLU,
 * [batch][h][w][Cout]; 16..20: outputs of the five max-pools; 21, 22: outputs
 * of dense layers 1 and 2 after ReLU, [batch][4096] (dims[2] = dims[3] = 1).
 * Element type is the config's dtype.  A forward-only pass does not write the
 * pre-pool output of a layer whose max-pool is fused into the convolution
 * (layers 2 and 4 at 224x224); a backward pass stores everything. */
/* Single dense layer (section 7.2's last three layers; the appendix table's `dot` rows), exposed like the
 * convolution layers for per-layer parity and timing.  layer in 1..3.  x: device [batch][In] in the config's
 * dtype (for layer 1 the flattened last pooling output, [batch][h][w][512] order).  y (or NULL): device
 * [batch][Out] in the config's dtype; y_f32 (or NULL): the same values as fp32 (how layer 3's logits leave); at
 * least one.  Bias added; ReLU applied for layers 1 and 2.  Needs the forward workspace. */
int vgg19_dense_layer_forward(vgg19_t *net, int32_t layer, const void *x, int32_t batch, void *y, float *y_f32,
                              void *stream);

/* Backward of one dense layer: dw fp32 [Out][In] and db fp32 [Out] from (x, dy); dx (or NULL) device
 * [batch][In] in the config's dtype = dy W, multiplied by (relu_mask > 0) when relu_mask (the layer's input,
 * itself a ReLU output; or NULL) is given.  dy: device [batch][Out] in the config's dtype, the gradient at the
 * layer's pre-activation.  Needs the backward workspace. */
int vgg19_dense_layer_backward(vgg19_t *net, int32_t layer, const void *x, const void *dy, int32_t batch, float *dw,
                               float *db, void *dx, const void *relu_mask, void *stream);

int vgg19_saved_tensor(const vgg19_t *net, int32_t batch, int32_t mode, int32_t index,
                       size_t *offset_bytes, int64_t dims[4]);

/* Filter and bias gradient of one 3x3 / pad 1 / stride 1 convolution without
 * any allocation.  (The paper has no counterpart: this entry point exists for
 * the library's users, not for the method.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained -
 * a plugin or callback invoked inside someone else's framework after that
 * framework has claimed the whole GPU for its own pool, or a process whose
 * memory budget was fixed at start-up - cannot create a network handle or
 * provide a workspace, because both need cudaMalloc.  This function needs
 * neither: it takes no handle, and the split-K scratch its kernel uses is a
 * fixed array of VGG19_STATIC_SCRATCH_BYTES compiled into the library (every
 * GPU on which the library's code is loaded carries that array until the
 * process exits; see below for when that happens).  It
 * calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   x  : device, [batch][height][width][cin]   layer input
 *   dz : device, [batch][height][width][cout]  gradient at the pre-activation
 *   dtype : VGG19_FP32 or VGG19_BF16, the element type of x and dz
 *   dw : device fp32 [cout][3][3][cin], db : device fp32 [cout]; overwritten
 *   needed_bytes : if not NULL, receives the scratch this shape needs
 * Same arithmetic as the CUDA-core path of vgg19_conv_layer_backward.
 *
 * Returns VGG19_ERR_WORKSPACE, and launches nothing, when the shape needs more
 * scratch than VGG19_STATIC_SCRATCH_BYTES (*needed_bytes says how much);
 * VGG19_ERR_ARG for null pointers or non-positive sizes.
 *
 * The first call on each device looks up the array's device address (that
 * device must be current); make that first call outside any stream capture.
 * With CUDA's default lazy module loading that first call is also when the
 * driver places the array, and the kernels' code, on the device: a process
 * that is about to hand the GPU's memory to someone else should make one call
 * per device at start-up, before the memory is claimed (or run with
 * CUDA_MODULE_LOADING=EAGER, which places everything when the library loads);
 * from the second call on, free device memory is unchanged by a call.  If the
 * lookup fails (for instance because the device is already full) the call and
 * every later one on that device return VGG19_ERR_CUDA.
 * All calls share the one array and it keeps whatever the last call left in
 * it; the kernels never rely on its previous contents.  Two calls that overlap
 * on the GPU (different streams) race on it: keep calls on one stream, or
 * order them with events. */
#define VGG19_STATIC_SCRATCH_BYTES (8u << 20)
int vgg19_conv_wgrad_static(const void *x, const void *dz, int32_t batch, int32_t height, int32_t width,
                            int32_t cin, int32_t cout, int32_t dtype, float *dw, float *db,
                            size_t *needed_bytes, void *stream);

/* Wait for the stream and report any device-side error recorded so far:
 * VGG19_ERR_DEVICE_TIMEOUT when a bounded wait inside a kernel ran out,
 * VGG19_ERR_ARG when a label outside [0,1000) reached the loss (the label is
 * never used as an index; that pass's loss is NaN).  The record is cleared,
 * and the handle stays usable. */
int vgg19_sync_status(vgg19_t *net, void *stream);

/* Diagnostic for the error path above.  Every wait inside the kernels (on a
 * copy, on the tensor cores, on a free buffer) is bounded; when one runs out
 * the kernel records a code, lets what it has in flight finish and returns.
 * This call enqueues one tiny kernel whose wait is certain to run out - a
 * barrier in shared memory on which nothing arrives, limit about a millisecond,
 * no copy engine or tensor memory involved - so that a caller (or a test) can
 * see the whole chain: the next vgg19_sync_status returns
 * VGG19_ERR_DEVICE_TIMEOUT, and passes enqueued afterwards run normally. */
int vgg19_selftest_wait_timeout(vgg19_t *net, void *stream);

/* Number of kernel launches (graph nodes) one forward / backward call makes. */
int vgg19_launch_count(const vgg19_t *net, int32_t mode, int32_t *n_kernels);

/* Human-readable layer table and kernel list (the counterpart of the paper's
 * @code_xla introspection macro, section 7.1).  Writes at most n bytes,
 * NUL-terminated; returns the length needed. */
int vgg19_describe(const vgg19_t *net, char *buf, size_t n);

/* Text of the last error on this handle (or of the last failed create when
 * net is NULL).  Never NULL. */
const char *vgg19_last_error(const vgg19_t *net);

#ifdef __cplusplus
}
#endif
#endif /* VGG19_B200_H_ */
