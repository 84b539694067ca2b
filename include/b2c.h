/*
 * b2c -- C ABI of the B200 (sm_100a) CNN training-step library.
 *
 * The library executes the per-replica training step of the paper's Algorithm 1 (inner loop:
 * forward pass, loss, backward pass, gradient synchronisation = mean over the data-parallel
 * replicas / micro-batches, parameter update) for CIFAR-shaped convolutional networks.
 *
 * General rules for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned, and must
 *     stay valid until the stream has passed the call.  Descriptor structs are HOST memory and
 *     are read before the call returns.  The library allocates no device memory in any call
 *     except b2c_create (one status word); b2c_net_create builds host-side tables only.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work and return.
 *   - Layouts: activations NHWC bf16; convolution weights KRSC bf16 (K output channels, R x S
 *     taps, C input channels); accumulation is always fp32; fp32 -> bf16 is round-to-nearest-even.
 *   - Errors found on the host return a status and enqueue nothing.  Errors found on the device
 *     (an mbarrier wait that ran out of its spin budget, a label outside [0, classes)) set a
 *     sticky word that b2c_get_device_status reads; the kernel in question still terminates and
 *     all writes stay inside the caller's buffers, but its results are unspecified.
 *   - One b2c_ctx per host thread.  Devices other than compute capability 10.x: B2C_ERR_ARCH.
 *   - Environment switches, read by b2c_create (kernel variants) and b2c_net_create (step plan); all default to the
 *     fastest measured setting and exist for A/B measurements:
 *       B2C_PDL=0            launch kernels without programmatic stream serialization
 *       B2C_CTA_PAIRS=0|1|2|3  CTA pairs in the forward / data-gradient kernel: never | 3x3 stride-1 layers with tiles of 128 or
 *                            256 channels (default) | wherever possible | 128-channel tiles only
 *       B2C_FULL_HALO=0      one load per tap group instead of one framed tile per channel block (3x3 stride-1 layers)
 *       B2C_HMERGE=0         3x3 stride-1 layers with 64 output channels: one MMA per tap (N = 64) instead of the three horizontal taps
 *                            merged into N = 192 MMAs whose column blocks the epilogue shifts and adds
 *       B2C_GROUP_KBLOCKS=0  forward / data gradient of stride-2 and 1x1 layers: one k-block per ring slot instead of two sharing a slot,
 *                            a barrier wait and a commit; weight gradient of layers with few MMAs per 64-pixel chunk: one chunk per slot
 *                            instead of two
 *       B2C_ISSUE_SPLIT=0    forward / data gradient, tiles wider than 128 channels: one MMA-issuing thread instead of two sharing every unit
 *       B2C_WGRAD_FRAME=0    weight gradient: one x box per horizontal shift instead of one framed box per channel block
 *       B2C_WGRAD_ISSUERS=1  weight gradient: one MMA-issuing thread instead of two on alternate chunks of one accumulator
 *       B2C_BN_GROUPED=1     b2c_train_step runs the BatchNorm backward as one cooperative launch per layer, group by group
 *                            (b2c_bn_relu_bwd_groups); off by default: measured slower inside the step
 *       B2C_FUSE_WIDE=0|1    BatchNorm statistics of tiles wider than 64 channels: never | always in the convolution epilogue
 *                            (default: where the unit's MMAs take longer than the epilogue's column sums)
 *       B2C_FUSE_BN_STATS=0  BatchNorm statistics by a separate pass instead of the convolution epilogue (b2c_train_step)
 *       B2C_CHUNK_MB=<n>     b2c_train_step takes layers whose tensors exceed n MB a few micro-batches at a time (0 = off, default)
 */
#ifndef B2C_H_
#define B2C_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    B2C_OK = 0,
    B2C_ERR_INVALID_ARG = 1,
    B2C_ERR_UNSUPPORTED_SHAPE = 2,
    B2C_ERR_MISALIGNED = 3,
    B2C_ERR_WORKSPACE_TOO_SMALL = 4,
    B2C_ERR_CUDA = 5,
    B2C_ERR_ARCH = 6,
    B2C_ERR_DEVICE_TIMEOUT = 7,
    B2C_ERR_BAD_LABEL = 8
} b2c_status;

/* Convolution geometry.  Input n x h x w x c, filter k x r x s x c, r == s in {1,3},
 * stride in {1,2}, pad = (r-1)/2.  Output p = (h + 2 pad - r)/stride + 1, q likewise.
 * Supported: c and k multiples of 16; p and q powers of two <= 128; h = p*stride, w = q*stride.
 * (Narrower tensors are zero-extended first: b2c_pad_channels for activations, zero filter rows.) */
typedef struct {
    int n, h, w, c, k, r, s, stride, pad;
} b2c_conv_desc;

typedef struct b2c_ctx b2c_ctx;
typedef struct b2c_net b2c_net;

/* Context: device handle, driver entry points, the sticky device status word. */
b2c_status b2c_create(b2c_ctx** out, int device);
void b2c_destroy(b2c_ctx* ctx);
const char* b2c_status_string(b2c_status s);
/* Synchronises `stream`, returns and clears the sticky device status (B2C_OK if none). */
b2c_status b2c_get_device_status(b2c_ctx* ctx, void* stream);
/* Spin budget of every device-side wait (iterations of mbarrier.try_wait); default 1<<22.
 * A wait that exhausts it records B2C_ERR_DEVICE_TIMEOUT and the kernel winds down. */
void b2c_set_spin_limit(b2c_ctx* ctx, unsigned limit);

/* Pipeline diagnostics of the convolution kernels.  `counters` is a DEVICE array of 8 unsigned 64-bit words owned
 * by the caller (NULL switches the feature off, the default).  Every CTA of the forward / data-gradient kernel adds
 * the SM clock cycles its roles spent waiting: [0] TMA producer for a free ring stage, [1] MMA thread for a loaded
 * stage, [2] MMA thread for a free accumulator, [3] first epilogue warp for a finished accumulator, [4] CTA lifetime.
 * The weight-gradient kernel adds [0] first producer waiting, [1] first MMA thread waiting, [4] that thread's lifetime,
 * [5] time at which warp 2 finished its reductions, [6] cycles the first MMA thread spent issuing, and keeps in [7] the
 * MAXIMUM over CTAs and warps of the finishing time (zero the array between launches that should not mix). */
void b2c_set_stall_counters(b2c_ctx* ctx, unsigned long long* counters);

/* ---- Forward pass (Algorithm 1, "Perform forward pass") -------------------------------- */

/* Bytes of caller-owned scratch one convolution call needs (which: 0 forward, 1 data gradient, 2 weight gradient).
 * Always 0: the three convolution entry points stage their operands in shared memory and accumulate in TMEM, and the
 * weight gradient adds its partial sums straight into dw.  Kept so that callers can size buffers uniformly. */
size_t b2c_conv2d_workspace_bytes(const b2c_conv_desc* d, int which);

/* y[n,p,q,k] = sum_{r,s,c} x[n, p*stride+r-pad, q*stride+s-pad, c] * w[k,r,s,c]  (+ bias[k]),
 * x zero outside the image (cross-correlation, no kernel flip).  Implicit GEMM on tcgen05:
 * M = n*p*q, N = k, K = r*s*c.
 *   x        bf16 [n,h,w,c]          w_krsc  bf16 [k,r,s,c]
 *   y        bf16 [n,p,q,k], or fp32 [n,p,q,k] when y_is_f32 != 0
 *   bias     fp32 [k] or NULL
 *   ch_stats fp64 [2*k] or NULL: the kernel ADDS per-channel sum and sum of squares of the
 *            values it stored (after bf16 rounding) into ch_stats[0..k) and ch_stats[k..2k);
 *            the caller zeroes it.  Feeds b2c_bn_relu_fwd. */
b2c_status b2c_conv2d_fwd(b2c_ctx* ctx, const b2c_conv_desc* d, const void* x, const void* w_krsc, void* y,
                          int y_is_f32, const float* bias, double* ch_stats, void* stream);

/* z = gamma*(y-mean)*invstd + beta (+ residual); a = relu ? max(z,0) : z, per channel over
 * m = n*h*w positions; mean = sum(y)/m, var = sum(y^2)/m - mean^2 (biased), invstd = (var+eps)^-1/2.
 *   y bf16 [n,h,w,c]; residual bf16 [n,h,w,c] or NULL; a bf16 [n,h,w,c]; gamma, beta fp32 [c]
 *   ch_stats fp64 [2*c]: if stats_ready != 0 it already holds sum / sum of squares of y (from
 *            b2c_conv2d_fwd); otherwise the call zeroes it and computes them (scratch owned by caller)
 *   save_mean, save_invstd fp32 [c] (outputs, used by the backward pass)
 *   run_mean, run_var fp32 [c] or NULL: running statistics, updated with `momentum` and the
 *            unbiased variance.   c must be a multiple of 8.
 *   relu_mask  NULL, or n*h*w*c/8 bytes (output, only written when relu != 0): bit i of byte j is "a[8j+i] > 0".
 *            b2c_bn_relu_bwd can read it in place of a (1/16 of the bytes). */
b2c_status b2c_bn_relu_fwd(b2c_ctx* ctx, int n, int h, int w, int c, const void* y, double* ch_stats, int stats_ready,
                           const float* gamma, const float* beta, const void* residual, int relu, float eps, void* a,
                           float* save_mean, float* save_invstd, float* run_mean, float* run_var, float momentum,
                           void* relu_mask, void* stream);

/* Global average pool: pooled[n,c] = mean over h*w of a[n,:,:,c]; bf16 in, bf16 out; c % 8 == 0. */
b2c_status b2c_avgpool_fwd(b2c_ctx* ctx, int n, int hw, int c, const void* a, void* pooled, void* stream);
/* da[n,i,c] = dpooled[n,c] / hw for every position i; bf16 in, bf16 out. */
b2c_status b2c_avgpool_bwd(b2c_ctx* ctx, int n, int hw, int c, const void* dpooled, void* da, void* stream);

/* Zero-extends the channel dimension: y[m, 0..c_in) = x[m, :], y[m, c_in..c_out) = 0; bf16.
 * Used for the 3-channel image batch (TMA rows must be multiples of 16 bytes). c_out % 8 == 0. */
b2c_status b2c_pad_channels(b2c_ctx* ctx, long m, int c_in, int c_out, const void* x, void* y, void* stream);

/* Patch matrix of a 3x3, stride 1, pad 1 convolution: y[m, (r*3+s)*c_in + ch] = x[n, h+r-1, w+s-1, ch] (zero outside the
 * image) for every pixel m = (n,h,w); columns 9*c_in .. c_out-1 are zero.  bf16 in, bf16 out; c_in <= 3, c_out >= 32, c_out % 8 == 0.
 * With it the first convolution of a network (3 input channels) is the 1x1 convolution of the patch matrix with the
 * filter bank viewed as [k][9*c_in] rows padded to c_out. */
b2c_status b2c_im2col_3x3(b2c_ctx* ctx, int n, int h, int w, int c_in, int c_out, const void* x, void* y, void* stream);

/* ---- Loss (Algorithm 1, "Compute loss") ------------------------------------------------- */

/* Softmax cross-entropy over rows of logits fp32 [n, logits_pitch] (first `classes` columns used,
 * logits_pitch >= classes) with labels int32 [n]:
 *   *loss   += loss_scale * sum_i (logsumexp(z_i) - z_i[label_i])        (fp32 device scalar, caller zeroes)
 *   dlogits  = (softmax(z_i) - onehot(label_i)) * grad_scale, bf16 [n, pitch], columns >= classes zero.
 * pitch >= classes, pitch % 8 == 0.  A label outside [0,classes) records B2C_ERR_BAD_LABEL and
 * contributes nothing. */
b2c_status b2c_softmax_xent_fwd_bwd(b2c_ctx* ctx, int n, int classes, const float* logits, int logits_pitch,
                                    const int32_t* labels, float loss_scale, float grad_scale, float* loss,
                                    void* dlogits, int pitch, void* stream);

/* ---- Backward pass (Algorithm 1, "Perform backward pass") -------------------------------- */

/* Bytes of scratch b2c_bn_relu_bwd needs for c channels. */
size_t b2c_bn_relu_bwd_workspace_bytes(int c);

/* Backward of b2c_bn_relu_fwd.  dz = (da1 + da2) * [a > 0] (mask only if relu; ReLU'(0) = 0);
 * dbeta = sum dz; dgamma = sum dz*xhat, xhat = (y-mean)*invstd;
 * dy = gamma*invstd*(dz - dbeta/m - xhat*dgamma/m);  dres = dz.
 *   da1 bf16; da2 bf16 or NULL; y, a bf16 (forward input / output); dy bf16; dres bf16 or NULL
 *   relu_mask  NULL, or the bit mask b2c_bn_relu_fwd wrote: then a is not read and may be NULL
 *   dgamma, dbeta fp32 [c]: overwritten if acc == 0, accumulated into if acc != 0
 *   ws: scratch of b2c_bn_relu_bwd_workspace_bytes(c) bytes; the call zeroes it itself. */
b2c_status b2c_bn_relu_bwd(b2c_ctx* ctx, int n, int h, int w, int c, const void* da1, const void* da2, const void* y,
                           const void* a, const float* gamma, const float* save_mean, const float* save_invstd,
                           int relu, void* dy, void* dres, float* dgamma, float* dbeta, int acc,
                           const void* relu_mask, void* ws, size_t ws_bytes, void* stream);

/* The same backward for several statistics groups side by side (replica-local BatchNorm of data parallelism: each
 * replica, or micro-batch, normalises over its own images; Section III-A, data parallelism): the tensors hold `groups`
 * runs of rows_per_group rows of c channels back to back, save_mean / save_invstd are fp32 [groups][c], and every
 * group is differentiated with its own statistics.  dgamma / dbeta receive the sum over the groups (overwritten if
 * acc == 0, accumulated into otherwise).  Both passes run in one cooperative launch, group by group: the reduction of
 * a group, a grid-wide barrier, then the apply pass of that group while its tensors are still in L2 (about 6 bytes
 * of DRAM traffic per element instead of 10).  Requires relu_mask when relu != 0.
 *   ws: scratch of b2c_bn_relu_bwd_groups_workspace_bytes(c, groups) bytes, 8-byte aligned; the call zeroes it. */
size_t b2c_bn_relu_bwd_groups_workspace_bytes(int c, int groups);
b2c_status b2c_bn_relu_bwd_groups(b2c_ctx* ctx, int groups, long long rows_per_group, int c, const void* da1,
                                  const void* da2, const void* y, const float* gamma, const float* save_mean,
                                  const float* save_invstd, int relu, void* dy, void* dres, float* dgamma,
                                  float* dbeta, int acc, const void* relu_mask, void* ws, size_t ws_bytes,
                                  void* stream);

/* (No counterpart in the paper: a packaging variant of b2c_bn_relu_bwd.)
 * The same computation, arguments and results as b2c_bn_relu_bwd, but without the `ws` argument: the per-channel
 * fp64 accumulators live in an array built into the library (B2C_BN_BWD_STATIC_MAX_C channels, 32 KB, resident on
 * every GPU that loads the library until the process exits).  It is meant for callers that cannot obtain device
 * memory of their own at the point of the call: code running under an allocator it does not control (a plug-in that
 * is handed only its input and output buffers), code with a fixed memory budget drawn up in advance, and code that
 * must not stall, since the CUDA allocation calls synchronise the device.  This entry point calls no allocating
 * routine at all, of CUDA or of any library.
 *   - c > B2C_BN_BWD_STATIC_MAX_C returns B2C_ERR_WORKSPACE_TOO_SMALL and enqueues nothing.
 *   - The context's device must be the current device.  The first call on a device looks up the array's device
 *     address (a set-up step); make that first call before any stream capture starts.
 *   - All calls on a device share the one array, which keeps the previous call's sums; each call clears what it
 *     uses before reducing into it.  Two calls whose kernels overlap on the GPU (different streams, or different
 *     host threads) race on it: serialise them on one stream. */
#define B2C_BN_BWD_STATIC_MAX_C 2048
b2c_status b2c_bn_relu_bwd_static(b2c_ctx* ctx, int n, int h, int w, int c, const void* da1, const void* da2,
                                  const void* y, const void* a, const float* gamma, const float* save_mean,
                                  const float* save_invstd, int relu, void* dy, void* dres, float* dgamma,
                                  float* dbeta, int acc, void* stream);

/* dx[n,h,w,c] = sum over (p,q,r,s,k) with p*stride+r-pad = h, q*stride+s-pad = w of dy[n,p,q,k]*w[k,r,s,c].
 *   dy bf16 [n,p,q,k]; dx bf16 [n,h,w,c] (every element written)
 *   w_crsk_flipped bf16 [c,r,s,k] with w_crsk_flipped[c,r,s,k] = w[k, R-1-r, S-1-s, c]
 *   (b2c_weight_pack_dgrad writes this layout). */
b2c_status b2c_conv2d_dgrad(b2c_ctx* ctx, const b2c_conv_desc* d, const void* dy, const void* w_crsk_flipped,
                            void* dx, void* stream);

/* dw[k,r,s,c] (+)= sum_{n,p,q} dy[n,p,q,k] * x[n, p*stride+r-pad, q*stride+s-pad, c].
 *   dy bf16 [n,p,q,k]; x bf16 [n,h,w,c]; dw fp32 [k,r,s,c]
 *   accumulate == 0: dw is zeroed first; != 0: the sum is added to dw (micro-batch accumulation).
 * Partial sums over pixel ranges are combined with fp32 atomic adds (order not deterministic). */
b2c_status b2c_conv2d_wgrad(b2c_ctx* ctx, const b2c_conv_desc* d, const void* dy, const void* x, float* dw_krsc,
                            int accumulate, void* stream);

/* db[k] (+)= sum_m dz[m, k] for bf16 dz [m, pitch]; fp32 db [k]. */
b2c_status b2c_bias_grad(b2c_ctx* ctx, int m, int k, int pitch, const void* dz, float* db, int accumulate, void* stream);

/* ---- Gradient averaging + update (Algorithm 1, "Synchronize gradients", "Update parameters") */

/* For i in [0,count): g = g_accum[i]*inv_n_micro + wd*w[i]; v[i] = momentum*v[i] + g;
 * w[i] -= lr*v[i]; w_bf16[i] = bf16(w[i]) if w_bf16 != NULL; g_accum[i] = 0 if zero_grad.
 * w, v, g_accum fp32 flat arrays; count % 4 == 0. */
b2c_status b2c_grad_accum_sgd_momentum(b2c_ctx* ctx, size_t count, float* w, float* v, float* g_accum,
                                       float inv_n_micro, float lr, float momentum, float wd, void* w_bf16,
                                       int zero_grad, void* stream);

/* One filter bank of a flat weight array: `offset` elements from the base, shape [k, rs, c]. */
typedef struct {
    long long offset;
    int k, rs, c;
} b2c_weight_seg;
/* For every segment: dst[offset + (c_*rs + t)*k + k_] = src[offset + (k_*rs + (rs-1-t))*c + c_],
 * i.e. the [c,r,s,k] tap-flipped layout b2c_conv2d_dgrad reads.  src, dst bf16; n_segs <= 128. */
b2c_status b2c_weight_pack_dgrad(b2c_ctx* ctx, const b2c_weight_seg* segs, int n_segs, const void* src_bf16,
                                 void* dst_bf16, void* stream);

/* ---- Whole step over a layer list ------------------------------------------------------- */

enum { B2C_LAYER_CONV = 0, B2C_LAYER_BN = 1, B2C_LAYER_AVGPOOL = 2, B2C_LAYER_FC = 3, B2C_LAYER_XENT = 4 };

/* Tensor 0 is the image batch; layer i writes tensor i+1.  `src` is the input tensor; for BN
 * layers `res` is the residual tensor (-1: none) and `relu` selects the activation.  For CONV,
 * c/k/r/stride describe the filter (pad = (r-1)/2) and h,w the input size; for BN/AVGPOOL c,h,w
 * describe the input; for FC c inputs and k outputs; for XENT k classes. */
typedef struct {
    int kind, src, res, relu;
    int c, k, r, stride, h, w;
} b2c_layer_desc;

/* Builds the execution plan for micro-batches of `micro_batch` images of hw x hw x image_c. */
b2c_status b2c_net_create(b2c_ctx* ctx, const b2c_layer_desc* layers, int n_layers, int micro_batch, b2c_net** out);
/* As b2c_net_create, but every pass of b2c_train_step runs n_concurrent micro-batches side by side as one
 * batch of micro_batch*n_concurrent images (larger GEMMs, fewer launches).  BatchNorm statistics stay per
 * micro-batch, so results equal those of n_concurrent == 1 up to summation order.  The workspace grows by
 * the same factor and b2c_train_step requires n_micro % n_concurrent == 0. */
b2c_status b2c_net_create_concurrent(b2c_ctx* ctx, const b2c_layer_desc* layers, int n_layers, int micro_batch,
                                     int n_concurrent, b2c_net** out);
void b2c_net_destroy(b2c_net* net);
/* Elements of the flat parameter arrays (fp32 master, momentum, gradient sum; a bf16 copy and a
 * bf16 dgrad-layout copy of the same length).  Includes zero padding (first conv: input channels
 * padded to 16) and is a multiple of 4. */
size_t b2c_net_param_count(const b2c_net* net);
/* Element offset of a layer's parameter inside the flat arrays.  which: 0 = weight (conv: [k,r,s,c_padded],
 * fc: [k,c]), 1 = BN gamma, 2 = BN beta, 3 = fc bias.  Returns -1 if the layer has no such parameter. */
long long b2c_net_param_offset(const b2c_net* net, int layer, int which);
/* Stored input width of the first convolution (what its weight layout uses): the image channels rounded up to 16,
 * or 32 when b2c_net_first_conv_im2col() is non-zero. */
int b2c_net_padded_image_channels(const b2c_net* net);
/* Non-zero if the first convolution (3x3, stride 1, at most 3 image channels) runs on the 3x3 patch matrix of the
 * image batch: its filter bank is then stored as [k][32] rows holding the [r][s][c] taps flattened (27 used). */
int b2c_net_first_conv_im2col(const b2c_net* net);
/* Bytes of activation/gradient workspace one micro-batch needs. */
size_t b2c_net_workspace_bytes(const b2c_net* net);
/* Byte offset inside the workspace of tensor t's activation (bf16; logits fp32), or of its
 * gradient contribution `which` (0 or 1) when grad != 0.  -1 if absent.  For tests/inspection. */
long long b2c_net_tensor_offset(const b2c_net* net, int tensor, int grad, int which);
/* Binds caller-owned device memory: five flat parameter arrays of b2c_net_param_count elements
 * (w_master, velocity, grad_sum fp32; w_bf16, w_bf16_dgrad bf16) and the workspace. */
b2c_status b2c_net_bind(b2c_net* net, float* w_master, float* velocity, float* grad_sum, void* w_bf16,
                        void* w_bf16_dgrad, void* workspace, size_t workspace_bytes);
/* Running statistics of the BatchNorm layers (optional; they do not enter the step's results).  After
 * b2c_net_bind_running_stats(net, running, momentum) every pass of b2c_train_step updates, after its forward pass,
 *   running_mean = (1 - momentum) * running_mean + momentum * mean,
 *   running_var  = (1 - momentum) * running_var  + momentum * var * m / (m - 1)      (unbiased, m rows per micro-batch)
 * for every BatchNorm layer, the micro-batches of a pass applied in order.  `running` is a caller-owned fp32 DEVICE
 * array of b2c_net_running_stats_count elements; layer i's block [mean c][var c] starts at
 * b2c_net_running_stats_offset(net, i) (-1 for layers without statistics).  The caller initialises it (mean 0,
 * variance 1).  running == NULL switches the update off (the default). */
size_t b2c_net_running_stats_count(const b2c_net* net);
long long b2c_net_running_stats_offset(const b2c_net* net, int layer);
b2c_status b2c_net_bind_running_stats(b2c_net* net, float* running, float momentum);
/* Refreshes w_bf16 and w_bf16_dgrad from w_master (call once after initialising the masters). */
b2c_status b2c_net_sync_weights(b2c_net* net, void* stream);
/* One optimiser step: for each of n_micro micro-batches (images bf16 [n_micro*micro_batch, h, w, c],
 * labels int32) forward, loss, backward with gradients summed into grad_sum; then one fused
 * average + SGD-momentum update which also refreshes both bf16 weight copies and zeroes grad_sum.
 * *loss_dev (fp32 device scalar) receives the mean loss over all images of the step.
 * If update == 0 the parameter update is skipped and grad_sum keeps the summed gradients. */
b2c_status b2c_train_step(b2c_net* net, const void* images, const int32_t* labels, int n_micro, float lr,
                          float momentum, float wd, float* loss_dev, int update, void* stream);

/* The gradient synchronisation + update alone: g = grad_sum / n_avg + wd*w; v = momentum*v + g; w -= lr*v; both bf16
 * weight copies are refreshed and grad_sum is zeroed.  Data-parallel replicas call b2c_train_step with update == 0,
 * sum grad_sum across replicas (e.g. an NCCL all-reduce), then call this with n_avg = n_micro * replicas. */
b2c_status b2c_net_apply_update(b2c_net* net, int n_avg, float lr, float momentum, float wd, void* stream);

/* Pieces of the update for data-parallel replicas that shard the optimiser state (gradient synchronisation fused with
 * the update: reduce-scatter of grad_sum, b2c_grad_accum_sgd_momentum on the replica's own slice of the flat arrays,
 * all-gather of the bf16 copy): the filter banks of the weight layers occupy [begin, end) element ranges of the flat
 * arrays in layer order (b2c_net_weight_range, index < b2c_net_weight_layer_count; the backward pass completes them
 * last layer first), and b2c_net_refresh_dgrad_weights rewrites w_bf16_dgrad from the current w_bf16. */
int b2c_net_weight_layer_count(const b2c_net* net);
/* Gradient-ready events for buckets of the flat arrays: after b2c_net_set_buckets, every b2c_train_step records event k
 * on its stream once weight layer first_layer[k] (an index < b2c_net_weight_layer_count) has finished its parameter
 * gradient for the step; every later weight layer, and with first_layer[k] == 0 everything else, is final by then.
 * b2c_net_bucket_wait makes `stream` (the stream of the collectives) wait for event k, so that a bucket's exchange
 * starts while the backward pass of the earlier layers still runs.  n_buckets == 0 removes the events. */
b2c_status b2c_net_set_buckets(b2c_net* net, int n_buckets, const int* first_layer);
b2c_status b2c_net_bucket_wait(b2c_net* net, int bucket, void* stream);
b2c_status b2c_net_weight_range(const b2c_net* net, int index, long long* begin, long long* end);
b2c_status b2c_net_refresh_dgrad_weights(b2c_net* net, void* stream);

/* ---- Per-component timing (the profiling phase of the paper's adaptive scheduling algorithm
 *      measures the execution time of each network component; this is the measurement hook) ---- */

/* Kernel families a step's launches are attributed to. */
enum {
    B2C_PROF_CONV_FWD = 0, B2C_PROF_CONV_DGRAD = 1, B2C_PROF_CONV_WGRAD = 2, B2C_PROF_BN_FWD = 3, B2C_PROF_BN_BWD = 4,
    B2C_PROF_OTHER = 5, B2C_PROF_UPDATE = 6, B2C_PROF_KINDS = 7
};
/* enable != 0: b2c_train_step brackets every launch site with CUDA events on its stream. */
b2c_status b2c_net_profile_enable(b2c_net* net, int enable);
/* Synchronises `stream`; ms[kind] = device time summed over the launch sites of that family since the
 * last read (0 unless enabled), launches[kind] = kernels launched since the last read (always counted).
 * Both arrays are HOST memory of B2C_PROF_KINDS entries.  Resets the sums. */
b2c_status b2c_net_profile_read(b2c_net* net, double* ms, long long* launches, void* stream);
/* The same records per network component (the partition of the model into logical components that the paper's
 * scheduling algorithm profiles is the layer list): ms[3*i + 0] = forward time of layer i, ms[3*i + 1] = its
 * parameter-gradient time (weight gradient; bias gradient), ms[3*i + 2] = its data-gradient time (convolution data
 * gradient, BatchNorm / pooling backward), summed since the last b2c_net_profile_read.  HOST memory of 3*n_layers
 * doubles; n_layers must equal b2c_net_layer_count.  Synchronises `stream`; does not reset the records, so call it
 * before b2c_net_profile_read.  All zero unless profiling is enabled. */
b2c_status b2c_net_profile_read_layers(b2c_net* net, double* ms, int n_layers, void* stream);
int b2c_net_layer_count(const b2c_net* net);

#ifdef __cplusplus
}
#endif
#endif /* B2C_H_ */
