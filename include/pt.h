/*
 * pt.h -- C ABI of the B200 (sm_100a) hot path of PruneTrain (arxiv 1901.09290).
 *
 * The library covers the convolution training step of a group-lasso-regularised CNN
 * whose channel counts keep shrinking: conv forward / data gradient / weight gradient
 * on ragged channel counts, the fused group-lasso + momentum-SGD update, zero-group
 * detection and channel-union compaction ("reconfiguration").
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - The caller allocates and frees every buffer, workspaces included. The library
 *     allocates device memory only inside pt_create (a status word and a small table
 *     arena) and frees it in pt_destroy.
 *   - Every call validates its arguments on the host before any launch, enqueues its
 *     kernels on `stream` (a cudaStream_t passed as void*) and returns without
 *     synchronising, except pt_reconfigure_plan (documented below).
 *   - Every call returns a pt_status. Device-side bounded waits that expire record
 *     PT_ERR_TIMEOUT in the context's status word, read by pt_poll_device_status.
 *   - There is no CPU fallback anywhere.
 *
 * Physical layouts
 *   activations x, y, dy, dx : [N][H][W][ld]   bf16 (or fp32 outputs when out_f32 = 1), channels
 *                              innermost, channel pitch ld >= channels, ld a multiple of 8 elements.
 *                              Pad lanes (channel index >= channels) are never read. bf16 outputs may get zeros
 *                              written into the pad lanes up to the next multiple of 16 channels where the pitch has
 *                              room for them (whole 32-byte sectors are stored: a half-written sector costs a
 *                              read-modify-write in the memory system), else up to the end of the last 16-byte
 *                              granule; other pad lanes are left untouched.
 *   master weights w, momentum v, gradient g/dw : [K][R][S][C] fp32, dense (no pitch).
 *   bf16 weight shadow       : [K][R][S][ldw]  bf16, ldw >= C, ldw a multiple of 8.
 *   Output size: P = floor((H + 2*pad - R)/stride) + 1, Q likewise from W and S.
 */
#ifndef PT_H_
#define PT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PT_OK = 0,
    PT_ERR_INVALID_ARG = 1,   /* null pointer, bad pitch/alignment/shape                */
    PT_ERR_UNSUPPORTED = 2,   /* legal but not implemented (e.g. a forced algo that cannot run the shape) */
    PT_ERR_WORKSPACE = 3,     /* workspace missing or smaller than pt_*_workspace_bytes */
    PT_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                      */
    PT_ERR_TIMEOUT = 5,       /* a bounded device-side wait expired                     */
    PT_ERR_ARCH = 6           /* the device is not sm_100                               */
} pt_status;

typedef struct pt_ctx pt_ctx;  /* opaque: device id, SM count, status word, table arena, arrival counters */

/* Create / destroy the per-device context. pt_create makes `device` current, checks that it is
 * an sm_100 part (else PT_ERR_ARCH) and allocates the status word and table arena. */
pt_status pt_create(pt_ctx **ctx, int device);
pt_status pt_destroy(pt_ctx *ctx);
const char *pt_status_string(pt_status s);
/* After a call returned PT_ERR_CUDA: the CUDA error's name and the runtime call that returned it, as text, for the calling
 * thread (an empty string if none failed yet). The pointer stays valid; the text changes with the thread's next failure. */
const char *pt_last_cuda_error(void);
/* Synchronises `stream`, reads and clears the device status word. PT_OK if no kernel recorded an error; PT_ERR_TIMEOUT for
 * an expired device-side wait; PT_ERR_INVALID_ARG for a channel index outside its tensor (pt_channel_gather,
 * pt_channel_scatter_add and pt_reconfigure skip such an entry). */
pt_status pt_poll_device_status(pt_ctx *ctx, void *stream);
/* Testing hooks for the bounded device-side waits (no counterpart in the paper). Every wait of a kernel on an mbarrier or on
 * another CTA has a time limit (2 s); a wait that runs out makes its CTA record the time-out, drain the copies it issued,
 * free its tensor memory and exit, and pt_poll_device_status then returns PT_ERR_TIMEOUT (and clears the arrival counters of
 * the split weight gradients, which a kernel that gave up leaves behind). These two calls let a test reach that path without
 * any fault: pt_test_set_wait_limit sets the limit for every context on the device (milliseconds; 0 restores 2 s; it
 * synchronises), and pt_test_skip_next_arrive makes ONE later launch leave out one arrival, so that its waits run out:
 *   which = 1: the next pt_conv_wgrad that splits its reduction over CTAs -- split 0 does not announce its partial tile;
 *   which = 2: the next forward / data-gradient launch of the pixel-linear (GEMM-form) kernel -- the activation producer of
 *              every CTA leaves out the first pipeline stage;   which = 0 disarms.
 * The outputs of that launch are undefined. Not for production use. */
pt_status pt_test_set_wait_limit(pt_ctx *ctx, uint32_t milliseconds);
pt_status pt_test_skip_next_arrive(pt_ctx *ctx, int32_t which);
/* Number of kernels this context has launched since creation (for launch accounting). */
uint64_t pt_launch_count(const pt_ctx *ctx);
/* Upper bound on the CTAs (one per SM) a pt_conv_wgrad launch may use; 0 restores the default, all SMs. The weight gradient
 * (Eq. 4) splits its reduction over the output pixels across CTAs, and the weight gradients of different layers are
 * independent of each other: launches that leave SMs free can run side by side on several streams, which amortises their
 * fixed cost (pipeline fill, partial-tile exchange). The setting changes the workspace pt_conv_workspace_bytes reports for
 * PT_CONV_WGRAD, so set it before sizing workspaces; it has no effect on results beyond the summation order of the splits
 * (still fixed for a given setting). PT_ERR_INVALID_ARG if max_ctas is negative.
 * The CTAs of a split launch wait (bounded) for one another and occupy an SM each, so all of them must be able to be on
 * the device at once: a caller that keeps weight-gradient launches in flight on S streams sets a limit L with
 * S * L <= the SM count. Beyond that the launches may starve each other until a wait expires (PT_ERR_TIMEOUT at the next
 * pt_poll_device_status; nothing hangs). */
pt_status pt_set_wgrad_cta_limit(pt_ctx *ctx, int max_ctas);

/* ------------------------------------------------------------------------------------------
 * Convolutions (paper Sec. 2.1: convolution layers dominate training time; Eq. 4: weight gradient).
 * Cross-correlation, square stride and padding, dilation 1, groups 1, no bias.
 * C and K are the CURRENT (pruned, possibly ragged: 11, 27, 93 ...) channel counts.
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t N, H, W, C, K, R, S, stride, pad;
    int32_t ldx;      /* channel pitch of x / dx  (elements, multiple of 8, >= C)           */
    int32_t ldy;      /* channel pitch of y / dy  (elements, multiple of 8, >= K)           */
    int32_t ldw;      /* channel pitch of the bf16 weight shadow (multiple of 8, >= C)      */
    int32_t out_f32;  /* fwd/dgrad: 0 = bf16 output, 1 = fp32 output (same pitch in elements) */
    int32_t algo;     /* 0 = automatic; 1 = force the SIMT kernels; 2 = force the tcgen05 kernels */
} pt_conv_desc;

enum { PT_CONV_FWD = 0, PT_CONV_DGRAD = 1, PT_CONV_WGRAD = 2 };

/* Bytes of caller-provided workspace the given pass needs for this descriptor (0 = none). */
size_t pt_conv_workspace_bytes(const pt_ctx *ctx, const pt_conv_desc *d, int which);
/* CTAs pt_conv_wgrad launches for this descriptor at the context's current limit (pt_set_wgrad_cta_limit): tiles x splits,
 * splits being the largest count that keeps the product within the limit (at least 1: a descriptor with more tiles than
 * the limit runs unsplit). *waits (optional) = 1 if those CTAs wait for one another (splits > 1), which is what the
 * co-residency rule of pt_set_wgrad_cta_limit is about. Lets a caller choose per-launch limits that waste no SMs.
 * 0 if the tcgen05 kernels do not take the descriptor. */
int32_t pt_conv_wgrad_ctas(const pt_ctx *ctx, const pt_conv_desc *d, int32_t *waits);

/* Stream order: the three calls below are ordinary stream work. Their kernels are launched with programmatic stream
 * serialization and read the WEIGHTS before waiting for the preceding kernel of the stream; that is invisible to callers
 * because only kernels that release their dependents early (griddepcontrol.launch_dependents before their last store) can be
 * overtaken: of this library's kernels the convolutions and the read-only sweeps of the lasso step do that, and none of them
 * writes weights (the update of pt_group_lasso_sgd_step and the gather of pt_reconfigure complete before their successors
 * start). A caller's own kernel that writes w and releases its dependents early must be followed by an event or another
 * kernel before a convolution reads w. */
/* y[n,p,q,k] = sum_{r,s,c} x[n, p*stride-pad+r, q*stride-pad+s, c] * w[k,r,s,c], zero outside the image.
 * x: bf16 [N][H][W][ldx]; w: bf16 shadow [K][R][S][ldw]; y: [N][P][Q][ldy] bf16 or fp32. fp32 accumulation. */
pt_status pt_conv_fwd(pt_ctx *ctx, const pt_conv_desc *d, const void *x, const void *w, void *y,
                      void *ws, size_t ws_bytes, void *stream);

/* The same forward convolution (bf16 output, tcgen05 kernels only: PT_ERR_UNSUPPORTED otherwise) that also takes the
 * statistics the batch normalisation after it needs (Sec. 2.1: the normalisation layers are bound by memory bandwidth because
 * they read their input several times): every epilogue warp adds, per output channel, the sum and the sum of squares of the bf16
 * values it stores -- from the tile that is still in shared memory -- into a row of its own. stats receives *n_parts (host, out)
 * rows of [2][ldy] floats (row r: sums, then sums of squares; columns >= K are zero); pt_bn_relu_fwd_stats combines them in a
 * fixed order. stats must hold pt_conv_fwd_stats_bytes(ctx, d) bytes (an upper bound that does not depend on which kernel
 * serves the layer); PT_ERR_WORKSPACE if it is smaller than this launch needs. Run-to-run identical. */
size_t pt_conv_fwd_stats_bytes(const pt_ctx *ctx, const pt_conv_desc *d);
pt_status pt_conv_fwd_stats(pt_ctx *ctx, const pt_conv_desc *d, const void *x, const void *w, void *y, float *stats,
                            size_t stats_bytes, int32_t *n_parts /*host*/, void *ws, size_t ws_bytes, void *stream);

/* dx[n,h,w,c] = sum over (k,r,s,p,q) with p*stride-pad+r = h and q*stride-pad+s = w of dy[n,p,q,k] * w[k,r,s,c].
 * Back-propagation through the layer (Sec. 2.1). Pixels no tap reaches are written as 0.
 * dy: bf16 [N][P][Q][ldy]; dx: [N][H][W][ldx] bf16 or fp32. */
pt_status pt_conv_dgrad(pt_ctx *ctx, const pt_conv_desc *d, const void *dy, const void *w, void *dx,
                        void *ws, size_t ws_bytes, void *stream);

/* dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] * x[n, p*stride-pad+r, q*stride-pad+s, c]   (Eq. 4).
 * dw: fp32 [K][R][S][C] dense. Deterministic: partial sums are combined in a fixed order. */
pt_status pt_conv_wgrad(pt_ctx *ctx, const pt_conv_desc *d, const void *x, const void *dy, float *dw,
                        void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * Group-lasso regularised momentum SGD (Eq. 1-2; Algorithm 1: GroupLassoReg(W_i) then Optimizer).
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    float *w;            /* fp32 master weights [K][RS][C], updated in place                        */
    const float *g;      /* fp32 gradient of the data loss (wgrad output), same layout               */
    float *v;            /* fp32 momentum, updated in place                                          */
    void *w_bf16;        /* bf16 shadow [K][RS][ldw], rewritten from the new w; may be NULL          */
    int32_t K, C, RS, ldw;
    uint8_t reg_in;      /* regularise the input-channel groups (0 for the first conv: its inputs are the image) */
    uint8_t reg_out;     /* regularise the output-channel groups                                      */
    float *sumsq_out;    /* K floats: sum of squares of each output-channel group of the PRE-update w */
    float *sumsq_in;     /* C floats: same for input-channel groups                                   */
    uint8_t *zero_out;   /* K bytes, written by pt_find_zero_groups (1 = group is zero)               */
    uint8_t *zero_in;    /* C bytes                                                                    */
} pt_layer;

typedef struct { float lambda, lr, momentum, weight_decay; } pt_sgd_hparams;

/* Workspace for pt_group_lasso_sgd_step and pt_find_zero_groups over this set of layers. */
size_t pt_group_lasso_workspace_bytes(const pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers);

/* For every layer:  s_out[k] = sum_{rs,c} w^2,  s_in[c] = sum_{k,rs} w^2  (pre-update weights),
 *   g~ = g + weight_decay*w + lambda*w*( [reg_out, s_out>1e-24]/sqrt(s_out[k]) + [reg_in, s_in>1e-24]/sqrt(s_in[c]) )
 *   v <- momentum*v + g~ ;  w <- w - lr*v ;  shadow <- round-to-nearest-even bf16 of the new w.
 * That is the gradient of Eq. 1 with the regulariser of Eq. 2 (one global lambda; input- and output-channel
 * groups overlap) followed by the optimiser step of Algorithm 1. An all-zero group has subgradient 0.
 * reg_sum_out (device, optional): receives sum over regularised groups of sqrt(sumsq) -- Eq. 2 without lambda.
 * layers is a HOST array; the library keeps device copies of the last three distinct layer sets given to this call (two for
 * pt_find_zero_groups) and uploads a table only when it is not among them. A CUDA graph captured around this call embeds
 * the table's device address: it stays valid until three other layer sets have been used with the same context. */
pt_status pt_group_lasso_sgd_step(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers,
                                  const pt_sgd_hparams *hp /*host*/, double *reg_sum_out,
                                  void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * Feature normalisation (Sec. 2.1: batch normalisation layers take about 30 % of CNN training time and are bound by memory
 * bandwidth because they read their input several times) with the residual add and ReLU of a ResNet block fused in.
 * Activations are NHWC bf16 with channel pitch ld, exactly as the convolutions read and write them; C is the CURRENT
 * (pruned, possibly ragged) channel count. Per channel, over the M = N*H*W positions:
 *     mean = sum(x)/M, var = sum((x-mean)^2)/M, xhat = (x-mean)/sqrt(var+eps), z = gamma*xhat + beta (+ residual),
 *     y = relu ? max(z, 0) : z;   running <- (1-momentum)*running + momentum*(mean | var*M/(M-1)).
 * Backward (dz = dy where y > 0, or dy without ReLU):
 *     dbeta = sum(dz), dgamma = sum(dz*xhat), dx = gamma/sqrt(var+eps)/M * (M*dz - dbeta - xhat*dgamma), dresidual = dz.
 * All pointers are device pointers; x, y, residual, dy, dx, dresidual are 16-byte aligned [N][H][W][ld] bf16 tensors whose
 * pad lanes (channel >= C) are read but never used, and are written as zeros in the outputs. Statistics, gamma, beta and
 * their gradients are fp32 vectors of C elements. Sums are combined in a fixed order (run-to-run identical).
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t N, H, W, C;
    int32_t ld;        /* channel pitch (elements, multiple of 8, >= C, <= 2048) */
    float eps;         /* >= 0 */
    float momentum;    /* of the moving statistics, in [0, 1] */
    int32_t relu;      /* 0 / 1 */
} pt_bn_desc;

/* Bytes of workspace both calls need for this descriptor (partial sums of the reduction blocks). */
size_t pt_bn_workspace_bytes(const pt_ctx *ctx, const pt_bn_desc *d);

/* y = relu(gamma*xhat + beta + residual). residual may be NULL. running_mean / running_var: both NULL (not kept) or both
 * given (updated in place). save_mean, save_invstd (C floats each) receive the batch statistics the backward pass needs.
 * PT_ERR_INVALID_ARG for bad sizes, pitches, alignment or missing pointers; PT_ERR_UNSUPPORTED for ld > 2048;
 * PT_ERR_WORKSPACE if ws is too small. */
pt_status pt_bn_relu_fwd(pt_ctx *ctx, const pt_bn_desc *d, const void *x, const void *residual, const float *gamma,
                         const float *beta, float *running_mean, float *running_var, float *save_mean, float *save_invstd,
                         void *y, void *ws, size_t ws_bytes, void *stream);

/* The same forward pass without its reduction over x: the batch statistics come from the rows of partial sums the producing
 * convolution left (pt_conv_fwd_stats: stats, n_parts; the sums are those of the stored bf16 values, exactly what the
 * reduction pass of pt_bn_relu_fwd would read). Two launches instead of three, one pass over x instead of two; no workspace. */
pt_status pt_bn_relu_fwd_stats(pt_ctx *ctx, const pt_bn_desc *d, const void *x, const void *residual, const float *gamma,
                               const float *beta, float *running_mean, float *running_var, float *save_mean, float *save_invstd,
                               void *y, const float *stats, int32_t n_parts, void *stream);

/* Gradients of the call above. y is the forward output (only its sign is used, and only with relu = 1; may be NULL
 * otherwise); dresidual may be NULL when the block has no residual input. */
pt_status pt_bn_relu_bwd(pt_ctx *ctx, const pt_bn_desc *d, const void *x, const void *y, const void *dy, const float *gamma,
                         const float *save_mean, const float *save_invstd, void *dx, void *dresidual, float *dgamma,
                         float *dbeta, void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * Max pooling (Sec. 2.1 counts the pooling layers among the cheap, bandwidth-bound layers; ResNet has one, after its first
 * convolution). Present so that a training step can be chained from the image to the last feature map. Activations as above:
 * [N][H][W][ld] bf16, 16-byte aligned, ld a multiple of 8; square window R, stride, padding pad < R; output
 * [N][P][Q][ld] with P = floor((H + 2*pad - R)/stride) + 1. Positions outside the image are never selected; of equal maxima the
 * first in scan order (rows, then columns of the window) is the selected one and receives the gradient. Pad lanes of the
 * outputs are written as zeros. Nothing is added atomically. `index` (device, optional, 8-byte aligned, uint8
 * [N][P][Q][ld], R*R <= 255): the forward pass leaves the selected position r*R + s of every window there (255: none, and in
 * the pad lanes) and the backward pass reads it; with index = NULL the backward pass recomputes the selections from x (R*R
 * loads per window instead of one). PT_ERR_INVALID_ARG for bad sizes, pitches, alignment or null pointers.
 * ------------------------------------------------------------------------------------------ */
typedef struct { int32_t N, H, W, C, ld, R, stride, pad; } pt_pool_desc;
pt_status pt_maxpool_fwd(pt_ctx *ctx, const pt_pool_desc *d, const void *x, void *y, void *index, void *stream);
/* dx[n,h,w,c] = sum of dy[n,p,q,c] over the windows (p,q) whose selected position is (h,w); x is the forward input (may be
 * NULL when index is given). */
pt_status pt_maxpool_bwd(pt_ctx *ctx, const pt_pool_desc *d, const void *x, const void *dy, const void *index, void *dx,
                         void *stream);

/* ------------------------------------------------------------------------------------------
 * Dynamic mini-batch adjustment (Sec. 4.3; Algorithm 1, "UpdateMiniBatch(system_memory, Net)"): after every reconfiguration
 * the memory one training iteration needs is re-evaluated for the smaller network, the mini-batch grows in steps of a
 * granularity (the paper uses 32 samples per GPU) as far as the device memory allows, and the learning rate grows by the
 * same ratio. Host-side arithmetic only; no device is touched.
 * The memory model is this library's own buffers (the paper gives none): per parameter fp32 weight, gradient and momentum
 * plus the bf16 shadow (14 bytes, pitch padding included for the shadow); per sample and per convolution the bf16 input
 * and output activations and their two gradients, at the channel pitch the tensors are stored with (multiple of 8).
 * ------------------------------------------------------------------------------------------ */
typedef struct { int32_t H, W, C, K, R, S, stride, pad; } pt_layer_shape;   /* CURRENT (pruned) sizes of one convolution */

/* Bytes one iteration needs at mini-batch `batch` (0 if an argument is invalid). */
size_t pt_training_memory_bytes(const pt_layer_shape *layers /*host*/, int32_t n_layers, int32_t batch);

/* new_batch = cur_batch + granularity * g with the largest g >= 0 whose memory fits capacity_bytes (the mini-batch never
 * shrinks: if even cur_batch does not fit, it is returned unchanged); new_lr = cur_lr * new_batch / cur_batch.
 * PT_ERR_INVALID_ARG for cur_batch < 1, granularity < 1, bad shapes or null pointers. */
pt_status pt_update_mini_batch(const pt_layer_shape *layers /*host*/, int32_t n_layers, size_t capacity_bytes, int32_t cur_batch,
                               float cur_lr, int32_t granularity, int32_t *new_batch /*host*/, float *new_lr /*host*/);

/* ------------------------------------------------------------------------------------------
 * Penalty coefficient set-up (Sec. 4.1, "Regularization Penalty Coefficient Setup", Eq. 3): lambda is chosen once, at the
 * first training iteration, so that the group-lasso term is a given share (the paper uses 20-25 %) of the total loss:
 *     ratio = lambda * R / (loss + lambda * R),  R = sum over groups of ||W_g||   =>   lambda = ratio * loss / ((1 - ratio) * R)
 * with loss the cross-entropy of the first forward pass and R the value pt_group_lasso_sgd_step writes to reg_sum_out.
 * ------------------------------------------------------------------------------------------ */

/* loss_out[0] (device, double) = mean over the batch of -log softmax(logits[i])[labels[i]].
 * logits: device, fp32, [n][ld] with ld >= classes (elements past `classes` are never read); labels: device, int32, each
 * in [0, classes). Rows are reduced in fp32 with the row maximum subtracted, the batch mean is accumulated in fp64 in a
 * fixed order (run-to-run identical). A label out of range makes the result NaN. ws: device scratch of at least
 * pt_cross_entropy_workspace_bytes(n) bytes. PT_ERR_INVALID_ARG for n < 1, classes < 1, ld < classes, null pointers. */
size_t pt_cross_entropy_workspace_bytes(int32_t n);
pt_status pt_cross_entropy(pt_ctx *ctx, const float *logits, const int32_t *labels, int32_t n, int32_t classes, int32_t ld,
                           double *loss_out, void *ws, size_t ws_bytes, void *stream);

/* lambda_out[0] (device, float) = ratio * loss[0] / ((1 - ratio) * reg_sum[0])  (Eq. 3 solved for lambda), computed in fp64.
 * loss, reg_sum: device doubles (from pt_cross_entropy and pt_group_lasso_sgd_step). reg_sum == 0 (no regularised group
 * left) gives lambda = 0. PT_ERR_INVALID_ARG unless 0 < ratio < 1. The caller reads lambda_out back to fill
 * pt_sgd_hparams.lambda for the steps that follow. */
pt_status pt_set_coeff(pt_ctx *ctx, const double *loss, const double *reg_sum, float ratio, float *lambda_out, void *stream);

/* The same step in two calls, for callers that want the group norms out of the way early: the norms depend on the weights
 * only (Algorithm 1 evaluates GroupLassoReg on W_i, the weights the forward pass used), not on the gradients, so
 * pt_group_lasso_norms may run on another stream while the backward pass is still producing g. It fills sumsq_out /
 * sumsq_in, reg_sum_out (optional) and the inverse norms kept in ws; pt_group_lasso_sgd_apply then performs the update
 * from them. Contract: same layers array, same ws, and the weights unchanged between the two calls; the pair computes
 * bit for bit what pt_group_lasso_sgd_step computes. (g may be NULL in the layers given to pt_group_lasso_norms.) */
pt_status pt_group_lasso_norms(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers, double *reg_sum_out,
                               void *ws, size_t ws_bytes, void *stream);
pt_status pt_group_lasso_sgd_apply(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers,
                                   const pt_sgd_hparams *hp /*host*/, void *ws, size_t ws_bytes, void *stream);
/* The update of layers [first, first + count) only, from the norms pt_group_lasso_norms left in ws (same layers array, same
 * ws). A layer's update needs its own gradient and nothing else, so a caller can apply it as soon as that gradient exists
 * (on the stream that produced it) instead of after the whole backward pass. Calls covering every layer exactly once compute
 * bit for bit what pt_group_lasso_sgd_apply computes. PT_ERR_INVALID_ARG for a range outside [0, n_layers). */
pt_status pt_group_lasso_sgd_apply_layers(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers, int32_t first,
                                          int32_t count, const pt_sgd_hparams *hp /*host*/, void *ws, size_t ws_bytes,
                                          void *stream);

/* The carried form of the step (Algorithm 1 evaluates GroupLassoReg on W_i: the sums of squares of W_{i+1} that step i + 1 needs
 * can be taken while step i writes W_{i+1}): the update uses the 1/norm factors that ws already holds and, in the same pass
 * over the weights, accumulates the sums of squares of the NEW weights -- and, with with_maxima != 0, the maxima of |w| that
 * pt_find_zero_groups_carried reads (ask for them in the step before a reconfiguration) -- from which a short finish kernel
 * rewrites the factors in ws, sumsq_out / sumsq_in (now those of the new weights) and the group maxima. A training loop then
 * moves 22 bytes per parameter and step instead of 26. Contract: ws must hold the factors of the current weights -- left
 * there by pt_group_lasso_norms or by the previous carried step on the same layers array and ws -- so call
 * pt_group_lasso_norms again after anything else changed the weights (zeroing, reconfiguration, a load).
 * reg_sum_next (device, optional) receives Eq. 2's sum for the NEW weights, i.e. the value the next iteration's loss uses.
 * The result is bit for bit pt_group_lasso_sgd_step's when the factors in ws are those pt_group_lasso_norms computes. */
pt_status pt_group_lasso_sgd_step_carried(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers,
                                          const pt_sgd_hparams *hp /*host*/, int32_t with_maxima, double *reg_sum_next,
                                          void *ws, size_t ws_bytes, void *stream);

/* zero_out[k] = (max_{rs,c} |w| < threshold), zero_in[c] = (max_{k,rs} |w| < threshold), strict <, in fp32
 * (Sec. 4.1: threshold 1e-4; Sec. 4.2 / Fig. 4: the absolute maximum of a channel's parameters). A NaN keeps
 * its groups. If zero_in_place != 0 the weights, momentum and shadow of every detected group are set to 0
 * (the group sums of squares are then stale until the next pt_group_lasso_sgd_step recomputes them). */
pt_status pt_find_zero_groups(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers, float threshold,
                              int32_t zero_in_place, void *ws, size_t ws_bytes, void *stream);
/* The same masks without reading the weights: from the group maxima the last pt_group_lasso_sgd_step_carried on these layers
 * (called with with_maxima != 0) and this ws left behind: the maxima of the weights that step wrote; max is order independent,
 * so the masks are bit for bit those of pt_find_zero_groups. Valid only while the weights are unchanged since that step. */
pt_status pt_find_zero_groups_carried(pt_ctx *ctx, const pt_layer *layers /*host*/, int32_t n_layers, float threshold,
                                      int32_t zero_in_place, void *ws, size_t ws_bytes, void *stream);

/* Zero-group detection of ONE weight tensor w[K][RS][C] without any allocation and without a workspace (no counterpart in
 * the paper: it exists for callers that may not allocate). It is for code that cannot call cudaMalloc: a host framework
 * whose caching allocator owns the whole device heap, a latency-critical loop where an allocation's implicit device
 * synchronisation is not acceptable, or a long-running service that must not meet an out-of-memory error in the middle
 * of a reconfiguration. Such callers have no workspace to pass either. Same masks, bit for bit, as
 * pt_find_zero_groups with zero_in_place = 0.
 *   - The scratch is a 256 KiB static device array inside the library, present on every GPU that loads the library until the
 *     process exits. Limit: K + C <= PT_NOALLOC_MAX_GROUPS, otherwise PT_ERR_UNSUPPORTED (use pt_find_zero_groups).
 *   - Calls on one device share that array and it keeps the last call's contents; each call clears what it uses first.
 *     Calls that overlap on the GPU (e.g. on two streams) race: serialise them.
 *   - The first call on a device resolves the array's device address (cudaGetSymbolAddress) with the caller's current device;
 *     make that first call before any stream capture begins. It needs no pt_ctx.
 * w, zero_out (K bytes), zero_in (C bytes): device pointers. */
#define PT_NOALLOC_MAX_GROUPS 65536
pt_status pt_find_zero_groups_noalloc(const float *w, int32_t K, int32_t C, int32_t RS, float threshold,
                                      uint8_t *zero_out, uint8_t *zero_in, void *stream);

/* ------------------------------------------------------------------------------------------
 * Reconfiguration (Sec. 4.2: prune only the intersection of the sparsified channels of adjacent layers;
 * channel union across all convs that share a residual node; surviving training variables kept as is).
 * A channel space is one set of channel indices shared by the convs that write it (as output channels)
 * and read it (as input channels).
 * ------------------------------------------------------------------------------------------ */
typedef struct { int32_t size; uint8_t fixed; } pt_space;      /* fixed: never pruned (the image, the classifier input) */
typedef struct {
    int32_t in_space, out_space;
    float *bn[4];                                              /* gamma, beta, running mean, running var (K floats each) or NULL */
} pt_layer_link;
typedef struct {
    const pt_space *spaces; int32_t n_spaces;                  /* host arrays */
    const pt_layer *layers; const pt_layer_link *links; int32_t n_layers;
} pt_graph;

/* Phase 0. From the zero masks of g's layers, for every space:
 *   keep[j] = fixed  OR  some writer has zero_out[j] = 0  OR  some reader has zero_in[j] = 0
 * new2old (device, sum of space sizes int32; space s starts at the sum of the sizes before it) receives
 * the kept indices in ascending order (entries past the count are -1); new_sizes (HOST, n_spaces) receives the
 * counts. This call synchronises `stream` once to return the counts. A count of 0 is reported, not clamped. */
pt_status pt_reconfigure_plan(pt_ctx *ctx, const pt_graph *g, int32_t *new2old, int32_t *new_sizes /*host*/, void *stream);

/* Phase 1. Gather every layer of old_g into the caller-allocated tensors of new_g:
 *   new.w[k',rs,c'] = old.w[new2old_out[k'], rs, new2old_in[c']]   (same for v and the bf16 shadow, bit for bit)
 *   new.bn[i][k']   = old.bn[i][new2old_out[k']]
 * new_g must have the same topology, and each space size equal to the count pt_reconfigure_plan returned.
 * Layers whose new K or C is 0 are skipped. A new space larger than its planned count makes the gather meet the -1 padding of
 * the map: such entries are skipped (the destination elements stay as they were) and pt_poll_device_status reports
 * PT_ERR_INVALID_ARG.
 * The graphs may hold a subset of a model's layers (the spaces stay whole), so a model can be gathered in parts, e.g. the first
 * layers ahead of the forward pass and the rest beside it. The library keeps the device tables of the last four distinct
 * argument sets; a CUDA graph captured around this call embeds its table's address, which stays valid until four other
 * argument sets have been used with the context. */
pt_status pt_reconfigure(pt_ctx *ctx, const pt_graph *old_g, const int32_t *new2old, const pt_graph *new_g, void *stream);

/* ------------------------------------------------------------------------------------------
 * Channel gating (Sec. 4.2: gating layers on each residual branch gather the dense channels at the branch's entry and scatter
 * them back at the merge point, so that every convolution of the branch works on dense channels only; the paper measured it
 * against channel union and found the tensor reshaping too costly). Tensors are NHWC bf16 with a channel pitch that is a
 * multiple of 8, 16-byte aligned, given as [npix][ld] with npix = N*H*W; all pointers are device pointers.
 * The gradient of the gather is the scatter-add (into the node's gradient) and the gradient of the scatter-add is the
 * gather, so these two calls serve the forward and the backward pass.
 * ------------------------------------------------------------------------------------------ */

/* idx[0..count) = the positions i < n with zero_flags[i] == 0, ascending (the dense channels of a group-mask produced by
 * pt_find_zero_groups); idx[count..n) = -1; *count (device) = their number. One small launch, no synchronisation. */
pt_status pt_dense_channel_list(pt_ctx *ctx, const uint8_t *zero_flags, int32_t n, int32_t *idx, int32_t *count, void *stream);

/* dst[p][j] = src[p][idx[j]] for j < n_sel; dst's pad lanes (n_sel <= j < ld_dst) are written as zeros. src has c_src
 * channels at pitch ld_src. idx (device, n_sel entries, each in [0, c_src)) may be in any order and may repeat.
 * PT_ERR_INVALID_ARG for null pointers, pitches that are not multiples of 8 or smaller than the channel counts, misaligned
 * tensors; PT_ERR_UNSUPPORTED for ld_dst > 4096. An out-of-range index is skipped (the lane reads as zero) and reported by
 * pt_poll_device_status. */
pt_status pt_channel_gather(pt_ctx *ctx, const void *src, int32_t ld_src, int32_t c_src, const int32_t *idx, int32_t n_sel,
                            void *dst, int32_t ld_dst, int64_t npix, void *stream);

/* node_out[p][c] = act(node_in[p][c] + b), c < c_node, where b = branch[p][j] if idx[j] == c for some j < n_sel, else 0;
 * act = max(., 0) if relu, identity otherwise; the sum is formed in fp32 and rounded once to bf16 (nearest even); pad lanes
 * of node_out are written as zeros. node_in may be NULL (read as zeros) and may be the same tensor as node_out. idx holds
 * n_sel DISTINCT channels of the node, in any order.
 * Errors as for pt_channel_gather (PT_ERR_UNSUPPORTED for ld_node > 4096). */
pt_status pt_channel_scatter_add(pt_ctx *ctx, const void *branch, int32_t ld_branch, const int32_t *idx, int32_t n_sel,
                                 const void *node_in, void *node_out, int32_t ld_node, int32_t c_node, int64_t npix,
                                 int32_t relu, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PT_H_ */
