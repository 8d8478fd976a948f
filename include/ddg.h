/*
 * ddg.h — C ABI of the B200 (sm_100a) DDG training-step library.
 *
 * The library runs one iteration of decoupled parallel backpropagation with delayed gradients (DDG):
 * a feed-forward network is cut into K modules of consecutive layers; in iteration t every module k
 * runs its forward pass on the current minibatch (Section 2, Eq. 3), its backward pass on the sample of
 * iteration s = t-K+k with the activations and weights it stored then and the error gradient it received
 * from module k+1 one iteration ago (Section 3.1, Eq. 6-7), and then updates its own weights with that
 * delayed gradient (Section 3.3, Eq. 8-9, Algorithm 1; Algorithm 2 for Adam).  All K modules run
 * concurrently as K CUDA streams on one GPU; activation, weight-version and error-gradient history lives
 * in per-module device ring buffers owned by the context.
 *
 * Conventions for every call
 *   - Pointers are marked "device" or "host".  The caller owns every buffer it passes; the library owns
 *     everything else and frees it in ddg_destroy.  No torch / C++ types cross this boundary.
 *   - Every call returns a ddg_status.  Nothing throws.  After DDG_ERR_CUDA or DDG_ERR_TIMEOUT the context
 *     answers DDG_ERR_STATE until it is destroyed.  ddg_last_error gives a library-owned message.
 *   - The library needs a CUDA device of compute capability 10.0; there is no CPU fallback.
 *   - A context is used from one host thread at a time.
 *
 * Flat parameter order ("canonical order") used by get/set weights and gradients: layers in network order;
 * per layer the conv / FC weight ([Cout][Cin][3][3] or [out][in], row-major), then bias, then BN gamma, then
 * BN beta; a basic block contributes conv1.w, bn1.gamma, bn1.beta, conv2.w, bn2.gamma, bn2.beta (then the projection
 * W_s [Cout][Cin] for DDG_BASIC_BLOCK_PROJ).  Always fp32, whatever the internal storage.
 */
#ifndef DDG_H_
#define DDG_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ddg_ctx ddg_ctx; /* opaque */

typedef enum {
    DDG_OK = 0,
    DDG_ERR_INVALID_ARG = 1, /* NULL pointer, wrong size, index out of range */
    DDG_ERR_BAD_SPEC = 2,    /* layer list / split points do not describe a valid network */
    DDG_ERR_UNSUPPORTED = 3, /* valid, but not implemented (e.g. conv bias) */
    DDG_ERR_OOM = 4,         /* device or host allocation failed */
    DDG_ERR_CUDA = 5,        /* a CUDA call or kernel failed; message in ddg_last_error */
    DDG_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out (reported at the next sync point) */
    DDG_ERR_STATE = 7        /* call not allowed in the context's current state */
} ddg_status;

/* Layer kinds.  The paper only names "ResNet" (Section 5, Table 2); the formulas are the usual ones:
 *  DDG_FC             y = x W^T + b                     (c_in -> c_out, optional bias, optional ReLU)
 *  DDG_CONV3X3        3x3 cross-correlation, pad 1, stride 1|2, no bias (optional ReLU)
 *  DDG_BN             train-mode batch normalisation over (N,H,W), biased variance, eps 1e-5 (optional ReLU)
 *  DDG_RELU           max(x, 0), derivative 0 at 0
 *  DDG_BASIC_BLOCK    out = relu(bn2(conv2(relu(bn1(conv1(x))))) + sc(x)); conv1 has the stride;
 *                     sc = identity, or for stride 2 / wider output x[:, ::2, ::2] zero-padded in channels
 *  DDG_GLOBAL_AVGPOOL mean over H x W
 *  DDG_BASIC_BLOCK_PROJ the same block with a projection shortcut: sc(x) = W_s x, a 1x1 convolution with the
 *                     block's stride, no bias, no batch norm (any c_in -> c_out)  */
typedef enum {
    DDG_FC = 0, DDG_CONV3X3 = 1, DDG_BN = 2, DDG_RELU = 3, DDG_BASIC_BLOCK = 4, DDG_GLOBAL_AVGPOOL = 5,
    DDG_BASIC_BLOCK_PROJ = 6
} ddg_layer_kind;

typedef struct {
    int kind;       /* ddg_layer_kind */
    int c_in;       /* input channels / features */
    int c_out;      /* output channels / features (= c_in for BN, RELU, GLOBAL_AVGPOOL) */
    int stride;     /* 1 or 2 (conv, block); ignored otherwise */
    int has_bias;   /* FC only */
    int relu_after; /* FC, CONV3X3, BN: apply ReLU to the output */
} ddg_layer;

typedef enum { DDG_OPT_SGD = 0, DDG_OPT_ADAM = 1 } ddg_opt_kind;

/* Optimiser.  SGD: d = g + weight_decay*w; v = momentum*v + d; w -= lr*v (Eq. 9 when momentum = decay = 0).
 * Adam: Algorithm 2, bias correction with the global iteration count.  A module whose delayed gradient does
 * not exist yet (t-K+k < 0, Eq. 8) is left untouched in that iteration. */
typedef struct {
    int kind; /* ddg_opt_kind */
    float lr, momentum, weight_decay, beta1, beta2, eps;
} ddg_opt;

typedef enum { DDG_FP32 = 0, DDG_BF16 = 1 } ddg_precision;

typedef struct {
    int precision;  /* DDG_FP32: everything fp32.  DDG_BF16: activations, error gradients and the weight
                       versions the sweeps read are bf16; accumulation, statistics, loss, parameter
                       gradients, master weights and optimiser state are fp32. */
    int batch;      /* B */
    int in_c, in_h, in_w;   /* input is [B][in_c][in_h][in_w] fp32 (use in_h = in_w = 1 for an MLP) */
    int num_classes;
    unsigned long long seed; /* seed of the library's own He-normal initialisation */
    int use_graph;  /* 1: replay the steady-state iteration from CUDA graphs (one per ring phase, module and sweep),
                       all recorded at the first iteration in which every module has a delayed gradient (t = K-1) */
    int debug_checks; /* 1: every activation slot, weight-version slot and error-gradient buffer carries a stamp of the
                       iteration (sample) that wrote it, set and compared on the device by one small kernel per sweep;
                       a slot that is not the one the delay pattern of Eq. 6-8 asks for raises an error word, and the
                       next sync point returns DDG_ERR_STATE.  Three extra launches per module and iteration. */
    void *const *streams; /* host array of K cudaStream_t to run the modules on, or NULL (library creates K) */
    int separate_bn_sums; /* 0 (default): the batch-norm sums are taken in the epilogue of the tensor-core convolution
                       that produces the tensor.  1: separate reduction kernels (same sums, other summation order). */
    int fuse_bn_apply; /* Where the normalise + ReLU pass of a batch norm runs.  0 (default): element-wise kernels of
                       their own.  1: inside a residual block, the first batch norm's pass runs on the operand path of
                       the second convolution (transform warps between the TMA box and the MMAs).  2: also the block's
                       closing pass relu(bn2(y2) + x), on the operand path of the NEXT block's first convolution.  Same
                       values bit for bit, 8 % / 15 % fewer launches - and, at the sizes measured (ResNet-110, batch
                       128), a slower iteration: the extra warps push the convolution CTA past half an SM's registers,
                       so that kernels of two module streams no longer share an SM.  Kept as an option. */
    int bn_fold; /* Who adds up the per-CTA partial sums a convolution epilogue leaves for the batch norm behind it.
                       1: the convolution's CTA that finishes last (ticket counter; costs that kernel ~4 us of serial
                       tail, but only one CTA, which leaves the rest of the GPU to the other module streams).  2: the
                       element-wise pass that consumes the sums, every CTA for itself (no tail; ~1.5 us more in every CTA
                       of that pass).  0 (default): the library's policy: 2 for K = 1, 1 when several module streams
                       share the GPU.  Both orders are fixed; the two settings differ in the last bits. */
    int launch_overlap; /* programmatic dependent launch (the next kernel of a stream is placed while the previous one
                       still runs).  0 (default): the library's policy: every kernel when K = 1; with several module
                       streams only the forward / input-gradient convolutions.  1: never.  2: every kernel. */
    int time_pieces; /* 1: bracket each module's forward sweep and its backward sweep + update with timing events on
                       the module's stream (two extra event records per piece), read back by ddg_piece_times. */
} ddg_cfg;

/* Build a context: validates the network (Section 2: L layers; Section 3: K groups of consecutive layers,
 * `split_after` = the K-1 strictly increasing 0-based layer indices after which a new module starts; NULL when
 * K = 1), allocates all device state, initialises the weights from cfg->seed.  host pointers only. */
ddg_status ddg_create(const ddg_layer *layers, int n_layers, const int *split_after, int K,
                      const ddg_opt *opt, const ddg_cfg *cfg, ddg_ctx **out);

/* One DDG iteration (Algorithm 1 / 2 with the sweeps of Eq. 3 and Eq. 6-7).
 *   x_dev: device, fp32, [B][in_c][in_h][in_w]; y_dev: device, int32 labels [B].
 *   loss_host: host, nullable.  Non-NULL: the call waits until this iteration's forward sweep has produced the
 *   loss and writes the mean cross-entropy of this iteration's minibatch; the backward sweeps and updates of the
 *   iteration may still be running when it returns (they only feed later iterations; ddg_sync, ddg_get_weights
 *   and ddg_get_grads wait for them).  NULL: the call only enqueues work; x_dev / y_dev must stay valid until
 *   ddg_sync (or a later call with loss_host != NULL) returns.  The inputs are copied into library-owned staging
 *   buffers before the forward sweep reads them, so a call that returned a loss is done with x_dev / y_dev. */
ddg_status ddg_step(ddg_ctx *ctx, const float *x_dev, const int *y_dev, float *loss_host);

/* The same iteration with host inputs: copies x_host / y_host (host, same shapes) to the device on the
 * context's first stream, runs ddg_step and, when loss_host is non-NULL, waits and returns the loss. */
ddg_status ddg_step_host(ddg_ctx *ctx, const float *x_host, const int *y_host, float *loss_host);

/* ddg_step_host without the host waiting for the device in every iteration: the call enqueues iteration t (input
 * copies, sweeps, updates) and the read-back of its loss, and hands out the loss of iteration t-1, which completed while
 * the host was preparing this call (NaN at the first call).  The host therefore runs one iteration ahead of the losses it
 * logs, and consecutive iterations overlap on the device exactly as with loss_host = NULL.  loss_prev_host: host,
 * nullable.  x_host / y_host of iteration t must stay valid until the call for iteration t+1 has returned a loss (or
 * ddg_sync / ddg_pipelined_loss returned).  ddg_pipelined_loss waits for the most recent iteration's loss and returns it
 * (the one no later call will hand out).  Do not mix with loss-returning ddg_step / ddg_step_host calls in between. */
ddg_status ddg_step_host_pipelined(ddg_ctx *ctx, const float *x_host, const int *y_host, float *loss_prev_host);
ddg_status ddg_pipelined_loss(ddg_ctx *ctx, float *loss_host);

/* The stepsize sequence {gamma_t} of Algorithm 1 is driven by the caller. */
ddg_status ddg_set_lr(ddg_ctx *ctx, float lr);

/* n: total parameter count; per_module: host array of K counts (nullable). */
ddg_status ddg_param_count(const ddg_ctx *ctx, size_t *n, size_t *per_module);

/* Copy the fp32 master weights out / in, canonical order, n = total parameter count.  dst/src is a device
 * pointer when *_on_device != 0, else host.  Both calls wait for all enqueued work first.  ddg_set_weights is
 * only allowed before the first step (afterwards: DDG_ERR_STATE). */
ddg_status ddg_get_weights(ddg_ctx *ctx, float *dst, size_t n, int dst_on_device);
ddg_status ddg_set_weights(ddg_ctx *ctx, const float *src, size_t n, int src_on_device);

/* The delayed gradient g_k^t (Eq. 8) that module k (0-based) applied in the last iteration, canonical order
 * of that module's slice, n = per_module[k].  *sample (nullable) receives s = t-K+k (1-based k), or -1 with a
 * zero-filled dst while the module is in warm-up. */
ddg_status ddg_get_grads(ddg_ctx *ctx, int k, float *dst, size_t n, int dst_on_device, long *sample);

/* Device address of the last iteration's loss (fp32 scalar), for consumers that stay on the device. */
ddg_status ddg_get_loss_dev(ddg_ctx *ctx, const float **loss_dev);

/* Number of the library's kernel launches the last ddg_step issued (graph replays count their kernel nodes). */
ddg_status ddg_last_step_launches(const ddg_ctx *ctx, long *launches);

/* Device time of the pieces of the last iteration (contexts created with time_pieces): fwd_ms[k] = the forward sweep
 * of module k+1 (Eq. 3 over G(k+1)), bwd_ms[k] = its backward sweep and update (Eq. 6-9), each from the moment the
 * piece's first kernel could start on the module's stream to the end of its last, in milliseconds; the pieces of
 * different modules overlap in time and share the GPU, which is what the method's cost model (forward in sequence,
 * backward sweeps side by side) is about.  Host arrays of K floats; waits for the K streams.  Each piece is also an
 * NVTX range ("F1", "B1+U1", ...) for a timeline tool. */
ddg_status ddg_piece_times(ddg_ctx *ctx, float *fwd_ms, float *bwd_ms);

/* Wait for all K streams; surfaces deferred device-side errors. */
ddg_status ddg_sync(ddg_ctx *ctx);

/* Exact checkpoint / resume.  A DDG run has state in flight between iterations: module k still owes the backward sweeps
 * of the K-k most recent samples, so besides the master weights and optimiser state a checkpoint holds every module's
 * activation ring and weight-version ring (Section 3.1: h^s and w^s of the pending samples), the error gradients handed
 * over but not yet consumed (Eq. 7), and the iteration count t.  ddg_state_bytes gives the size; ddg_save_state waits
 * for all enqueued work and copies the state into a host buffer of that size; ddg_load_state restores it into a context
 * created with the same network, split, precision, batch and optimiser kind (anything else: DDG_ERR_INVALID_ARG), after
 * which the run continues bit for bit as the saved one would have (same kernels, fixed summation orders).  The step
 * size is the caller's (ddg_set_lr) and is not part of the state. */
ddg_status ddg_state_bytes(const ddg_ctx *ctx, size_t *bytes);
ddg_status ddg_save_state(ddg_ctx *ctx, void *dst_host, size_t bytes);
ddg_status ddg_load_state(ddg_ctx *ctx, const void *src_host, size_t bytes);

/* Diagnostics (no counterpart in the paper).  Every device-side wait in the library is bounded: a wait that runs out
 * raises the context's error word instead of hanging, the kernel returns, and the next sync point (ddg_sync,
 * ddg_get_weights, ddg_get_grads, ddg_step with a loss) answers DDG_ERR_TIMEOUT, after which the context is in
 * DDG_ERR_STATE.  ddg_debug_wait_timeout exercises exactly that path without a stuck pipeline: it enqueues, on the
 * first module's stream, a one-CTA kernel that waits with a limit of `polls` polls (a few hundred nanoseconds each) on
 * a barrier nothing arrives on, gives up and returns.
 * ddg_debug_shift_stamps (contexts created with debug_checks) adds `delta` to the iteration counter module k's forward
 * sweep stamps its ring slots with, as an indexing error of the rings would: the next sweeps see stamps that do not
 * match and the next sync point answers DDG_ERR_STATE. */
ddg_status ddg_debug_wait_timeout(ddg_ctx *ctx, unsigned polls);
ddg_status ddg_debug_shift_stamps(ddg_ctx *ctx, int k, long delta);

const char *ddg_last_error(const ddg_ctx *ctx); /* ctx may be NULL: error of the last failed ddg_create */
void ddg_destroy(ddg_ctx *ctx);

/* ---------------------------------------------------------------------------------------------------------
 * Single-kernel entry points, for per-kernel parity tests and roofline measurements.  All pointers are device
 * pointers; tensors are NHWC ([B][H][W][C]) in the precision given (fp32 or bf16 elements); weights are in
 * canonical [Cout][Cin][3][3] order in the same element type; parameter gradients and statistics are fp32.
 * `stream` is a cudaStream_t (NULL = default stream).  The calls only enqueue.
 * --------------------------------------------------------------------------------------------------------- */

/* 1 when the bf16 forward / input-gradient convolution of this shape runs on the tensor-core (tcgen05) kernels,
 * 2 when the weight gradient does too (3 = both), 0 when the CUDA-core kernels take it.  Needs a CUDA device. */
int ddg_tensor_core_path(int B, int H, int W, int Cin, int Cout, int stride);

/* y = conv3x3(x, w), pad 1 (layer forward, Eq. 3).  x [B][H][W][Cin], y [B][Ho][Wo][Cout], Ho = (H-1)/stride+1. */
ddg_status ddg_conv3x3_fwd(int precision, const void *x, const void *w, void *y, int B, int H, int W, int Cin,
                           int Cout, int stride, void *stream);
/* dx = conv3x3 input gradient (Eq. 5 / Eq. 7).  dy [B][Ho][Wo][Cout], dx [B][H][W][Cin]. */
ddg_status ddg_conv3x3_dgrad(int precision, const void *dy, const void *w, void *dx, int B, int H, int W, int Cin,
                             int Cout, int stride, void *stream);
/* The tensor-core convolution reads its filter from a pre-arranged image (what the training step keeps per weight
 * version, refreshed by the optimiser update): ddg_conv3x3_packed_bytes gives its size for a stride-1 C->C bf16
 * convolution on [B][H][W][C] (0 when the tensor-core path does not take the shape), ddg_conv3x3_pack writes it from a
 * canonical bf16 filter, ddg_conv3x3_packed runs the forward (dgrad = 0) or input-gradient (dgrad = 1) convolution
 * with it (Eq. 3 / Eq. 5).  All pointers device. */
size_t ddg_conv3x3_packed_bytes(int B, int H, int W, int C);
ddg_status ddg_conv3x3_pack(const void *w, void *packed, int C, void *stream);
ddg_status ddg_conv3x3_packed(int dgrad, const void *src, const void *w, const void *packed, void *dst, int B, int H,
                              int W, int C, void *stream);

/* The fused forms the training step launches on the tensor-core path (bf16, stride 1, C -> C channels with
 * ddg_tensor_core_path(...) & 1; other shapes: DDG_ERR_UNSUPPORTED).  packed: nullable filter image as above.
 * scratch: device fp32, ddg_conv3x3_fused_scratch_elems(B, H, W, C) elements, contents undefined on entry and exit.
 *
 * ddg_conv3x3_fwd_stats: y = conv3x3(x, w) (Eq. 3) and, from the values as stored (bf16), the statistics of the batch
 * norm that follows: mean[c] and invstd[c] = 1 / sqrt(biased variance + 1e-5) over (B, H, W), fp32 [C], taken in the
 * convolution's epilogue (per-CTA partial sums, folded in a fixed order by the CTA that finishes last).
 *
 * ddg_conv3x3_dgrad_fused: dx = input gradient of conv3x3 given dy (Eq. 5 / Eq. 7), plus
 *   - res_dout, res_out (both or neither; [B][H][W][C]): the gradient of an identity shortcut,
 *     dx += res_dout * [res_out > 0] (the residual block's output ReLU and add, differentiated);
 *   - bn_mask, bn_x, bn_mean, bn_invstd, dbeta, dgamma (all or none): the two reductions of the batch-norm backward
 *     pass whose incoming gradient is dx: with dz = dx(as stored) * [bn_mask > 0] and xhat = (bn_x - mean) * invstd,
 *     dbeta[c] = sum dz, dgamma[c] = sum dz * xhat (fp32 [C]). */
size_t ddg_conv3x3_fused_scratch_elems(int B, int H, int W, int C);
ddg_status ddg_conv3x3_fwd_stats(const void *x, const void *w, const void *packed, void *y, float *mean, float *invstd,
                                 float *scratch, int B, int H, int W, int C, void *stream);
/* ddg_conv3x3_fwd_stats for a scratch whose first 128 bytes are already zero (every call of either form leaves them
 * zero): no clearing memset in front of the kernel, so that consecutive launches chain exactly as they do inside the
 * training step.  For timing the kernel in the form the step launches it. */
ddg_status ddg_conv3x3_fwd_stats_prepared(const void *x, const void *w, const void *packed, void *y, float *mean,
                                          float *invstd, float *scratch, int B, int H, int W, int C, void *stream);
/* ddg_conv3x3_fwd_stats_prepared with the launch plan the training step uses while K > 1 module streams share the GPU
 * (fewer CTAs with at least two tiles per pipeline, the programmatic launch attribute as on the step's convolutions):
 * the same y bit for bit, the statistics from a different number of per-CTA partial sums.  For checking and timing the
 * kernel in exactly the form a DDG step with several modules launches it. */
ddg_status ddg_conv3x3_fwd_stats_shared(const void *x, const void *w, const void *packed, void *y, float *mean,
                                        float *invstd, float *scratch, int B, int H, int W, int C, void *stream);
ddg_status ddg_conv3x3_dgrad_fused(const void *dy, const void *w, const void *packed, void *dx, const void *res_dout,
                                   const void *res_out, const void *bn_mask, const void *bn_x, const float *bn_mean,
                                   const float *bn_invstd, float *dbeta, float *dgamma, float *scratch, int B, int H,
                                   int W, int C, void *stream);
/* ddg_conv3x3_dgrad_fused under the same shared-GPU launch plan: the same dx bit for bit, the sums from a different
 * number of per-CTA partial sums. */
ddg_status ddg_conv3x3_dgrad_fused_shared(const void *dy, const void *w, const void *packed, void *dx,
                                          const void *res_dout, const void *res_out, const void *bn_mask, const void *bn_x,
                                          const float *bn_mean, const float *bn_invstd, float *dbeta, float *dgamma,
                                          float *scratch, int B, int H, int W, int C, void *stream);
/* The same two fused forms as a single stream launches them when it has the GPU to itself (K = 1): the convolution only
 * leaves the per-CTA partial sums of its epilogue, part [*n_part_host][2C] fp32 (device, at least
 * ddg_conv3x3_fused_scratch_elems floats; *n_part_host, host, receives the number of rows = CTAs of the launch), and
 * the element-wise batch-norm pass that consumes the sums adds the rows up itself, every CTA the same rows in the same
 * fixed order: no ticket counter and no serial tail in the convolution.
 *   ddg_conv3x3_fwd_partials    y = conv3x3(x, w); partials of (sum y, sum y^2) over the values as stored.
 *   ddg_bn_fwd_partials         out = [relu](gamma * (y - mean) * invstd + beta [+ res]) with mean / invstd computed from
 *                               the partials and written to mean / invstd (fp32 [C]).
 *   ddg_conv3x3_dgrad_partials  as ddg_conv3x3_dgrad_fused with the batch-norm sums left as partials of (sum dz,
 *                               sum dz * xhat); bn_* must be given.
 *   ddg_bn_bwd_partials         dx = gamma * invstd * (dz - dbeta / n - xhat * dgamma / n), dz = dout * [out > 0] (relu),
 *                               with dbeta / dgamma computed from the partials and written out.
 * bf16, C in {16, 32, 64} (DDG_ERR_UNSUPPORTED otherwise). */
ddg_status ddg_conv3x3_fwd_partials(const void *x, const void *w, const void *packed, void *y, float *part,
                                    int *n_part_host, int B, int H, int W, int C, void *stream);
ddg_status ddg_bn_fwd_partials(const void *y, const void *gamma, const void *beta, const void *res, void *out,
                               const float *part, int n_part, float *mean, float *invstd, int B, int HW, int C, int relu,
                               void *stream);
ddg_status ddg_conv3x3_dgrad_partials(const void *dy, const void *w, const void *packed, void *dx, const void *res_dout,
                                      const void *res_out, const void *bn_mask, const void *bn_x, const float *bn_mean,
                                      const float *bn_invstd, float *part, int *n_part_host, int B, int H, int W, int C,
                                      void *stream);
ddg_status ddg_bn_bwd_partials(const void *dout, const void *out, const void *x, const void *gamma, const float *mean,
                               const float *invstd, void *dx, float *dgamma, float *dbeta, const float *part, int n_part,
                               int B, int HW, int C, int relu, void *stream);

/* ddg_conv3x3_bnrelu_fwd_stats: the second convolution of a residual block as the training step launches it.  x is the
 * RAW output of the first convolution; the kernel applies that convolution's batch norm and ReLU on its own operand
 * path, a = relu(gamma * (x - mean_in) * invstd_in + beta) rounded to bf16 (gamma, beta bf16 [C]; mean_in, invstd_in
 * fp32 [C]), stores a to a_out ([B][H][W][C], what the backward sweep reads) and computes y = conv3x3(a, w) with the
 * statistics of y as ddg_conv3x3_fwd_stats does (Eq. 3 for batch norm -> ReLU -> convolution).  res (nullable, same
 * shape as x): the batch norm closes a residual block and a = relu(bn(x) + res), which is how the first convolution of
 * the NEXT block consumes the previous block's output. */
ddg_status ddg_conv3x3_bnrelu_fwd_stats(const void *x, const void *res, const void *gamma, const void *beta,
                                        const float *mean_in, const float *invstd_in, void *a_out, const void *w,
                                        const void *packed, void *y,
                                        float *mean, float *invstd, float *scratch, int B, int H, int W, int C,
                                        void *stream);
/* Input gradient of the stride-2 convolution of a down-sampling block (Cin -> 2 Cin, bf16, tensor-core path only) with
 * the gradient of the block's parameter-free shortcut added: dx[n][2j][2i][c] += res_dout[n][j][i][c] *
 * [res_out[n][j][i][c] > 0] for c < Cin (the shortcut reads every second pixel of every second row and pads the
 * channels with zeros).  dy, res_dout, res_out: [B][H/2][W/2][2 Cin]; dx: [B][H][W][Cin].  res_* nullable (both). */
ddg_status ddg_conv3x3_s2_dgrad_shortcut(const void *dy, const void *w, void *dx, const void *res_dout,
                                         const void *res_out, int B, int H, int W, int Cin, void *stream);

/* The 1x1 convolution of a projection shortcut (Eq. 3 and Eq. 4-5 for y = W_s x with a spatial stride, no bias).
 * x [B][H][W][Cin], w [Cout][Cin], y / dout / out [B][Ho][Wo][Cout] with Ho = (H-1)/stride+1, all in the precision's
 * element type; Cin * Cout <= 4096.
 *   ddg_conv1x1_fwd        y = W_s x.
 *   ddg_conv1x1_dgrad_add  dx[n][s*h][s*w][:] += W_s^T dz[n][h][w][:], dz = dout * [out > 0] (out nullable: dz = dout);
 *                          dx is read and written (the 3x3 convolution's input gradient is already in it).
 *   ddg_conv1x1_wgrad      dw[co][ci] = sum dz[p][co] x[s*p][ci], fp32; scratch: ddg_conv1x1_wgrad_scratch_elems floats. */
ddg_status ddg_conv1x1_fwd(int precision, const void *x, const void *w, void *y, int B, int H, int W, int Cin, int Cout,
                           int stride, void *stream);
ddg_status ddg_conv1x1_dgrad_add(int precision, const void *dout, const void *out, const void *w, void *dx, int B, int H,
                                 int W, int Cin, int Cout, int stride, void *stream);
size_t ddg_conv1x1_wgrad_scratch_elems(int Cin, int Cout);
ddg_status ddg_conv1x1_wgrad(int precision, const void *x, const void *dout, const void *out, float *dw, float *scratch,
                             int B, int H, int W, int Cin, int Cout, int stride, void *stream);

/* dw = conv3x3 weight gradient (Eq. 4 / Eq. 6), fp32 [Cout][Cin][3][3].  scratch: device, fp32,
 * ddg_conv3x3_wgrad_scratch_elems(...) elements, contents undefined on entry and exit. */
size_t ddg_conv3x3_wgrad_scratch_elems(int B, int H, int W, int Cin, int Cout, int stride);
ddg_status ddg_conv3x3_wgrad(int precision, const void *x, const void *dy, float *dw, float *scratch, int B, int H,
                             int W, int Cin, int Cout, int stride, void *stream);
/* Fully connected layer h = x W^T + b (Eq. 3) and its backward pass (Eq. 4-5 / Eq. 6-7).  x [B][in], W [out][in] and
 * bias [out] (nullable) in the precision's element type; y and dy [B][out] are fp32 when out_f32 != 0 (the network's
 * last layer: logits and the loss gradient), else the element type; dW [out][in] and db [out] (nullable) fp32; dx
 * [B][in] (nullable) in the element type.  With relu != 0 the forward output is max(., 0) and the backward pass masks dy
 * with [y > 0] (y = forward output).  In bf16 the layer runs on the tensor cores (tcgen05 MMAs fed by TMA) when
 * ddg_fc_tensor_core_path(B, in, out) is 1 and x, W, dx, dW start on 16-byte boundaries; otherwise on CUDA cores. */
int ddg_fc_tensor_core_path(int B, int in, int out);
ddg_status ddg_fc_fwd(int precision, const void *x, const void *W, const void *bias, void *y, int B, int in, int out,
                      int relu, int out_f32, void *stream);
ddg_status ddg_fc_bwd(int precision, const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW,
                      float *db, int B, int in, int out, int relu, int out_f32, void *stream);

/* Batch-norm forward, fused: statistics over (B,H,W), then y = [relu](gamma*xhat + beta [+ res]).  res nullable
 * (same shape as y).  gamma/beta in the activation element type; mean/invstd fp32 [C] outputs; scratch fp32,
 * ddg_bn_scratch_elems(C) elements. */
size_t ddg_bn_scratch_elems(int C);
ddg_status ddg_bn_fwd(int precision, const void *x, const void *gamma, const void *beta, const void *res, void *y,
                      float *mean, float *invstd, float *scratch, int B, int HW, int C, int relu, void *stream);
/* The same operation as ddg_bn_fwd without the scratch argument, for callers that cannot allocate device memory
 * (code running inside someone else's memory pool, latency-critical loops that must avoid cudaMalloc's implicit
 * synchronisation, processes whose device memory is budgeted up front).  The paper has no counterpart: this is a
 * deployment convenience.  The scratch lives in a fixed array inside the library image (about 592 KiB per GPU that
 * loads the library, held until the process exits), which limits the call to C <= 64; larger C returns
 * DDG_ERR_UNSUPPORTED with a message in ddg_last_error(NULL).  The call itself allocates nothing (no cudaMalloc,
 * cudaFree or allocating library routine).  The first call on each device looks up the array's device address
 * (with that device current): make that first call before any stream capture.  All calls share the one array and
 * it keeps the previous call's contents (the call clears the part that must start at zero), so two calls that
 * overlap on the GPU - different streams, or the same call from two threads - race; serialise them. */
ddg_status ddg_bn_fwd_noalloc(int precision, const void *x, const void *gamma, const void *beta, const void *res,
                              void *y, float *mean, float *invstd, int B, int HW, int C, int relu, void *stream);

/* Batch-norm backward: dz = dout * [out > 0] when relu != 0 (out = forward output), else dout;
 * dgamma = sum dz*xhat, dbeta = sum dz, dx = gamma*invstd*(dz - dbeta/n - xhat*dgamma/n). */
ddg_status ddg_bn_bwd(int precision, const void *dout, const void *out, const void *x, const void *gamma,
                      const float *mean, const float *invstd, void *dx, float *dgamma, float *dbeta, float *scratch,
                      int B, int HW, int C, int relu, void *stream);
/* The reduction half of ddg_bn_bwd alone (dgamma, dbeta), for timing the kernel by itself.  Same arguments. */
ddg_status ddg_bn_bwd_reduce(int precision, const void *dout, const void *out, const void *x, const float *mean,
                             const float *invstd, float *dgamma, float *dbeta, float *scratch, int B, int HW, int C,
                             int relu, void *stream);

/* Fused SGD update over n parameters (Eq. 9 with momentum and weight decay): d = g + wd*w; v = mu*v + d;
 * w -= lr*v; w_version = cast(w).  w, v, g fp32; w_version in the precision's element type. */
ddg_status ddg_sgd_update(int precision, float *w, float *v, const float *g, void *w_version, size_t n, float lr,
                          float momentum, float weight_decay, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DDG_H_ */
