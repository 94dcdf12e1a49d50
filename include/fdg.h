/*
 * libfdg -- fully decoupled training with delayed gradients (FDG) on one B200.
 *
 * The network (a residual CNN) is split into K modules; each module is a worker
 * on its own CUDA stream.  One call of fdg_step() is one iteration t of
 * Algorithm I of the FDG paper for every module k = 1..K:
 *
 *   forward   (Section 3.1 "forward")   module k forwards batch t-k+1, the output
 *                                       module k-1 produced in iteration t-1;
 *   backward  (Section 3.1 "backward",  module k back-propagates batch t-2K+k+1 from
 *              Eq. 10, Eq. 15)          the gradient module k+1 produced in iteration
 *                                       t-1, multiplied by the shrinking factor beta
 *                                       (modules k < K only), through the activations
 *                                       saved by the forward of that same batch;
 *   update    (Eq. 11)                  SGD with momentum and weight decay on the
 *                                       module's own parameters;
 *   handoff   (Section 3.1              output activation -> module k+1, input gradient
 *              "communication")         -> module k-1, both consumed in iteration t+1.
 *
 * Conventions
 *   - Every function returns an fdg_status; none throws, aborts or exits.
 *   - "dev" pointers are device pointers on the device that was current at
 *     fdg_create(); "host or device" pointers may be either (unified addressing).
 *   - The library allocates no device memory: the caller passes one workspace of
 *     fdg_workspace_bytes() bytes (256-byte aligned) that the context owns until
 *     fdg_destroy().
 *   - Activations are NHWC; convolution weights are [C_out][R][S][C_in].
 *   - Modules and blocks are numbered from 1 as in the paper.
 *   - Threading: a context is used by one host thread at a time (its calls enqueue work on its streams and
 *     update host-side bookkeeping without a lock); different contexts may be used from different threads.
 *
 * Flat parameter layout of a module (fp32), the order fdg_param_layout() reports:
 *   units in network order: stem (module 1), residual blocks, head (module K);
 *   FDG_RESNET_6N2: stem  = conv.w, bn.gamma, bn.beta
 *                   block = conv1.w, bn1.gamma, bn1.beta, conv2.w, bn2.gamma, bn2.beta
 *                           [, sc.w (1x1), scbn.gamma, scbn.beta  when the shape changes]
 *                   head  = fc.w [classes][features], fc.b
 *   FDG_WRN:        stem  = conv.w
 *                   block = bn1.gamma, bn1.beta, conv1.w, bn2.gamma, bn2.beta, conv2.w
 *                           [, sc.w (1x1)  when the shape changes]
 *                   head  = bn.gamma, bn.beta, fc.w, fc.b
 */
#ifndef FDG_H_
#define FDG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fdg_ctx fdg_ctx;            /* opaque; created by fdg_create, freed by fdg_destroy */
typedef void* fdg_stream;                  /* a cudaStream_t, passed as a plain pointer (NULL = default stream) */

typedef enum {
  FDG_OK = 0,
  FDG_ERR_INVALID_ARG = 1,
  FDG_ERR_WORKSPACE_TOO_SMALL = 2,
  FDG_ERR_CUDA = 3,
  FDG_ERR_STATE = 4,
  FDG_ERR_UNSUPPORTED = 5,
  FDG_ERR_NONFINITE = 6,
  FDG_ERR_TIMEOUT = 7
} fdg_status;

enum { FDG_RESNET_6N2 = 0, FDG_WRN = 1 };                 /* fdg_arch.family   */
enum { FDG_SHORTCUT_PROJECTION = 0, FDG_SHORTCUT_ZERO_PAD = 1 };   /* fdg_arch.shortcut */
enum { FDG_BACKWARD_FIRST = 0, FDG_FORWARD_FIRST = 1 };   /* fdg_config.order  */
enum { FDG_STASHED = 0, FDG_CURRENT = 1 };                /* fdg_config.weight_reading */
enum { FDG_FP32_CUDACORE = 0, FDG_BF16_TC = 1 };          /* fdg_config.precision */
enum { FDG_PARAM_CONV = 0, FDG_PARAM_BN_GAMMA = 1, FDG_PARAM_BN_BETA = 2,
       FDG_PARAM_FC_W = 3, FDG_PARAM_FC_B = 4 };          /* fdg_param_entry.kind */

/* The network: a stem convolution, n_stages stages of residual blocks (stride 2 at the first block of every
 * stage but the first), a classifier.  The paper defines no architecture of its own; these are the networks of
 * its tables: the 6n+2 networks (3 stages of n blocks at 16/32/64), the CIFAR ResNet-18 (4 stages of 2 blocks at
 * 64/128/256/512), WRN-28-10 (3 stages of 4 pre-activation blocks at 160/320/640). */
typedef struct {
  int family;            /* FDG_RESNET_6N2 (post-activation blocks) | FDG_WRN (pre-activation blocks) */
  int n_stages;          /* 1..4 */
  int blocks[4];         /* residual blocks per stage (ResNet-110: 18,18,18; WRN-28-10: 4,4,4) */
  int widths[4];         /* channels per stage */
  int stem_width;        /* output channels of the stem convolution */
  int shortcut;          /* where a block changes the shape: FDG_SHORTCUT_PROJECTION = 1x1 convolution (+ BN in the
                            post-activation family); FDG_SHORTCUT_ZERO_PAD (FDG_RESNET_6N2 only) = the input at every
                            second pixel with (C_out - C_in)/2 zero channels in front and behind, no parameters */
  int in_h, in_w, in_c;  /* image size; in_h and in_w multiples of 2^(n_stages-1), at least 4 */
  int num_classes;
  int batch;
  float bn_eps;
} fdg_arch;

/* The inputs Algorithm I asks for (a learning rate per iteration, the number of modules K, the shrinking
 * factor beta), plus the optimiser constants of the experiments section. */
typedef struct {
  int K;                          /* number of modules, >= 1 */
  const int* split_after_block;   /* K-1 ascending block indices in [1, total blocks - 1]: module k ends after that block */
  float beta;                     /* shrinking factor, 0 < beta <= 1 (Eq. 15) */
  float lr, momentum, weight_decay;
  int order;                      /* FDG_BACKWARD_FIRST = Algorithm I; FDG_FORWARD_FIRST = Appendix A variant */
  int weight_reading;             /* FDG_STASHED: delayed backward uses the weights of that batch's forward (Eq. 10) */
  int precision;                  /* FDG_FP32_CUDACORE: fp32 storage and arithmetic;
                                     FDG_BF16_TC: bf16 activations/weights for the convolutions, fp32 accumulation,
                                     fp32 master weights, statistics and loss */
  int serial;                     /* 1 = run all modules on the caller's stream in order (debug) */
  int graphs;                     /* 1 = once the pipeline is full, record each iteration into a CUDA graph (one per
                                     phase of the rings, a power of two >= 2K of them) and replay it from then on.
                                     Iterations then follow one another on the caller's stream while the K modules of
                                     one iteration still run side by side; the ring buffers are rounded up to powers
                                     of two, so the workspace grows.  Results are identical to graphs = 0.  With
                                     serial = 1 the recorded graph is a single chain.  fdg_profile_enable is refused
                                     (FDG_ERR_STATE). */
} fdg_config;

typedef struct {            /* one tensor of a module's flat parameter vector */
  int kind;                 /* FDG_PARAM_* */
  int unit;                 /* 0 = stem, b = residual block b (1-based), -1 = head */
  int dims[4];              /* conv: C_out,R,S,C_in; fc_w: classes,features,1,1; vectors: n,1,1,1 */
  size_t offset;            /* first element in the flat vector */
  size_t count;             /* number of elements */
} fdg_param_entry;

typedef struct {            /* one row of the schedule log: what module k did in iteration t */
  int64_t t;                /* iteration, from 1 */
  int32_t k;                /* module, from 1 */
  int64_t tau_f;            /* batch forwarded (t-k+1), or -1 while the pipeline fills */
  int64_t tau_b;            /* batch back-propagated (t-2K+k+1), or -1 */
  int64_t ver_f;            /* number of updates the weights used by the forward had received, or -1 */
  int64_t ver_b;            /* same for the weights used by the backward, or -1 */
  int32_t slot_f;           /* activation-FIFO slot written by the forward, or -1 */
  int32_t slot_b;           /* activation-FIFO slot read by the backward, or -1 */
} fdg_sched_entry;

/* Bytes of device workspace fdg_create() needs for this network and configuration.
 * Errors: FDG_ERR_INVALID_ARG (null pointer, bad sizes or split points),
 * FDG_ERR_UNSUPPORTED (a shape the kernels do not cover). */
fdg_status fdg_workspace_bytes(const fdg_arch* arch, const fdg_config* cfg, size_t* out_bytes);

/* Builds a context in `dev_workspace` (caller-owned, 256-byte aligned, `bytes` >=
 * fdg_workspace_bytes; must outlive the context).  `streams` is an array of K
 * cudaStream_t owned by the caller, or NULL to let the library create its own.
 * Parameters start at zero: call fdg_set_params for every module before stepping.
 * The iteration counter starts at t = 0 with an empty pipeline.  Blocks the host
 * until the workspace has been cleared. */
fdg_status fdg_create(const fdg_arch* arch, const fdg_config* cfg, void* dev_workspace, size_t bytes,
                      const fdg_stream* streams, fdg_ctx** out_ctx);

/* Waits for all enqueued work, releases streams/events the library created, frees the
 * host-side context.  The workspace returns to the caller. */
fdg_status fdg_destroy(fdg_ctx* ctx);

/* Number of fp32 parameters of module `module` (1..K). */
fdg_status fdg_param_count(const fdg_ctx* ctx, int module, size_t* out_n);

/* Table of the module's parameter tensors in flat order.  Writes at most `cap` entries
 * to `dst` (may be NULL with cap = 0) and the total number to *out_n. */
fdg_status fdg_param_layout(const fdg_ctx* ctx, int module, fdg_param_entry* dst, size_t cap, size_t* out_n);

/* Copies n = fdg_param_count floats from `src` (host or device) into the module's
 * master weights and refreshes the copies the kernels compute with; momentum is left
 * as it is.  Blocks the host.  Meant for initialisation or a cold restart: batches
 * in flight keep their saved activations but lose their stashed weight versions. */
fdg_status fdg_set_params(fdg_ctx* ctx, int module, const float* src, size_t n);
/* Same for the momentum buffer (checkpoint restore). */
fdg_status fdg_set_momentum(fdg_ctx* ctx, int module, const float* src, size_t n);

/* Copy out (to host or device memory; blocks the host until the module's stream has
 * drained): fp32 master weights; the last shrunk delayed gradient ghat_theta of Eq. 15
 * before weight decay is added (zeros before the module's first backward); momentum. */
fdg_status fdg_get_params(fdg_ctx* ctx, int module, float* dst, size_t n);
fdg_status fdg_get_grads(fdg_ctx* ctx, int module, float* dst, size_t n);
fdg_status fdg_get_momentum(fdg_ctx* ctx, int module, float* dst, size_t n);

/* Learning rate gamma_t used by every update enqueued from the next fdg_step on
 * (Algorithm I takes gamma_t per iteration). */
fdg_status fdg_set_lr(fdg_ctx* ctx, float lr);

/* The learning-rate schedule of the experiments section: start at base_lr, multiply by `gamma` at each
 * milestone epoch (150, 225, 275 with gamma 0.1 in the paper), and optionally run the first `warmup_epochs`
 * epochs at `warmup_lr` (3 epochs at 0.01 for the deep networks and K = 3, 4).  Epoch e (from 0) holds
 * iterations e*iters_per_epoch + 1 .. (e+1)*iters_per_epoch.  fdg_lr_at is the pure function;
 * fdg_set_lr_schedule (NULL: off) makes every following fdg_step set gamma_t = fdg_lr_at(schedule, t) itself. */
typedef struct {
  int64_t iters_per_epoch;
  float base_lr;
  int n_milestones;            /* at most 8 */
  int milestones[8];           /* ascending epochs */
  float gamma;
  int warmup_epochs;
  float warmup_lr;
} fdg_lr_schedule;
fdg_status fdg_lr_at(const fdg_lr_schedule* schedule, int64_t iteration, float* out_lr);
fdg_status fdg_set_lr_schedule(fdg_ctx* ctx, const fdg_lr_schedule* schedule);

/* Running batch-norm statistics, kept for inference (the paper reports test errors, Tables 3-6, without saying
 * how test batches are normalised; reading taken: exponential running average with momentum 0.1 of the batch
 * mean and the unbiased batch variance, started at mean 0 / variance 1, updated by every training forward).
 * Flat vector of a module: for each batch norm in network order (block: BN1, BN2, shortcut BN), its running
 * mean [C] then its running variance [C].  Host or device memory; both calls block the host. */
fdg_status fdg_bn_running_count(const fdg_ctx* ctx, int module, size_t* out_n);
fdg_status fdg_get_bn_running(fdg_ctx* ctx, int module, float* dst, size_t n);
fdg_status fdg_set_bn_running(fdg_ctx* ctx, int module, const float* src, size_t n);

/* Inference: forwards one batch (fp32 [batch][in_h][in_w][in_c], device) through all K modules with their
 * current weights and the running statistics, outside the training pipeline (nothing in flight is touched).
 * `logits_dev` (nullable) receives fp32 [batch][num_classes]; `correct_dev` (nullable, needs `labels_dev`) is
 * INCREMENTED by the number of samples whose largest logit is at their label (top-1; ties go to the lowest
 * class), so a test set can be summed over batches.  Waits for the training work in flight first (blocks the
 * host), then enqueues on `stream`. */
fdg_status fdg_eval(fdg_ctx* ctx, fdg_stream stream, const float* images_dev, const int32_t* labels_dev,
                    float* logits_dev, int* correct_dev);

/* End of training.  After T iterations module k still holds 2(K-k) batches whose gradient has not arrived
 * (Section 3.1: the backward of batch b reaches module k at iteration b + 2K - k - 1); the paper does not say
 * what becomes of them.  fdg_drain runs the 2K - 2 further iterations of Algorithm I in which no new batch
 * enters, so that every batch is back-propagated and applied by every module; `losses_dev` (nullable, device,
 * 2K - 2 floats) receives the loss of the batch the top module handles in each of them (entries of
 * iterations where it has none are left untouched).  Afterwards nothing is in flight and the iteration
 * counter restarts at 0 with the trained weights, momentum and running statistics.  Blocks the host. */
fdg_status fdg_drain(fdg_ctx* ctx, fdg_stream stream, float* losses_dev);

/* Checkpoint of a run in flight: everything a continued run depends on (weights and their versions, momentum,
 * activation FIFOs, mailboxes, label ring, running statistics, counters), so that fdg_load_state followed by
 * the same inputs continues bit for bit.  `dst` / `src`: fdg_state_bytes bytes of host or device memory.
 * A state can be loaded only into a context created with the same architecture and configuration
 * (FDG_ERR_INVALID_ARG otherwise).  The learning rate is part of the state; a schedule is not (set it again).
 * Both block the host. */
fdg_status fdg_state_bytes(const fdg_ctx* ctx, size_t* out_bytes);
fdg_status fdg_save_state(fdg_ctx* ctx, void* dst, size_t bytes);
fdg_status fdg_load_state(fdg_ctx* ctx, const void* src, size_t bytes);

/* One iteration of Algorithm I.  `images_dev` is batch t, fp32 [batch][in_h][in_w][in_c];
 * `labels_dev` int32 [batch] in [0, num_classes).  Both are read only by work enqueued
 * behind `stream` inside this call, so the caller may overwrite them as soon as `stream`
 * has passed the step.  `loss_dev` (nullable, device) receives the mean cross-entropy of
 * batch t-K+1 computed in this iteration; it is written on a module stream, so read it
 * after fdg_sync; it is left untouched while t < K.  Does not block the host.
 * Errors: FDG_ERR_INVALID_ARG (null ctx/images/labels), FDG_ERR_CUDA (a launch failed;
 * the context is then unusable), a latched asynchronous error. */
fdg_status fdg_step(fdg_ctx* ctx, fdg_stream stream, const float* images_dev, const int32_t* labels_dev,
                    float* loss_dev);

/* The same iteration fed from host memory: copies `images_host` (fp32, same layout) and
 * `labels_host` to a staging area of the workspace with cudaMemcpyAsync, runs fdg_step on
 * them, and enqueues a device-to-host copy of the loss of batch t-K+1 into `loss_host`
 * (nullable; untouched while t < K).  The two copies go on a stream of the context, ordered
 * only behind the previous call's read of the staging area, so that from pinned memory they
 * run beside the previous iteration's module-steps; `stream` waits for them before the step.
 * They are NOT ordered behind earlier work on `stream`: the host buffers must hold the batch
 * when the call is made.  Pinned host buffers keep the call asynchronous; pageable ones make
 * the copies block.  The host buffers may be reused once `stream` has passed the step; read
 * *loss_host after fdg_sync.  Errors as fdg_step. */
fdg_status fdg_step_host(fdg_ctx* ctx, fdg_stream stream, const float* images_host, const int32_t* labels_host,
                         float* loss_host);

/* Makes `stream` wait for every module stream, then blocks the host until `stream` is idle.
 * Returns FDG_ERR_NONFINITE if any loss computed since the last call was NaN/Inf, FDG_ERR_INVALID_ARG if a
 * label was outside [0, num_classes) (it was treated as class 0), FDG_ERR_TIMEOUT (latched) if a bounded wait
 * inside a tensor-core kernel ran out, FDG_ERR_CUDA on an asynchronous CUDA error.  The first two are
 * reported once and cleared. */
fdg_status fdg_sync(fdg_ctx* ctx, fdg_stream stream);

/* Fault injection from the host, for testing the error paths without making a kernel misbehave: sets one of
 * the device status words exactly as a kernel would (0: a non-finite loss, 1: a label out of range, 2: a
 * bounded wait of a tensor-core kernel ran out).  The next fdg_sync reports it: FDG_ERR_NONFINITE,
 * FDG_ERR_INVALID_ARG, or FDG_ERR_TIMEOUT; the first two clear with that report and the context carries on,
 * the time-out is latched (a kernel left early, the in-flight state is undefined) and every later fdg_step /
 * fdg_sync returns it.  Blocks the host. */
fdg_status fdg_debug_raise_flag(fdg_ctx* ctx, int which);

/* Guard regions.  Every buffer the library carves out of the workspace is followed by 256 bytes that no kernel
 * may write; fdg_create fills them with a pattern.  fdg_debug_check_guards waits for the context's work, compares
 * every region and returns in *first_bad the index of the first region (in workspace order) that changed, or -1:
 * a kernel that ran past the end of its buffer is then named by the buffer it overran.  fdg_debug_guard_count and
 * fdg_debug_guard_offset give the number of regions and the byte offset of region `index` from the workspace
 * base the caller passed to fdg_create (for a report, or for a test that damages one on purpose from the host).
 * The regions are part of fdg_workspace_bytes and of a saved state.  No counterpart in the paper: a debugging aid. */
fdg_status fdg_debug_guard_count(const fdg_ctx* ctx, size_t* out_count);
fdg_status fdg_debug_guard_offset(const fdg_ctx* ctx, size_t index, size_t* out_byte_offset);
fdg_status fdg_debug_check_guards(fdg_ctx* ctx, long long* first_bad);

/* A wait that really runs out, without a kernel that misbehaves: enqueues on `stream` a one-warp kernel that
 * waits, with the bounded wait of the tensor-core kernels, on a barrier nothing ever arrives at.  After
 * `poll_limit` polls (1..2^20; a poll is well under a microsecond) the wait gives up, the kernel raises the
 * time-out status word as a convolution kernel would, and returns: no copy is in flight and no tensor memory
 * is held.  The next fdg_sync returns FDG_ERR_TIMEOUT (latched); the CUDA context stays usable.  Does not block. */
fdg_status fdg_debug_wait_probe(fdg_ctx* ctx, fdg_stream stream, unsigned poll_limit);

/* The most recent output activation of module k (1..K-1), and the most recent gradient
 * with respect to the input of module k (2..K; the gradient with respect to the images
 * is never formed, so k = 1 is FDG_ERR_INVALID_ARG), as fp32 NHWC to host or device memory.  `n` must equal the tensor's element
 * count, which fdg_boundary_elems reports.  *batch_index receives the batch the tensor
 * belongs to, or -1 (and nothing is copied) while the pipeline has not produced one.
 * The input gradient is returned as produced, i.e. before the receiver applies beta.
 * Both block the host. */
fdg_status fdg_get_module_output(fdg_ctx* ctx, int module, float* dst, size_t n, int64_t* batch_index);
fdg_status fdg_get_input_grad(fdg_ctx* ctx, int module, float* dst, size_t n, int64_t* batch_index);
/* Element counts of those two tensors: the output of module k (0 for k = K) and its input. */
fdg_status fdg_boundary_elems(const fdg_ctx* ctx, int module, size_t* out_elems, size_t* in_elems);

/* Inspection of the activation FIFO: copies one tensor the forward of module `module`
 * saved for its most recent batch, as fp32 NHWC, to host or device memory.  `unit` is the
 * position of the stem/block inside the module (0-based); `which` selects the tensor:
 *   FDG_RESNET_6N2 block: 0 = conv1 output, 1 = ReLU(BN1(.)), 2 = conv2 output, 3 = block output,
 *                         4 = projection-shortcut convolution output (projection blocks only);
 *   FDG_RESNET_6N2 stem:  0 = convolution output, 3 = stem output;
 *   FDG_WRN block:        0 = ReLU(BN1(input)), 1 = conv1 output, 2 = ReLU(BN2(.)), 3 = block output;
 *   FDG_WRN stem:         3 = stem output.
 * `n` must equal the tensor's element count, which is written to *out_elems when `dst` is NULL.
 * *batch_index receives the batch the slot holds, or -1 (nothing copied) before the first
 * forward.  Blocks the host.  Errors: FDG_ERR_INVALID_ARG (bad module/unit/which/n). */
fdg_status fdg_get_saved_tensor(fdg_ctx* ctx, int module, int unit, int which, float* dst, size_t n,
                                size_t* out_elems, int64_t* batch_index);

/* The same for the slot that holds batch `batch` (a batch still in flight in this module, e.g. the one the
 * next backward will read); `batch` < 0 selects the most recent forward.  *batch_index = -1 and nothing is
 * copied when no slot holds that batch. */
fdg_status fdg_get_saved_tensor_of(fdg_ctx* ctx, int module, int unit, int which, int64_t batch, float* dst, size_t n,
                                   size_t* out_elems, int64_t* batch_index);

/* Inspection of the delayed backward (Eq. 10 with the shrunk gradient of Eq. 15): while a capture is on for a
 * module, every backward pass of that module copies each gradient tensor it forms, in stream order, into
 * `dev_buffer` (device memory owned by the caller, 16-byte aligned, at least fdg_capture_bytes; it must stay
 * valid until fdg_capture_end).  The kernels and their launch shapes are unchanged; only device-to-device
 * copies are added.  Refused with FDG_ERR_STATE on a context created with graphs = 1.  Both calls block the host.
 * fdg_get_captured returns one tensor of the most recent captured pass as fp32 NHWC (host or device memory);
 * `unit` as in fdg_get_saved_tensor, `which`:
 *   FDG_RESNET_6N2 block: 0 = gradient of the block output (already shrunk for the module's last block),
 *                         1 = gradient of conv2's output (after the backward of ReLU and BN2),
 *                         2 = gradient of ReLU(BN1(.)) (conv2's data gradient), 3 = gradient of conv1's output,
 *                         4 = gradient of the block input, 5 = gradient of the projection convolution's output;
 *   FDG_RESNET_6N2 stem:  0 = gradient of the stem output, 3 = gradient of the convolution output;
 *   FDG_WRN block:        0 = gradient of the block output, 1 = gradient of ReLU(BN2(.)), 2 = gradient of conv1's
 *                         output, 3 = gradient of ReLU(BN1(input)), 4 = gradient of the block input,
 *                         5 = the projection's share of 3;
 *   FDG_WRN stem:         0 = gradient of the stem output.
 * *batch_index receives the batch of that pass, or -1 (nothing copied) before the first captured pass. */
fdg_status fdg_capture_bytes(const fdg_ctx* ctx, int module, size_t* out_bytes);
fdg_status fdg_capture_begin(fdg_ctx* ctx, int module, void* dev_buffer, size_t bytes);
fdg_status fdg_capture_end(fdg_ctx* ctx, int module);
fdg_status fdg_get_captured(fdg_ctx* ctx, int module, int unit, int which, float* dst, size_t n, size_t* out_elems,
                            int64_t* batch_index);

/* Copies at most `cap` rows of the schedule log (oldest first) and writes the number
 * of rows recorded so far to *out_n.  The log keeps every row of the last 4096 iterations. */
fdg_status fdg_get_schedule_log(const fdg_ctx* ctx, fdg_sched_entry* dst, size_t cap, size_t* out_n);

/* Optional per-launch profiler.  While enabled, every kernel launch is bracketed by two
 * CUDA events on its own stream (up to 65536 launches between reads; later ones are not
 * timed).  fdg_profile_read blocks until the device is idle, writes one row per kernel class
 * (at most `cap`; the number of classes goes to *out_n) and clears the record.  `bytes` and
 * `flops` are algorithmic: each operand tensor counted once per launch, 2 flops per
 * multiply-add.  With one stream per module the kernels of different modules overlap, so a
 * launch's duration includes time shared with others; enable on a serial context to time
 * kernels alone.  Both calls block the host. */
typedef struct {
  char name[32];
  uint64_t launches;
  double total_ms;
  double bytes;
  double flops;
} fdg_kernel_stat;
fdg_status fdg_profile_enable(fdg_ctx* ctx, int on);
/* Per-module busy time while the profiler was on: busy_ms[k-1] = device time between the start and the end
 * of module k's passes (forward; backward + update), summed over the iterations since the last read, the
 * waits for its neighbours excluded.  With one stream per module the passes of different modules share
 * the GPU, so this is the analogue of the per-GPU utilisation column of the paper's speed table; on a
 * serial context it is each module's share of the iteration.  Writes min(cap, K) values, K to *out_n.
 * Blocks the host. */
fdg_status fdg_profile_read_modules(fdg_ctx* ctx, double* busy_ms, size_t cap, size_t* out_n);
fdg_status fdg_profile_read(fdg_ctx* ctx, fdg_kernel_stat* dst, size_t cap, size_t* out_n);

/* Number of kernel launches the library has enqueued since fdg_create. */
fdg_status fdg_launch_count(const fdg_ctx* ctx, uint64_t* out_n);

const char* fdg_status_string(fdg_status s);
/* Human-readable description of the last error on this context ("" if none).  The
 * pointer stays valid until the next call on the context. */
const char* fdg_last_error(const fdg_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* FDG_H_ */
