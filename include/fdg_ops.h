/*
 * libfdg, operator level: the convolution kernels of the FDG module-step as stand-alone
 * calls.  The paper's module forward and backward (Section 3.1; Eq. 8 / Eq. 9 for the chain
 * rule) consist of these contractions; they are exposed so that each kernel can be checked
 * against the CPU oracle and profiled on its own.
 *
 * All pointers are DEVICE pointers.  Storage type follows `precision`: FDG_FP32_CUDACORE =
 * float, FDG_BF16_TC = bf16 (weight gradients are always fp32).  Activations are NHWC,
 * weights [Co][R][S][Ci], square filters R x R.  Calls are asynchronous on `stream`; no
 * call allocates memory.  Return: FDG_OK, FDG_ERR_INVALID_ARG (null pointer, bad shape or
 * precision), FDG_ERR_WORKSPACE_TOO_SMALL, FDG_ERR_CUDA (launch failure).
 *
 * `status_dev` (nullable) is a device int the tensor-core kernels set to 1 if one of their
 * bounded waits ran out (the kernel then leaves early and its output is undefined).
 */
#ifndef FDG_OPS_H_
#define FDG_OPS_H_

#include "fdg.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int N, H, W, Ci;    /* input tensor [N][H][W][Ci] */
  int Co;             /* output channels */
  int R;              /* filter size (R x R) */
  int stride, pad;
} fdg_conv_shape;

/* Optional extras of a convolution call (pass NULL for none; zero-initialise before setting fields).
 * They expose what the module-step does around its convolutions, so that each variant can be checked
 * on its own:
 *   share          launch shape: the tensor-core kernel takes about (SM count / share) CTAs and walks
 *                  several image tiles per CTA, as it does when `share` modules run side by side
 *                  (0 or 1: one launch may take every SM).
 *   wgrad_cta_cap  fdg_conv_wgrad: upper bound of the pixel split (0 = none); the module-step issues its
 *                  weight gradients with 16 on a side stream.
 *   dy_spread      stride-2 gradients (bf16): scratch of N*H*W*Co bf16 elements.  With it the data and
 *                  weight gradients of a 3x3 stride-2 layer run as the stride-1 tensor-core kernels on dy
 *                  spread onto the even pixels of the input grid (the call fills it); without it they
 *                  run on the CUDA cores.
 *   reduce         a per-channel reduction formed in the epilogue of the bf16 tensor-core kernels, one row of
 *                  2*C floats per CTA in `partial` (capacity `partial_floats` >= FDG_CONV_PARTIAL_ROWS*2*C);
 *                  `nparts` receives the number of rows, 0 if the shape took a kernel that forms none.  The
 *                  consumer adds the rows in row order: fdg_bn_apply / fdg_bn_backward with `partial` (up to
 *                  128 channels), or fdg_bn_stats_from_partials (any width).
 *                    1 (fdg_conv_forward): sum y, sum y^2 over the stored y: the batch-norm statistics; the
 *                      halo-tile kernel (3x3, stored tensor of 16, 32 or 64 channels) and the per-tap and
 *                      patch-tile kernels of wider layers and of 1x1 shortcuts (up to 640 output channels);
 *                    2 (fdg_conv_dgrad):   sum dz, sum dz*xhat with dz = dx*[next_mask > 0] and
 *                      xhat = (next_x - mean)*invstd from next_stats[2*C]: the two sums of the batch-norm
 *                      backward that dx feeds (Eq. 9 applied to a normalisation layer). */
#define FDG_CONV_PARTIAL_ROWS 256
typedef struct {
  int share;
  int wgrad_cta_cap;
  void* dy_spread;
  int reduce;
  const void* next_mask;
  const void* next_x;
  const float* next_stats;
  float* partial;
  size_t partial_floats;
  int nparts;               /* out */
} fdg_conv_extra;

/* y = conv(x, w) [+ res], y and res [N][P][Q][Co] with P = (H + 2*pad - R)/stride + 1. */
fdg_status fdg_conv_forward(int precision, const fdg_conv_shape* shape, const void* x, const void* w, void* y,
                            const void* res, fdg_conv_extra* extra, int* status_dev, fdg_stream stream);

/* dx = conv^T(dy, w) [+ res * [res_mask > 0]], dx/res/res_mask [N][H][W][Ci], dy [N][P][Q][Co].
 * `w_flipped` (nullable) is the copy made by fdg_conv_flip_weights; with it, bf16 3x3 shapes run on the
 * tensor cores (stride 2: also needs extra->dy_spread) and so do 1x1 shapes without padding (stride 2 without
 * res: dx is cleared, then written at its even pixels); without it every shape runs on the CUDA cores. */
fdg_status fdg_conv_dgrad(int precision, const fdg_conv_shape* shape, const void* dy, const void* w,
                          const void* w_flipped, void* dx, const void* res, const void* res_mask,
                          fdg_conv_extra* extra, int* status_dev, fdg_stream stream);

/* stats[0..C) = mean, stats[C..2C) = 1/sqrt(var + eps) from `nparts` rows of (sum, sum of squares) partial sums,
 * partial[nparts][2*C], that a convolution with reduce = 1 left; `rows` = values per channel behind the sums.
 * The rows are added in a fixed order (fp64).  Asynchronous on `stream`. */
fdg_status fdg_bn_stats_from_partials(const float* partial, int nparts, size_t rows, int C, float eps, float* stats,
                                      fdg_stream stream);

/* Probe of the tensor pipe, for roofline arguments (no counterpart in the paper): on every SM one thread issues
 * reps * 4 * accumulators tcgen05.mma instructions (M = 128, N = n, K = 16, bf16, operands in shared memory) back to
 * back, rotating over `accumulators` (1..3, n * accumulators <= 512) accumulators in tensor memory; `unrolled` = 1
 * issues them as straight-line code, 0 keeps the rotation as a run-time loop (a counter and a branch between two
 * instructions: what a kernel's issuing loop costs when it is not unrolled).
 * cycles_dev[0] = SM cycles until the last one was issued, cycles_dev[1] = until it completed (device pointer to two
 * 64-bit integers, written by the first CTA).  n: multiple of 16 in 16..256.  Its wait is bounded like every other;
 * status_dev as above.  Asynchronous on `stream`. */
fdg_status fdg_probe_mma_rate(int n, int accumulators, int reps, int unrolled, long long* cycles_dev, int* status_dev,
                              fdg_stream stream);

/* w_flipped[ci][R-1-r][R-1-s][co] = w[co][r][s][ci] (bf16, R = 3 or 1): the operand layout of the
 * tensor-core data-gradient kernel. */
fdg_status fdg_conv_flip_weights(const fdg_conv_shape* shape, const void* w_bf16, void* w_flipped_bf16,
                                 fdg_stream stream);

/* dw[co][r][s][ci] (fp32) = sum over pixels of dy * shifted x.  The sum over pixels is split
 * into slices whose partial results go to `scratch` (fdg_conv_wgrad_scratch_bytes) and are
 * added in a fixed order, so the result does not depend on scheduling. */
fdg_status fdg_conv_wgrad_scratch_bytes(int precision, const fdg_conv_shape* shape, size_t* bytes);
fdg_status fdg_conv_wgrad(int precision, const fdg_conv_shape* shape, const void* x, const void* dy, float* dw,
                          void* scratch, size_t scratch_bytes, fdg_conv_extra* extra, int* status_dev,
                          fdg_stream stream);

/* fdg_conv_wgrad for callers that cannot hand over scratch memory.  The paper has no
 * counterpart to this call; it exists for hosts of the library that are not allowed to
 * allocate device memory at the point where they need a weight gradient: code running under a
 * memory plan that was fixed up front, inside a stream-ordered region where cudaMalloc would
 * synchronise the device, or behind an allocator they do not own.  Same arguments and result as
 * fdg_conv_wgrad on the CUDA-core path, but the partial sums go to a buffer that is part of the
 * library image: FDG_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library,
 * held until the process exits.  The call itself allocates and frees nothing.
 *   - The call always takes the CUDA-core kernel, whose slice buffer is what
 *     fdg_conv_wgrad_scratch_bytes reports for FDG_FP32_CUDACORE (for bf16 shapes that fdg_conv_wgrad
 *     would run on the tensor cores the bf16 figure is larger and does not apply here).  Shapes whose
 *     slice buffer exceeds FDG_STATIC_SCRATCH_BYTES are refused with FDG_ERR_WORKSPACE_TOO_SMALL and
 *     nothing is launched.
 *   - The first call on each device looks up the buffer's device address (a host-side query,
 *     made with that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one buffer, and it keeps what the previous call left.
 *     Every slice of partial sums a launch reads was written by that same launch, so nothing
 *     has to be cleared, but two calls whose kernels may overlap on the GPU (different
 *     streams without an ordering between them) race on it: order them. */
#define FDG_STATIC_SCRATCH_BYTES ((size_t)8 << 20)
fdg_status fdg_conv_wgrad_static(int precision, const fdg_conv_shape* shape, const void* x, const void* dy,
                                 float* dw, fdg_stream stream);

/* Which path a call takes, given every optional operand (w_flipped, dy_spread): op 0 = forward,
 * 1 = dgrad, 2 = wgrad. */
fdg_status fdg_conv_path(int precision, const fdg_conv_shape* shape, int op, int* uses_tensor_cores);

/* ---- the memory-bound steps of the module-step, on tensors seen as [rows = N*H*W][C] ------------
 * Batch normalisation in training mode: per-channel mean and biased variance over the rows of the
 * current batch; stats[0..C) = mean, stats[C..2C) = 1/sqrt(var + eps).  Sums are fp32 per thread and
 * block, fp64 across blocks, in a fixed order.  `scratch`: fdg_bn_scratch_bytes(C) bytes of device memory
 * (any contents).  Threading: the calls of this header may be made from several host threads; calls that
 * share a scratch buffer or an output must be ordered by the caller. */
fdg_status fdg_bn_scratch_bytes(int C, size_t* bytes);
fdg_status fdg_bn_stats(int precision, const void* x, size_t rows, int C, float eps, float* stats, void* scratch,
                        size_t scratch_bytes, fdg_stream stream);
/* y = [relu]( gamma*(x - mean)*invstd + beta + residual ), residual = none (res NULL) | res | the batch norm
 * of res with (res_stats, res_gamma, res_beta).  With `partial` (nparts rows of (sum x, sum x^2) left by
 * fdg_conv_forward with reduce = 1) the statistics are formed from those rows first and written to `stats`;
 * `block_cap` (0 = none) then bounds the grid, since every block repeats that addition (the module-step
 * uses 4 * 148 / K). */
fdg_status fdg_bn_apply(int precision, const void* x, float* stats, const float* gamma, const float* beta,
                        const void* res, const float* res_stats, const float* res_gamma, const float* res_beta, int relu,
                        void* y, size_t rows, int C, float eps, const float* partial, int nparts, int block_cap,
                        fdg_stream stream);
/* Backward of y = BN(x) under a ReLU gate: dz = dy * [mask > 0] (mask NULL: dz = dy);
 *   dbeta = sum dz, dgamma = sum dz*xhat, dx = gamma*invstd*(dz - dbeta/M - xhat*dgamma/M) [+ res].
 * With (x2, stats2, gamma2) the same dz is also taken through a second normalisation (the projection
 * shortcut of a block): dx2, dgamma2, dbeta2.  With `partial` (rows left by fdg_conv_dgrad with reduce = 2)
 * the sums are read from those rows instead of being formed here (single normalisation only).  With dx NULL
 * only the sums, i.e. the parameter gradients, are formed. */
fdg_status fdg_bn_backward(int precision, const void* dy, const void* mask, const void* x, const float* stats,
                           const float* gamma, const void* x2, const float* stats2, const float* gamma2, const void* res,
                           void* dx, void* dx2, float* dgamma, float* dbeta, float* dgamma2, float* dbeta2, size_t rows,
                           int C, const float* partial, int nparts, int block_cap, void* scratch, size_t scratch_bytes,
                           fdg_stream stream);
/* out = beta * in: the shrinking of the received delayed gradient (Eq. 15). */
fdg_status fdg_shrink(int precision, const void* in, void* out, float beta, size_t n, fdg_stream stream);
/* The update of Eq. 11 with the optimiser of the experiments section: g' = grad + wd*theta;
 * v = momentum*v + g'; theta -= lr*v; the new theta is also written to next_fp32 and (nullable) next_bf16,
 * the weight version the following forward reads.  fp32 pointers 16-byte aligned. */
fdg_status fdg_sgd_update(float* theta, float* momentum_buf, const float* grad, float* next_fp32, void* next_bf16,
                          size_t n, float lr, float momentum, float weight_decay, fdg_stream stream);
/* Image ingest: fp32 [rows][c_in] -> storage type [rows][c_out] with channels c_in.. zero; labels copied. */
fdg_status fdg_ingest(int precision, const float* images, void* out, size_t rows, int c_in, int c_out,
                      const int32_t* labels_in, int32_t* labels_out, int batch, fdg_stream stream);
/* The classifier of the top module and its backward: global average pool over `hw` pixels, fully connected
 * layer (w [classes][features], b), mean softmax cross-entropy against `labels` (the paper's f, Eq. 1), then
 * dlogits, dw, db and dx [batch][hw][features] (the gradient handed to the last block; never shrunk).
 * pooled [batch][features], dlogits [batch][classes], loss_n [batch] are fp32 outputs; *loss the mean.
 * flags[0] is raised on a non-finite loss, flags[1] on a label outside [0, classes) (treated as class 0). */
fdg_status fdg_head(int precision, const void* x, const float* w, const float* b, const int32_t* labels, int batch,
                    int hw, int features, int classes, float* pooled, float* dlogits, float* loss_n, void* dx,
                    float* dw, float* db, float* loss, int* flags, fdg_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* FDG_OPS_H_ */
