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

/* y = conv(x, w) [+ res], y and res [N][P][Q][Co] with P = (H + 2*pad - R)/stride + 1. */
fdg_status fdg_conv_forward(int precision, const fdg_conv_shape* shape, const void* x, const void* w, void* y,
                            const void* res, int* status_dev, fdg_stream stream);

/* dx = conv^T(dy, w) [+ res * [res_mask > 0]], dx/res/res_mask [N][H][W][Ci], dy [N][P][Q][Co].
 * `w_flipped` (nullable) is the copy made by fdg_conv_flip_weights; with it, bf16 3x3 stride-1
 * shapes run on the tensor cores, without it every shape runs on the CUDA cores. */
fdg_status fdg_conv_dgrad(int precision, const fdg_conv_shape* shape, const void* dy, const void* w,
                          const void* w_flipped, void* dx, const void* res, const void* res_mask, int* status_dev,
                          fdg_stream stream);

/* w_flipped[ci][2-r][2-s][co] = w[co][r][s][ci] (bf16, R = 3): the operand layout of the
 * tensor-core data-gradient kernel. */
fdg_status fdg_conv_flip_weights(const fdg_conv_shape* shape, const void* w_bf16, void* w_flipped_bf16,
                                 fdg_stream stream);

/* dw[co][r][s][ci] (fp32) = sum over pixels of dy * shifted x.  The sum over pixels is split
 * into slices whose partial results go to `scratch` (fdg_conv_wgrad_scratch_bytes) and are
 * added in a fixed order, so the result does not depend on scheduling. */
fdg_status fdg_conv_wgrad_scratch_bytes(int precision, const fdg_conv_shape* shape, size_t* bytes);
fdg_status fdg_conv_wgrad(int precision, const fdg_conv_shape* shape, const void* x, const void* dy, float* dw,
                          void* scratch, size_t scratch_bytes, int* status_dev, fdg_stream stream);

/* fdg_conv_wgrad for callers that cannot hand over scratch memory.  The paper has no
 * counterpart to this call; it exists for hosts of the library that are not allowed to
 * allocate device memory at the point where they need a weight gradient: code running under a
 * memory plan that was fixed up front, inside a stream-ordered region where cudaMalloc would
 * synchronise the device, or behind an allocator they do not own.  Same arguments and result as
 * fdg_conv_wgrad on the CUDA-core path, but the partial sums go to a buffer that is part of the
 * library image: FDG_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the library,
 * held until the process exits.  The call itself allocates and frees nothing.
 *   - Shapes whose fdg_conv_wgrad_scratch_bytes exceeds FDG_STATIC_SCRATCH_BYTES are refused
 *     with FDG_ERR_WORKSPACE_TOO_SMALL and nothing is launched.
 *   - The first call on each device looks up the buffer's device address (a host-side query,
 *     made with that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one buffer, and it keeps what the previous call left.
 *     Every slice of partial sums a launch reads was written by that same launch, so nothing
 *     has to be cleared, but two calls whose kernels may overlap on the GPU (different
 *     streams without an ordering between them) race on it: order them. */
#define FDG_STATIC_SCRATCH_BYTES ((size_t)8 << 20)
fdg_status fdg_conv_wgrad_static(int precision, const fdg_conv_shape* shape, const void* x, const void* dy,
                                 float* dw, fdg_stream stream);

/* Which path a call takes: op 0 = forward, 1 = dgrad (with w_flipped), 2 = wgrad. */
fdg_status fdg_conv_path(int precision, const fdg_conv_shape* shape, int op, int* uses_tensor_cores);

#ifdef __cplusplus
}
#endif
#endif /* FDG_OPS_H_ */
