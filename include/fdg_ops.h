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

/* Which path a call takes: op 0 = forward, 1 = dgrad (with w_flipped), 2 = wgrad. */
fdg_status fdg_conv_path(int precision, const fdg_conv_shape* shape, int op, int* uses_tensor_cores);

#ifdef __cplusplus
}
#endif
#endif /* FDG_OPS_H_ */
