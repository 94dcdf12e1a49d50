"""fdg_conv_wgrad_static: the weight gradient for callers that cannot allocate scratch memory
(its partial sums go to a buffer built into the library).  Checked through the C ABI against
fdg_conv_wgrad, which takes caller-provided scratch, on two calls in a row with different
inputs, so that anything the first call left in the shared buffer would show in the second.
fdg_conv_wgrad is itself held to the oracle on shapes of this kind (tests/test_gpu_conv_ops.py);
the second call here is compared with the oracle's convolution backward directly as well.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

# (N, H, W, Ci, Co, R, stride, pad): shapes whose pixel sum is split into many slices
SHAPES = [(16, 32, 32, 16, 16, 3, 1, 1), (8, 16, 16, 16, 32, 3, 2, 1), (6, 12, 20, 5, 7, 3, 1, 1)]


@pytest.mark.parametrize("prec_name", ["fp32", "bf16"])
def test_static_scratch_matches_caller_scratch_twice(prec_name):
    from paper_1906_09108_b200 import binding as B
    prec = B.FDG_BF16_TC if prec_name == "bf16" else B.FDG_FP32_CUDACORE
    ops = B.ConvOps(prec)
    tol = 1e-3 if prec_name == "bf16" else 2e-5          # the tolerances of tests/test_gpu_conv_ops.py
    g = torch.Generator(device="cuda").manual_seed(11)
    for shape in SHAPES:
        n, h, w, ci, co, r, st, pad = shape
        s = B.fdg_conv_shape(n, h, w, ci, co, r, st, pad)
        need = C.c_size_t()
        assert ops.lib.fdg_conv_wgrad_scratch_bytes(prec, C.byref(s), C.byref(need)) == B.FDG_OK
        assert need.value > 4 * co * r * r * ci            # more than one slice: the scratch is really used
        p, q = ops.out_hw(s)
        for call in range(2):
            x = torch.randn((n, h, w, ci), generator=g, device="cuda").to(ops.dtype)
            dy = torch.randn((n, p, q, co), generator=g, device="cuda").to(ops.dtype) * (call + 1)
            want = ops.wgrad(s, x, dy).cpu().numpy()
            got = ops.wgrad_static(s, x, dy).cpu().numpy()
            err = np.abs(got - want).max() / max(np.abs(want).max(), 1e-30)
            assert err <= tol, (shape, call, err)
        from oracle import layers as L
        dwo = L.conv2d_backward(dy.float().cpu().numpy().astype(np.float64), x.float().cpu().numpy().astype(np.float64),
                                np.zeros((co, r, r, ci)), st, pad)[1]
        assert np.abs(got - dwo).max() / np.abs(dwo).max() <= tol, shape


def test_static_scratch_rejects_oversized_shapes():
    from paper_1906_09108_b200 import binding as B
    ops = B.ConvOps(B.FDG_FP32_CUDACORE)
    s = B.fdg_conv_shape(2, 8, 8, 512, 512, 3, 1, 1)      # 9*512*512 floats per slice, several slices
    need = C.c_size_t()
    assert ops.lib.fdg_conv_wgrad_scratch_bytes(B.FDG_FP32_CUDACORE, C.byref(s), C.byref(need)) == B.FDG_OK
    assert need.value > (8 << 20)
    x = torch.zeros((2, 8, 8, 512), device="cuda")
    dy = torch.zeros((2, 8, 8, 512), device="cuda")
    dw = torch.zeros((512, 3, 3, 512), device="cuda")
    rc = ops.lib.fdg_conv_wgrad_static(B.FDG_FP32_CUDACORE, C.byref(s), x.data_ptr(), dy.data_ptr(), dw.data_ptr(),
                                       torch.cuda.current_stream().cuda_stream)
    assert rc == 2                                         # FDG_ERR_WORKSPACE_TOO_SMALL
