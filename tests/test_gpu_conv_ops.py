"""Operator-level parity: fdg_conv_forward / dgrad / wgrad through the C ABI against the
oracle's convolution (oracle/layers.py), element by element.  bf16 cases feed both sides
the same bf16-rounded inputs; the oracle then works in float64, so the only differences
are fp32 accumulation order and the final rounding of the output to bf16 (2^-9 relative)."""
import numpy as np
import pytest
import torch

from oracle import layers as L

pytestmark = pytest.mark.gpu


def _mk(shape, seed, dtype):
    g = np.random.default_rng(seed)
    a = g.standard_normal(shape).astype(np.float32)
    t = torch.from_numpy(a).cuda().to(dtype)
    return t, t.float().cpu().numpy().astype(np.float64)


def _rel(a, b):
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


# (N, H, W, Ci, Co, R, stride, pad)
SHAPES_ANY = [(3, 12, 20, 5, 7, 3, 1, 1), (2, 16, 16, 8, 16, 3, 2, 1), (2, 16, 16, 16, 24, 1, 2, 0),
              (5, 8, 8, 3, 8, 3, 1, 1), (3, 16, 16, 6, 32, 1, 1, 0), (3, 16, 16, 12, 32, 1, 2, 0)]
SHAPES_TC = [(4, 32, 32, 16, 16, 3, 1, 1),      # 32 tiles of 4 image rows, 32-byte swizzle
             (6, 16, 16, 32, 32, 3, 1, 1),      # 8 rows per tile, 64-byte swizzle
             (10, 8, 8, 64, 64, 3, 1, 1),       # two images per tile, 128-byte swizzle
             (2, 32, 32, 16, 48, 3, 1, 1),      # c_in != c_out
             (2, 16, 16, 128, 160, 3, 1, 1),    # two channel chunks, wide N
             (300, 8, 8, 64, 64, 3, 1, 1),      # more tiles than SMs: several tiles per CTA
             (5, 12, 20, 16, 32, 3, 1, 1),      # non-square image, c_in != c_out, odd batch
             (3, 6, 10, 64, 16, 3, 1, 1),
             (37, 16, 16, 32, 64, 3, 1, 1),     # ragged last tile in the weight gradient's pixel split
             (301, 8, 8, 64, 64, 3, 1, 1),      # ragged last tile with several images per tile
             (130, 32, 32, 16, 16, 3, 1, 1),    # stage-1 shape of the 6n+2 networks, more images than weight-gradient CTAs
             (6, 32, 32, 16, 32, 3, 2, 1),      # stride 2: forward = the stride-1 kernel stored at the even pixels
             (9, 16, 16, 32, 64, 3, 2, 1),
             (2, 16, 16, 320, 320, 3, 1, 1),    # WRN stage 2: five 64-channel chunks, two 160-column N tiles
             (4, 8, 8, 640, 640, 3, 1, 1),      # WRN stage 3: four N tiles, the weight gradient in 10 x 10 channel chunks
             (2, 32, 32, 160, 320, 3, 2, 1),    # the stride-2 layers of WRN-28-10 (per-tap kernel at full resolution)
             (2, 16, 16, 320, 640, 3, 2, 1),
             # the exact-tile weight-gradient kernel of wide layers: several 64-pixel slabs per CTA (the shared-memory
             # ring wraps), a last block of 32 output channels, two rows of 8 pixels per reduction step
             (24, 16, 16, 320, 320, 3, 1, 1),
             (3, 32, 32, 160, 160, 3, 1, 1),
             (16, 8, 8, 640, 640, 3, 1, 1),
             (5, 16, 16, 128, 256, 3, 1, 1),
             # 1x1 projection shortcuts on the per-tap kernel: stride 2 reads the even pixels of x as a strided tensor
             # and writes dx at the even pixels of a cleared tensor; the weight gradient of wide ones on the exact-tile kernel
             (4, 32, 32, 160, 320, 1, 2, 0),
             (8, 16, 16, 320, 640, 1, 2, 0),
             (2, 32, 32, 16, 160, 1, 1, 0),
             (6, 16, 16, 32, 64, 1, 2, 0),
             # CIFAR ResNet-18 shapes: 64 channels on 32x32 images (too large for a halo tile: exact-tile weight gradient
             # with one 64-channel sub-tile), and few-pixel layers whose forward tiles are narrowed to fill the SMs
             (8, 32, 32, 64, 64, 3, 1, 1),
             (8, 32, 32, 64, 128, 3, 2, 1),
             (16, 4, 4, 512, 512, 3, 1, 1),
             (32, 8, 8, 256, 256, 3, 1, 1)]

# shapes whose three operators all take the halo-tile tensor-core kernels
ALL_TC = {(4, 32, 32, 16, 16), (6, 16, 16, 32, 32), (10, 8, 8, 64, 64), (300, 8, 8, 64, 64), (5, 12, 20, 16, 32),
          (3, 6, 10, 64, 16), (37, 16, 16, 32, 64), (301, 8, 8, 64, 64), (130, 32, 32, 16, 16)}


def _run(prec_name, shape, expect_tc):
    from paper_1906_09108_b200 import binding as B
    prec = B.FDG_BF16_TC if prec_name == "bf16" else B.FDG_FP32_CUDACORE
    ops = B.ConvOps(prec)
    n, h, w, ci, co, r, st, pad = shape
    s = B.fdg_conv_shape(n, h, w, ci, co, r, st, pad)
    p, q = ops.out_hw(s)
    x, xo = _mk((n, h, w, ci), 1, ops.dtype)
    wt, wo = _mk((co, r, r, ci), 2, ops.dtype)
    dy, dyo = _mk((n, p, q, co), 3, ops.dtype)
    res, reso = _mk((n, h, w, ci), 4, ops.dtype)
    mask, masko = _mk((n, h, w, ci), 5, ops.dtype)
    resy, resyo = _mk((n, p, q, co), 6, ops.dtype)
    tol = 1e-2 if prec_name == "bf16" else 2e-5
    assert ops.path(s, 0) == expect_tc
    if prec_name == "bf16" and shape[:5] in ALL_TC:
        assert ops.path(s, 1) and ops.path(s, 2)

    y = ops.forward(s, x, wt).float().cpu().numpy()
    assert _rel(y, L.conv2d_forward(xo, wo, st, pad)) < tol
    y = ops.forward(s, x, wt, res=resy).float().cpu().numpy()
    assert _rel(y, L.conv2d_forward(xo, wo, st, pad) + resyo) < tol

    dxo, dwo = L.conv2d_backward(dyo, xo, wo, st, pad)
    wf = ops.flip_weights(s, wt) if (prec_name == "bf16" and r in (1, 3)) else None
    dx = ops.dgrad(s, dy, wt, wf).float().cpu().numpy()
    assert _rel(dx, dxo) < tol
    dx = ops.dgrad(s, dy, wt, wf, res=res, res_mask=mask).float().cpu().numpy()
    assert _rel(dx, dxo + reso * (masko > 0)) < tol
    if wf is not None:          # the CUDA-core path of the same call must agree as well
        dx = ops.dgrad(s, dy, wt, None).float().cpu().numpy()
        assert _rel(dx, dxo) < tol

    dw = ops.wgrad(s, x, dy).cpu().numpy()
    assert _rel(dw, dwo) < (1e-3 if prec_name == "bf16" else 2e-5)
    if expect_tc:
        # the launch shapes of a module-step: a quarter of the SMs per kernel (four modules side by side),
        # the weight gradient's pixel split capped at 16 CTAs (side stream), and, for stride 2, both
        # gradients on the tensor cores through the spread-out dy
        sp = st == 2
        if sp:
            assert ops.path(s, 1)
        y = ops.forward(s, x, wt, res=resy, share=4).float().cpu().numpy()
        assert _rel(y, L.conv2d_forward(xo, wo, st, pad) + resyo) < tol
        dx = ops.dgrad(s, dy, wt, wf, res=res, res_mask=mask, share=4, spread=sp).float().cpu().numpy()
        assert _rel(dx, dxo + reso * (masko > 0)) < tol
        dx = ops.dgrad(s, dy, wt, wf, spread=sp).float().cpu().numpy()
        assert _rel(dx, dxo) < tol
        for cap in (0, 16):
            dw = ops.wgrad(s, x, dy, cta_cap=cap, spread=sp).cpu().numpy()
            assert _rel(dw, dwo) < 1e-3, cap
    assert not ops.timed_out()


@pytest.mark.parametrize("shape", SHAPES_ANY + SHAPES_TC[:3])
def test_conv_ops_fp32(shape):
    _run("fp32", shape, False)


@pytest.mark.parametrize("shape", SHAPES_ANY)
def test_conv_ops_bf16_cuda_core_shapes(shape):
    _run("bf16", shape, False)


@pytest.mark.parametrize("shape", SHAPES_TC)
def test_conv_ops_bf16_tensor_core_shapes(shape):
    _run("bf16", shape, True)


@pytest.mark.parametrize("co,ci,r", [(16, 16, 3), (64, 160, 3), (320, 160, 1), (24, 20, 3), (10, 6, 1), (200, 72, 3),
                                     (640, 640, 3), (65, 64, 3)])
def test_flipped_weight_copy_is_the_index_permutation(co, ci, r):
    """dst[ci][R-1-r][R-1-s][co] = src[co][r][s][ci], bit for bit: channel counts that take the 16-byte vector
    tiles (multiples of 8), ragged last tiles (200, 72), and counts that take the element-wise tiles."""
    from paper_1906_09108_b200 import binding as B
    ops = B.ConvOps(B.FDG_BF16_TC)
    s = B.fdg_conv_shape(1, 8, 8, ci, co, r, 1, r // 2)
    rng = np.random.default_rng(7)
    w = torch.from_numpy(rng.standard_normal((co, r, r, ci)).astype(np.float32)).to(torch.bfloat16).cuda()
    got = ops.flip_weights(s, w).view(ci, r, r, co).float().cpu().numpy()
    want = w.float().cpu().numpy()[:, ::-1, ::-1, :].transpose(3, 1, 2, 0)
    assert np.array_equal(got, want)
