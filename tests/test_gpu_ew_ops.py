"""Operator-level parity of the memory-bound steps and of the reductions fused into the
convolution epilogues, through the C ABI (include/fdg_ops.h) against the oracle's layer
functions (oracle/layers.py) in float64, element by element.

Both sides get the same inputs (bf16 cases: the same bf16-rounded values), so no ReLU gate
can fall differently; what remains is fp32 arithmetic, the order of the sums and, in bf16
mode, the final rounding of a stored tensor (one bf16 ulp = 2^-8 of the element).  Bars:
1e-2 max relative error for bf16 tensors, 1e-5 for fp32 ones and for fp32 reductions."""
import numpy as np
import pytest
import torch

from oracle import layers as L

pytestmark = pytest.mark.gpu
EPS = 1e-5


def _mk(shape, seed, dtype, scale=1.0, shift=0.0):
    g = np.random.default_rng(seed)
    a = (g.standard_normal(shape) * scale + shift).astype(np.float32)
    t = torch.from_numpy(a).cuda().to(dtype)
    return t, t.float().cpu().numpy().astype(np.float64)


def _f32(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).cuda()


def _rel(a, b):
    a = a.float().cpu().numpy().astype(np.float64) if isinstance(a, torch.Tensor) else np.asarray(a, dtype=np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def _ops(prec_name):
    from paper_1906_09108_b200 import binding as B
    prec = B.FDG_BF16_TC if prec_name == "bf16" else B.FDG_FP32_CUDACORE
    return B, B.EwOps(prec), (1e-2 if prec_name == "bf16" else 1e-5)


def _stats_ref(xo):
    mean = xo.mean(axis=(0, 1, 2))
    var = ((xo - mean) ** 2).mean(axis=(0, 1, 2))
    return mean, 1.0 / np.sqrt(var + EPS)


# (N, H, W, C): stage shapes of the 6n+2 networks at small batch, a WRN width, odd sizes
BN_SHAPES = [(8, 32, 32, 16), (6, 16, 16, 32), (10, 8, 8, 64), (3, 16, 16, 160), (5, 12, 20, 24), (2, 6, 10, 5)]


@pytest.mark.parametrize("prec_name", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", BN_SHAPES)
def test_bn_forward(prec_name, shape):
    B, ew, tol = _ops(prec_name)
    c = shape[-1]
    if prec_name == "bf16" and c % 8:
        pytest.skip("bf16 storage needs channel counts that are multiples of 8")
    x, xo = _mk(shape, 1, ew.dtype, scale=1.7, shift=0.3)
    res, reso = _mk(shape, 2, ew.dtype)
    gam, beta = 1.0 + 0.2 * np.random.default_rng(3).standard_normal(c), 0.1 * np.random.default_rng(4).standard_normal(c)
    gam2, beta2 = 1.0 + 0.2 * np.random.default_rng(5).standard_normal(c), 0.1 * np.random.default_rng(6).standard_normal(c)
    stats = ew.bn_stats(x, EPS)
    mean, invstd = _stats_ref(xo)
    assert _rel(stats[:c], mean) <= 1e-5 + 1e-6 / max(np.abs(mean).max(), 1e-6)
    assert _rel(stats[c:], invstd) <= 1e-5
    bn = L.batchnorm_forward(xo, gam, beta, EPS)[0]
    y = ew.bn_apply(x, stats, _f32(gam), _f32(beta), relu=True)
    assert _rel(y, L.relu_forward(bn)) <= tol
    y = ew.bn_apply(x, stats, _f32(gam), _f32(beta), relu=False)
    assert _rel(y, bn) <= tol
    y = ew.bn_apply(x, stats, _f32(gam), _f32(beta), res=res, relu=True)           # identity shortcut
    assert _rel(y, L.relu_forward(bn + reso)) <= tol
    rstats = ew.bn_stats(res, EPS)                                                   # projection shortcut: BN of the residual
    y = ew.bn_apply(x, stats, _f32(gam), _f32(beta), res=res, res_bn=(rstats, _f32(gam2), _f32(beta2)), relu=True)
    assert _rel(y, L.relu_forward(bn + L.batchnorm_forward(reso, gam2, beta2, EPS)[0])) <= tol


@pytest.mark.parametrize("prec_name", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", BN_SHAPES)
def test_bn_backward(prec_name, shape):
    B, ew, tol = _ops(prec_name)
    c = shape[-1]
    if prec_name == "bf16" and c % 8:
        pytest.skip("bf16 storage needs channel counts that are multiples of 8")
    x, xo = _mk(shape, 11, ew.dtype, scale=1.3, shift=-0.2)
    x2, x2o = _mk(shape, 12, ew.dtype, scale=0.7, shift=0.4)
    dy, dyo = _mk(shape, 13, ew.dtype)
    mask, masko = _mk(shape, 14, ew.dtype)
    res, reso = _mk(shape, 15, ew.dtype)
    gam = 1.0 + 0.2 * np.random.default_rng(16).standard_normal(c)
    gam2 = 1.0 + 0.2 * np.random.default_rng(17).standard_normal(c)
    stats, stats2 = ew.bn_stats(x, EPS), ew.bn_stats(x2, EPS)
    sv = L.batchnorm_forward(xo, gam, np.zeros(c), EPS)[1]
    sv2 = L.batchnorm_forward(x2o, gam2, np.zeros(c), EPS)[1]
    # plain, gated, gated with residual
    for m_t, m_o, r_t, r_o in ((None, None, None, None), (mask, masko, None, None), (mask, masko, res, reso)):
        dz = dyo if m_o is None else L.relu_backward(dyo, m_o)
        dxo, dgo, dbo = L.batchnorm_backward(dz, sv, gam)
        if r_o is not None:
            dxo = dxo + r_o
        dx, dg, db = ew.bn_backward(dy, m_t, x, stats, _f32(gam), res=r_t)
        assert _rel(dx, dxo) <= tol
        assert _rel(dg, dgo) <= 1e-4 and _rel(db, dbo) <= 1e-4
    # the projection block: one dz through two normalisations
    dz = L.relu_backward(dyo, masko)
    dxo, dgo, dbo = L.batchnorm_backward(dz, sv, gam)
    dx2o, dg2o, db2o = L.batchnorm_backward(dz, sv2, gam2)
    dx, dg, db, dx2, dg2, db2 = ew.bn_backward(dy, mask, x, stats, _f32(gam), second=(x2, stats2, _f32(gam2)))
    assert _rel(dx, dxo) <= tol and _rel(dx2, dx2o) <= tol
    for got, want in ((dg, dgo), (db, dbo), (dg2, dg2o), (db2, db2o)):
        assert _rel(got, want) <= 1e-4


# (N, H, W, Ci, Co, stride, share): every epilogue variant of the halo-tile kernel (16 output channels keep
# per-thread sums, wider ones go through the shuffle reduction), several image tiles per CTA (share > 1 or
# more images than SMs), a stride-2 layer, ragged last tiles.
FUSED_SHAPES = [(8, 32, 32, 16, 16, 1, 1), (128, 32, 32, 16, 16, 1, 3), (6, 16, 16, 32, 32, 1, 1), (37, 16, 16, 32, 32, 1, 4),
                (10, 8, 8, 64, 64, 1, 1), (301, 8, 8, 64, 64, 1, 2), (6, 32, 32, 16, 32, 2, 1), (20, 16, 16, 32, 64, 2, 3),
                (5, 12, 20, 16, 32, 1, 2)]


@pytest.mark.parametrize("shape", FUSED_SHAPES)
@pytest.mark.parametrize("with_res", [False, True])
def test_conv_forward_with_fused_statistics(shape, with_res):
    """fdg_conv_forward with reduce = 1, then fdg_bn_apply on the partial rows: the convolution output, the
    summed rows, the statistics the apply kernel derives from them and the normalised output."""
    from paper_1906_09108_b200 import binding as B
    n, h, w, ci, co, stride, share = shape
    ops, ew = B.ConvOps(B.FDG_BF16_TC), B.EwOps(B.FDG_BF16_TC)
    s = B.fdg_conv_shape(n, h, w, ci, co, 3, stride, 1)
    p, q = ops.out_hw(s)
    x, xo = _mk((n, h, w, ci), 21, ops.dtype)
    wt, wo = _mk((co, 3, 3, ci), 22, ops.dtype, scale=(2.0 / (9 * ci)) ** 0.5)
    res, reso = _mk((n, p, q, co), 23, ops.dtype)
    gam, beta = 1.0 + 0.2 * np.random.default_rng(24).standard_normal(co), 0.1 * np.random.default_rng(25).standard_normal(co)
    y, part = ops.forward(s, x, wt, res=res if with_res else None, share=share, reduce=True)
    assert part.shape[0] >= 1 and not ops.timed_out()
    yo = L.conv2d_forward(xo, wo, stride, 1) + (reso if with_res else 0.0)
    assert _rel(y, yo) <= 1e-2
    ys = y.float().cpu().numpy().astype(np.float64)                 # the sums are taken over the stored values
    tot = part.double().sum(dim=0).cpu().numpy()
    assert _rel(tot[:co], ys.sum(axis=(0, 1, 2))) <= 1e-5 + 1e-3 / max(np.abs(ys.sum(axis=(0, 1, 2))).max(), 1e-3)
    assert _rel(tot[co:], (ys * ys).sum(axis=(0, 1, 2))) <= 1e-5
    stats = torch.full((2 * co,), float("nan"), dtype=torch.float32, device="cuda")
    a = ew.bn_apply(y, stats, _f32(gam), _f32(beta), relu=True, eps=EPS, partial=part, block_cap=148)
    mean, invstd = _stats_ref(ys)
    assert _rel(stats[:co], mean) <= 1e-4 and _rel(stats[co:], invstd) <= 1e-5
    assert _rel(a, L.relu_forward(L.batchnorm_forward(ys, gam, beta, EPS)[0])) <= 1e-2


# (N, H, W, Ci, Co, R, stride): the wide layers' kernels -- patch tiles (16x16 and 32x32 images), per-tap tiles (8x8, also
# with narrowed column tiles), a strided 3x3 layer computed at full resolution, 1x1 shortcuts of both strides
WIDE_FUSED_SHAPES = [(6, 16, 16, 320, 320, 3, 1), (3, 32, 32, 160, 160, 3, 1), (16, 8, 8, 640, 640, 3, 1),
                     (4, 32, 32, 160, 320, 3, 2), (32, 8, 8, 256, 256, 3, 1), (4, 32, 32, 160, 320, 1, 2),
                     (2, 32, 32, 16, 160, 1, 1)]


@pytest.mark.parametrize("shape", WIDE_FUSED_SHAPES)
@pytest.mark.parametrize("with_res", [False, True])
def test_wide_conv_forward_with_fused_statistics(shape, with_res):
    """fdg_conv_forward with reduce = 1 on the wide layers' kernels, then fdg_bn_stats_from_partials: the
    convolution output, the summed rows against the stored output, and the statistics derived from them."""
    from paper_1906_09108_b200 import binding as B
    n, h, w, ci, co, r, stride = shape
    ops = B.ConvOps(B.FDG_BF16_TC)
    s = B.fdg_conv_shape(n, h, w, ci, co, r, stride, 1 if r == 3 else 0)
    p, q = ops.out_hw(s)
    x, xo = _mk((n, h, w, ci), 41, ops.dtype)
    wt, wo = _mk((co, r, r, ci), 42, ops.dtype, scale=(2.0 / (r * r * ci)) ** 0.5)
    res, reso = _mk((n, p, q, co), 43, ops.dtype)
    y, part = ops.forward(s, x, wt, res=res if with_res else None, reduce=True)
    assert part.shape[0] >= 1 and not ops.timed_out()
    yo = L.conv2d_forward(xo, wo, stride, 1 if r == 3 else 0) + (reso if with_res else 0.0)
    assert _rel(y, yo) <= 1e-2
    ys = y.float().cpu().numpy().astype(np.float64)                 # the sums are taken over the stored values
    tot = part.double().sum(dim=0).cpu().numpy()
    assert np.abs(tot[:co] - ys.sum(axis=(0, 1, 2))).max() <= 1e-4 * np.abs(ys).sum(axis=(0, 1, 2)).max()
    assert _rel(tot[co:], (ys * ys).sum(axis=(0, 1, 2))) <= 1e-5
    stats = torch.full((2 * co,), float("nan"), dtype=torch.float32, device="cuda")
    rc = ops.lib.fdg_bn_stats_from_partials(part.data_ptr(), part.shape[0], n * p * q, co, EPS, stats.data_ptr(),
                                            torch.cuda.current_stream().cuda_stream)
    assert rc == B.FDG_OK
    mean, invstd = _stats_ref(ys)
    assert np.abs(stats[:co].cpu().numpy() - mean).max() <= 1e-5 * max(np.abs(ys).max(), 1.0)
    assert _rel(stats[co:], invstd) <= 1e-5


@pytest.mark.parametrize("shape", FUSED_SHAPES)
@pytest.mark.parametrize("with_res", [False, True])
def test_conv_dgrad_with_fused_bn_backward_sums(shape, with_res):
    """fdg_conv_dgrad with reduce = 2 (the sums of the batch-norm backward its output feeds), then
    fdg_bn_backward on the partial rows; stride-2 layers through the spread-out dy."""
    from paper_1906_09108_b200 import binding as B
    n, h, w, ci, co, stride, share = shape
    ops, ew = B.ConvOps(B.FDG_BF16_TC), B.EwOps(B.FDG_BF16_TC)
    s = B.fdg_conv_shape(n, h, w, ci, co, 3, stride, 1)
    p, q = ops.out_hw(s)
    assert ops.path(s, 1)
    wt, wo = _mk((co, 3, 3, ci), 31, ops.dtype, scale=(2.0 / (9 * ci)) ** 0.5)
    wf = ops.flip_weights(s, wt)
    dy, dyo = _mk((n, p, q, co), 32, ops.dtype)
    res, reso = _mk((n, h, w, ci), 33, ops.dtype)
    rmask, rmasko = _mk((n, h, w, ci), 34, ops.dtype)
    nmask, nmasko = _mk((n, h, w, ci), 35, ops.dtype)               # output of the ReLU behind the next batch norm
    nx, nxo = _mk((n, h, w, ci), 36, ops.dtype, scale=1.4, shift=0.2)  # the tensor that batch norm normalised
    gam = 1.0 + 0.2 * np.random.default_rng(37).standard_normal(ci)
    nstats = ew.bn_stats(nx, EPS)
    dx, part = ops.dgrad(s, dy, wt, wf, res=res if with_res else None, res_mask=rmask if with_res else None, share=share,
                         spread=stride == 2, next_bn=(nmask, nx, nstats))
    assert part.shape[0] >= 1 and not ops.timed_out()
    dxo = L.conv2d_backward(dyo, np.zeros((n, h, w, ci)), wo, stride, 1)[0] + (reso * (rmasko > 0) if with_res else 0.0)
    assert _rel(dx, dxo) <= 1e-2
    dxs = dx.float().cpu().numpy().astype(np.float64)
    sv = L.batchnorm_forward(nxo, gam, np.zeros(ci), EPS)[1]
    want_dx, want_dg, want_db = L.batchnorm_backward(L.relu_backward(dxs, nmasko), sv, gam)
    tot = part.double().sum(dim=0).cpu().numpy()
    scale = max(np.abs(want_dg).max(), np.abs(want_db).max())
    assert np.abs(tot[:ci] - want_db).max() <= 1e-4 * scale and np.abs(tot[ci:] - want_dg).max() <= 1e-4 * scale
    got_dx, dg, db = ew.bn_backward(dx, nmask, nx, nstats, _f32(gam), partial=part, block_cap=148)
    assert np.abs(dg.cpu().numpy() - want_dg).max() <= 1e-4 * scale and np.abs(db.cpu().numpy() - want_db).max() <= 1e-4 * scale
    assert _rel(got_dx, want_dx) <= 1e-2


@pytest.mark.parametrize("prec_name", ["fp32", "bf16"])
def test_shrink_ingest_and_update(prec_name):
    B, ew, tol = _ops(prec_name)
    g, go = _mk((3, 16, 16, 32), 41, ew.dtype)
    out = ew.shrink(g, 0.2)                                             # Eq. 15
    want = np.float32(0.2) * go.astype(np.float32)
    assert _rel(out, (L.round_bf16(want) if prec_name == "bf16" else want).astype(np.float64)) <= 1e-7
    img = torch.from_numpy(np.random.default_rng(42).standard_normal((4, 8, 8, 3)).astype(np.float32)).cuda()
    lab = torch.arange(4, dtype=torch.int32, device="cuda")
    o, lo = ew.ingest(img, 8, lab)
    o = o.float().cpu().numpy()
    src = img.cpu().numpy()
    assert np.array_equal(o[..., :3], L.round_bf16(src) if prec_name == "bf16" else src) and not o[..., 3:].any()
    assert torch.equal(lo, lab)
    # Eq. 11 with momentum and weight decay: two updates in a row against the closed form in float64
    n = 4099                                                          # not a multiple of 4: the scalar tail runs too
    rng = np.random.default_rng(43)
    th0, g1, g2 = rng.standard_normal(n), rng.standard_normal(n), rng.standard_normal(n)
    theta, mom = _f32(th0), torch.zeros(n, dtype=torch.float32, device="cuda")
    lr, mu, wd = 0.05, 0.9, 5e-4
    n32, n16 = ew.sgd_update(theta, mom, _f32(g1), lr, mu, wd)
    th0 = th0.astype(np.float32).astype(np.float64)
    v1 = g1.astype(np.float32) + wd * th0
    th1 = th0 - lr * v1
    assert _rel(theta, th1) <= 1e-6 and _rel(n32, th1) <= 1e-6 and _rel(mom, v1) <= 1e-6
    assert _rel(n16, th1) <= 2.0 ** -8
    ew.sgd_update(theta, mom, _f32(g2), lr, mu, wd)
    v2 = mu * v1 + g2.astype(np.float32) + wd * th1
    assert _rel(theta, th1 - lr * v2) <= 1e-6 and _rel(mom, v2) <= 1e-6


@pytest.mark.parametrize("prec_name", ["fp32", "bf16"])
@pytest.mark.parametrize("bhwfc", [(8, 8, 8, 64, 10), (5, 4, 4, 32, 7), (6, 8, 8, 640, 100), (7, 3, 5, 18, 7),
                                   (4, 8, 8, 2056, 5), (9, 2, 2, 48, 3), (130, 4, 4, 512, 10)])
def test_head(prec_name, bhwfc):
    B, ew, tol = _ops(prec_name)
    b, h, w, f, classes = bhwfc
    x, xo = _mk((b, h, w, f), 51, ew.dtype, scale=0.8, shift=0.5)
    rng = np.random.default_rng(52)
    wt = (rng.standard_normal((classes, f)) / np.sqrt(f)).astype(np.float32)
    bias = (0.1 * rng.standard_normal(classes)).astype(np.float32)
    labels = rng.integers(0, classes, size=b).astype(np.int32)
    o = ew.head(x, _f32(wt), _f32(bias), torch.from_numpy(labels).cuda())
    pooled = L.gap_forward(xo)
    logits = L.fc_forward(pooled, wt.astype(np.float64), bias.astype(np.float64))
    loss, probs = L.softmax_xent_forward(logits, labels.astype(np.int64))
    dlog = L.softmax_xent_backward(probs, labels.astype(np.int64))
    dpool, dw, db = L.fc_backward(dlog, pooled, wt.astype(np.float64))
    dx = L.gap_backward(dpool, xo.shape)
    assert abs(float(o["loss"].item()) - loss) <= 1e-5 * abs(loss)
    assert _rel(o["pooled"], pooled) <= 1e-5 and _rel(o["dlogits"], dlog) <= 1e-5
    assert _rel(o["dw"], dw) <= 1e-5 and _rel(o["db"], db) <= 1e-5
    assert _rel(o["dx"], dx) <= tol
    assert not o["flags"].any()
    bad = labels.copy()
    bad[0] = classes                                                   # out of range: flagged, treated as class 0
    o = ew.head(x, _f32(wt), _f32(bias), torch.from_numpy(bad).cuda())
    assert o["flags"][1].item() == 1 and o["flags"][0].item() == 0
