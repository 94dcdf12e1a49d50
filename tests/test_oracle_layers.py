"""Pins for oracle/layers.py: central finite differences (fp64) and the
corresponding torch.nn.functional routines under autograd."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import layers as L

RNG = np.random.default_rng(7)


def fd_grad(fun, x, h=1e-6):
    """Central finite differences of the scalar fun at x (any shape)."""
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        old = x[i]
        x[i] = old + h; fp = fun()
        x[i] = old - h; fm = fun()
        x[i] = old
        g[i] = (fp - fm) / (2 * h)
    return g


def relerr(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-30)


@pytest.mark.parametrize("stride,pad,r,h,w", [(1, 1, 3, 5, 6), (2, 1, 3, 6, 6), (2, 1, 3, 5, 7),
                                              (2, 0, 1, 6, 4), (1, 0, 1, 3, 3)])
def test_conv_fd_and_torch(stride, pad, r, h, w):
    x = RNG.standard_normal((2, h, w, 3)); wt = RNG.standard_normal((4, r, r, 3))
    y = L.conv2d_forward(x, wt, stride, pad)
    yt = F.conv2d(torch.tensor(x).permute(0, 3, 1, 2), torch.tensor(wt).permute(0, 3, 1, 2),
                  stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    assert y.shape == yt.shape and relerr(y, yt) < 1e-13
    c = RNG.standard_normal(y.shape)
    dx, dw = L.conv2d_backward(c, x, wt, stride, pad)
    f = lambda: float((L.conv2d_forward(x, wt, stride, pad) * c).sum())
    assert relerr(dx, fd_grad(f, x)) < 1e-7
    assert relerr(dw, fd_grad(f, wt)) < 1e-7


def test_conv_brute_force_tiny():
    """The definition as six nested loops, independent of the tap/matmul form."""
    x = RNG.standard_normal((1, 4, 3, 2)); w = RNG.standard_normal((3, 3, 3, 2))
    for stride in (1, 2):
        y = L.conv2d_forward(x, w, stride, 1)
        ref = np.zeros_like(y)
        for p in range(y.shape[1]):
            for q in range(y.shape[2]):
                for o in range(3):
                    for r in range(3):
                        for s in range(3):
                            hh, ww = p * stride + r - 1, q * stride + s - 1
                            if 0 <= hh < 4 and 0 <= ww < 3:
                                ref[0, p, q, o] += (x[0, hh, ww, :] * w[o, r, s, :]).sum()
        assert relerr(y, ref) < 1e-13


def test_batchnorm_fd_and_torch():
    x = RNG.standard_normal((3, 4, 2, 5)) * 2 + 1
    g = RNG.uniform(0.5, 1.5, 5); b = RNG.standard_normal(5)
    eps = 1e-5
    y, sv = L.batchnorm_forward(x, g, b, eps)
    xt = torch.tensor(x, requires_grad=True); gt = torch.tensor(g, requires_grad=True)
    bt = torch.tensor(b, requires_grad=True)
    yt = F.batch_norm(xt.permute(0, 3, 1, 2), None, None, gt, bt, training=True, eps=eps).permute(0, 2, 3, 1)
    assert relerr(y, yt.detach().numpy()) < 1e-12
    # zero mean / unit variance per channel before the affine map
    xhat = sv[0]
    assert np.abs(xhat.mean(axis=(0, 1, 2))).max() < 1e-12
    c = RNG.standard_normal(y.shape)
    dx, dg, db = L.batchnorm_backward(c, sv, g)
    (yt * torch.tensor(c)).sum().backward()
    assert relerr(dx, xt.grad.numpy()) < 1e-10
    assert relerr(dg, gt.grad.numpy()) < 1e-12 and relerr(db, bt.grad.numpy()) < 1e-12
    f = lambda: float((L.batchnorm_forward(x, g, b, eps)[0] * c).sum())
    assert relerr(dx, fd_grad(f, x)) < 1e-6
    assert relerr(dg, fd_grad(f, g)) < 1e-7 and relerr(db, fd_grad(f, b)) < 1e-7
    # the gradient wrt x of a training-mode BN sums to zero per channel
    assert np.abs(dx.sum(axis=(0, 1, 2))).max() < 1e-10


def test_relu():
    x = np.array([-1.0, 0.0, 2.0]); y = L.relu_forward(x)
    assert (y == [0, 0, 2]).all()
    assert (L.relu_backward(np.ones(3), y) == [0, 0, 1]).all()


def test_head_fd_and_torch():
    x = RNG.standard_normal((4, 3, 2, 6)); w = RNG.standard_normal((5, 6)); b = RNG.standard_normal(5)
    labels = np.array([0, 4, 2, 2])

    def f():
        logits = L.fc_forward(L.gap_forward(x), w, b)
        return float(L.softmax_xent_forward(logits, labels)[0])

    pooled = L.gap_forward(x)
    logits = L.fc_forward(pooled, w, b)
    loss, p = L.softmax_xent_forward(logits, labels)
    lt = F.cross_entropy(torch.tensor(logits), torch.tensor(labels))
    assert abs(loss - float(lt)) < 1e-12
    # uniform logits give log(classes)
    assert abs(L.softmax_xent_forward(np.zeros((2, 10)), np.array([3, 7]))[0] - np.log(10)) < 1e-14
    # shift invariance and large logits stay finite
    assert abs(L.softmax_xent_forward(logits + 1000.0, labels)[0] - loss) < 1e-9
    dl = L.softmax_xent_backward(p, labels)
    assert np.abs(dl.sum(axis=1)).max() < 1e-15
    dp, dw, db = L.fc_backward(dl, pooled, w)
    dx = L.gap_backward(dp, x.shape)
    assert relerr(dx, fd_grad(f, x)) < 1e-7
    assert relerr(dw, fd_grad(f, w)) < 1e-7
    assert relerr(db, fd_grad(f, b)) < 1e-7


def test_round_bf16_matches_torch():
    """The oracle's bfloat16 rounding against torch's own conversion: random values over
    many exponents, exact ties (round to even), values that round up into the next
    binade, zeros and subnormals' neighbours."""
    import torch
    g = np.random.default_rng(7)
    a = (g.standard_normal(200000) * np.exp(g.uniform(-30, 30, 200000))).astype(np.float32)
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 1.0 + 2.0 ** -7 + 2.0 ** -8,
                     2.0 - 2.0 ** -9, 0.0, -0.0, 1e-38, 3.0e38], dtype=np.float32)
    a = np.concatenate([a, ties])
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    got = L.round_bf16(a)
    assert got.dtype == np.float32 and np.array_equal(got, want)
    got64 = L.round_bf16(a.astype(np.float64))
    assert got64.dtype == np.float64 and np.array_equal(got64.astype(np.float32), want)
