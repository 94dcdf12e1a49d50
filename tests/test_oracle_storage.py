"""Pins of the oracle's storage-precision switch (oracle/nets.py, set_storage).

The switch makes the oracle round to bfloat16 the tensors a path keeps between two of its steps.  The
rounding function itself is pinned against torch in tests/test_oracle_layers.py; these tests pin WHERE it is
applied, against the list written down in the design notes and restated here, and what it can and cannot
change:

  forward, basic block    conv1 output, ReLU(BN1) output, conv2 output, [projection conv output], block output;
                          convolution weights before use
  backward, basic block   gradient of conv2's output, of ReLU(BN1)'s output (the data gradient of conv2), of
                          conv1's output, [of the projection conv's output, the projection's data gradient],
                          of the block input
  never rounded           batch-norm outputs before their ReLU, the residual sum before its ReLU, a ReLU
                          derivative times its incoming gradient, statistics, parameter gradients, the head
"""
import numpy as np

import fdg_synth as S
from oracle import fdg as ofdg
from oracle import layers as L
from oracle import nets


def _is_bf16(a):
    return np.array_equal(L.round_bf16(a), a)


def _block(ci, co, stride, storage, seed=0):
    arch = nets.Arch(batch=4)
    blk = nets.BasicBlock(arch, ci, co, stride, 1)
    nets.set_storage([blk], storage)
    rng = np.random.default_rng(seed)
    p = {}
    for name, kind, shape in blk.param_spec():
        p[name] = rng.standard_normal(shape) * (0.2 if kind == "conv" else 0.1) + (1.0 if kind == "bn_gamma" else 0.0)
    x = L.round_bf16(rng.standard_normal((4, 8, 8, ci)))
    dy = L.round_bf16(rng.standard_normal((4, 8 // stride, 8 // stride, co)))
    return blk, p, x, dy


class _Spy:
    """Stands in for the rounding function: records every tensor it is asked to round."""

    def __init__(self):
        self.seen = []

    def __call__(self, a):
        self.seen.append(np.array(a, copy=True))
        return L.round_bf16(a)


def test_rounding_points_of_a_basic_block_are_the_documented_ones():
    for ci, co, stride in ((8, 8, 1), (8, 16, 2)):
        blk, p, x, dy = _block(ci, co, stride, None)
        proj = blk.proj
        spy_a, spy_w = _Spy(), _Spy()
        blk.q, blk.qw = spy_a, spy_w
        y, ctx = blk.forward(x, p)
        # forward: conv1 out, ReLU(BN1) out, conv2 out, [projection conv out], block out
        assert len(spy_a.seen) == (5 if proj else 4)
        assert len(spy_w.seen) == (3 if proj else 2)                  # every convolution's weights, nothing else
        w1, w2 = L.round_bf16(p["conv1.w"]), L.round_bf16(p["conv2.w"])
        c1 = L.conv2d_forward(x, w1, stride, 1)
        assert np.array_equal(spy_a.seen[0], c1)                      # rounded as it leaves the convolution
        a1 = L.relu_forward(L.batchnorm_forward(L.round_bf16(c1), p["bn1.g"], p["bn1.b"], blk.eps)[0])
        assert np.array_equal(spy_a.seen[1], a1)                      # BN1's output is rounded only after its ReLU
        c2 = L.conv2d_forward(L.round_bf16(a1), w2, 1, 1)
        assert np.array_equal(spy_a.seen[2], c2)
        b2 = L.batchnorm_forward(L.round_bf16(c2), p["bn2.g"], p["bn2.b"], blk.eps)[0]
        if proj:
            cs = L.conv2d_forward(x, L.round_bf16(p["sc.w"]), stride, 0)
            assert np.array_equal(spy_a.seen[3], cs)
            sc = L.batchnorm_forward(L.round_bf16(cs), p["scbn.g"], p["scbn.b"], blk.eps)[0]
        else:
            sc = x
        assert np.array_equal(spy_a.seen[-1], L.relu_forward(b2 + sc))   # the residual sum is not rounded before its ReLU
        assert np.array_equal(y, L.round_bf16(L.relu_forward(b2 + sc)))
        # backward: dc2, da1, dc1, [dcs, dxs], dx
        spy_a.seen.clear()
        dx, grads = blk.backward(dy, ctx, p)
        assert len(spy_a.seen) == (6 if proj else 4)
        dsum = L.relu_backward(dy, ctx["y"])
        dc2 = L.batchnorm_backward(dsum, ctx["sv2"], p["bn2.g"])[0]
        assert np.array_equal(spy_a.seen[0], dc2)                     # the gated gradient is not rounded before BN2's backward
        assert _is_bf16(dx)
        for name, gval in grads.items():                              # parameter gradients keep full precision
            assert gval.dtype == np.float64 and not _is_bf16(gval), name


def test_everything_kept_between_steps_is_bf16_and_nothing_else_changes():
    for storage in (None, "bf16"):
        blk, p, x, dy = _block(8, 16, 2, storage)
        y, ctx = blk.forward(x, p)
        dx, _ = blk.backward(dy, ctx, p)
        kept = [y, ctx["a1"], ctx["y"], dx]
        assert all(_is_bf16(t) for t in kept) == (storage == "bf16")
    # an identity in place of the rounding function is the plain oracle, bit for bit
    blk, p, x, dy = _block(8, 8, 1, None)
    y0, ctx0 = blk.forward(x, p)
    dx0, g0 = blk.backward(dy, ctx0, p)
    blk.q = blk.qw = lambda a: a
    y1, ctx1 = blk.forward(x, p)
    dx1, g1 = blk.backward(dy, ctx1, p)
    assert np.array_equal(y0, y1) and np.array_equal(dx0, dx1)
    assert all(np.array_equal(g0[k], g1[k]) for k in g0)


def test_storage_mode_stays_within_the_rounding_budget_of_the_plain_oracle():
    """Forward with identical weights: every rounding point adds at most half a bfloat16 unit (2^-9 relative)
    to the tensor it rounds, so after d rounded tensors on the longest path the two oracles differ by a small
    multiple of d * 2^-9 of the largest activation -- far from a dropped or misplaced step, which changes
    values by O(1)."""
    arch = nets.Arch(n_per_stage=2, widths=(16, 32, 64), stem_width=16, in_h=16, in_w=16, batch=8)
    cfg = ofdg.FDGConfig(K=1, split_after_block=(), lr=0.0, weight_decay=0.0)
    outs = {}
    for storage in (None, "bf16"):
        orc = ofdg.FDGOracle(arch, cfg, storage=storage)
        flat = S.init_params(0, 1, orc.param_spec(1), jitter=True)
        if storage is None:                                       # same weights on both sides: the rounded ones
            named = nets.unflatten(flat.astype(np.float64), orc.param_spec(1))
            for (name, kind, _) in orc.param_spec(1):
                if kind == "conv":
                    named[name][...] = L.round_bf16(named[name])
            flat = nets.flatten(named, orc.param_spec(1), np.float64)
        orc.set_params(1, flat)
        x = L.round_bf16(S.images(0, 1, 8, 16, 16, 3).astype(np.float64))
        m = orc.modules[0]
        named = nets.unflatten(m.theta, m.spec)
        acts = []
        for u in m.units[:-1]:
            x, _ = u.forward(x, nets.unit_params(named, u))
            acts.append(x)
        outs[storage] = acts
    for depth, (a, b) in enumerate(zip(outs[None], outs["bf16"]), start=1):
        err = np.abs(a - b).max() / np.abs(a).max()
        roundings = 1 + 4 * depth                                  # stem + 4 rounded tensors per block on the way
        assert 0 < err <= roundings * 2.0 ** -9, (depth, err)
