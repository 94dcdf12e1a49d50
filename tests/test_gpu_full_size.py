"""The headline workload at its full size, in the launch configuration the benchmark times
(ResNet-110, K = 4, batch 128, bfloat16 storage, one CUDA graph per ring phase, convolution
launches sized for four module streams side by side, several image tiles per CTA).

The oracle cannot run this network end to end in test time, and batch normalisation couples
all 128 images, so no output can be had sample by sample.  What it can do in milliseconds is
one layer on a full-size tensor.  The forward test therefore takes the tensors every block
saved in the activation FIFO and recomputes each layer of each block with the oracle from the
library's own input to that layer: every convolution, every batch norm (whose statistics
come from sums formed in the convolution epilogues, one partial row per CTA), every
residual sum, all elements.  The end-to-end test runs a shallow network of the same layer
shapes, batch and launch shapes against the oracle, forward, backward and update."""
import numpy as np
import pytest

import fdg_synth as S
from oracle import layers as L

pytestmark = pytest.mark.gpu

ARCH = dict(family="resnet6n2", n_per_stage=18, widths=(16, 32, 64), stem_width=16, in_h=32, in_w=32, in_c=3,
            num_classes=10, batch=128)
SPLITS = (13, 27, 41)
EPS = 1e-5


def _relmax(a, b):
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def _make(B, **kw):
    g = B.FDG(B.make_arch(**ARCH), K=4, split_after_block=SPLITS, beta=0.2, momentum=0.9, precision=B.FDG_BF16_TC, **kw)
    params = {}
    for k in range(1, 5):
        params[k] = S.init_params(0, k, g.param_layout(k), jitter=True)
        g.set_params(k, params[k])
    return g, params


def _units(layout):
    """[(unit name, {position in unit: (offset, shape)})] in module order."""
    units = []
    for name, kind, shape in layout:
        unit, off = name.split("@")
        if not units or units[-1][0] != unit:
            units.append((unit, []))
        units[-1][1].append((int(off), tuple(shape)))
    return units


def _take(flat, entry):
    off, shape = entry
    return flat[off:off + int(np.prod(shape))].reshape(shape).astype(np.float64)


def test_forward_of_every_block_at_full_size():
    import torch
    from paper_1906_09108_b200 import binding as B
    g, params = _make(B, lr=0.0, weight_decay=0.0, graphs=True)
    b = ARCH["batch"]
    for t in range(1, 7):                                   # module 4 forwards its first batch at t = 4
        x = torch.from_numpy(S.images(0, t, b, 32, 32, 3)).cuda()
        y = torch.from_numpy(S.labels(0, t, b, 10)).cuda()
        g.step(x, y)
    g.sync()
    worst = {}
    checked = 0
    for k in range(1, 5):
        units = _units(g.param_layout(k))
        flat = params[k]
        for u in range(1, len(units)):
            name, ent = units[u]
            if not name.startswith("block"):
                continue
            w1 = L.round_bf16(_take(flat, ent[0])); g1, b1 = _take(flat, ent[1]), _take(flat, ent[2])
            w2 = L.round_bf16(_take(flat, ent[3])); g2, b2 = _take(flat, ent[4]), _take(flat, ent[5])
            co, ci = w1.shape[0], w1.shape[3]
            proj = len(ent) > 6
            stride = 2 if proj else 1
            bx, x_in = g.saved_tensor(k, u - 1, 3)
            hw_in = int(round((x_in.size / (b * ci)) ** 0.5))
            x_in = x_in.reshape(b, hw_in, hw_in, ci).astype(np.float64)
            hw = hw_in // stride
            got = {}
            for which, key in ((0, "c1"), (1, "a1"), (2, "c2"), (3, "y")) + (((4, "cs"),) if proj else ()):
                bb, a = g.saved_tensor(k, u, which)
                assert bb == bx
                got[key] = a.reshape(b, hw, hw, co).astype(np.float64)
            ref = {}
            ref["c1"] = L.round_bf16(L.conv2d_forward(x_in, w1, stride, 1))
            ref["a1"] = L.round_bf16(L.relu_forward(L.batchnorm_forward(got["c1"], g1, b1, EPS)[0]))
            ref["c2"] = L.round_bf16(L.conv2d_forward(got["a1"], w2, 1, 1))
            if proj:
                ws = L.round_bf16(_take(flat, ent[6])); gs, bs = _take(flat, ent[7]), _take(flat, ent[8])
                ref["cs"] = L.round_bf16(L.conv2d_forward(x_in, ws, stride, 0))
                sc = L.batchnorm_forward(got["cs"], gs, bs, EPS)[0]
            else:
                sc = x_in
            ref["y"] = L.round_bf16(L.relu_forward(L.batchnorm_forward(got["c2"], g2, b2, EPS)[0] + sc))
            for key in ref:
                err = _relmax(got[key], ref[key])
                worst[key] = max(worst.get(key, 0.0), err)
                assert err <= 1e-2, (k, name, key, err)         # one bfloat16 ulp of the largest element is 4e-3
            checked += 1
    assert g.check_guards() == -1          # no kernel wrote past the end of a workspace buffer
    g.close()
    assert checked == 51                                      # every block whose input is saved in the same module (13 + 13 + 13 + 12)
    print("worst relative errors over %d blocks:" % checked, worst)


def test_backward_of_every_block_at_full_size():
    """The backward twin of the test above (Eq. 10 with the shrunk gradient of Eq. 15): ResNet-110, K = 4, batch 128,
    one stream per module plus the side stream of the weight gradients, i.e. the kernels and launch shapes the
    benchmark's graphs replay (a convolution on a quarter of the SMs, the weight gradients' pixel split capped at
    16 CTAs).  A capture keeps every gradient tensor of each module's backward pass at iteration 2K - 1, the first
    one in which all four modules back-propagate.  Every layer of every block is then recomputed by the oracle
    from the library's own inputs to that layer -- the incoming gradient it captured and the activations it saved
    for that batch, so every ReLU gate is the same on both sides -- and compared element by element at 1e-2: the
    batch-norm backwards (whose sums come from the data-gradient epilogues for identity blocks and from the
    reduction kernel for projection blocks), the 3x3 data gradients with their fused residual, the stride-2 and
    1x1 projection gradients, all weight gradients, the stem and the classifier."""
    from paper_1906_09108_b200 import binding as B
    from tests.layerwise import check_backward_layerwise
    g, params = _make(B, lr=0.0, weight_decay=0.0)
    checked, worst = check_backward_layerwise(g, params, ARCH, 4)
    assert g.check_guards() == -1          # no kernel wrote past the end of a workspace buffer
    g.close()
    assert checked == 54
    print("worst relative errors over %d blocks:" % checked, {k_: float("%.2g" % v) for k_, v in worst.items()})


def test_bench_launch_shapes_against_oracle():
    """Forward, backward and update at the benchmark's layer shapes, batch and launch shapes, end to end
    against the oracle: a 6n+2 network with n = 2 (14 layers) cut into K = 4 modules, batch 128, graphs on.
    Every convolution launch is then what the benchmark issues (128 image tiles on 32 CTAs, 4 tiles
    per CTA, per-CTA partial sums for both kinds of fused reduction, the pixel-split weight gradient),
    and the network is shallow enough for the oracle to run and for bfloat16 gate flips not to pile up
    (the comparison of a 110-layer gradient between two launch shapes of this same library differs by
    O(1): what is compared has to be shallow, or one layer at a time as above)."""
    from tests.fdg_pair import run_pair
    arch = dict(ARCH, n_per_stage=2)
    res = run_pair(arch, 4, (1, 3, 5), 10, beta=0.2, lr=0.02, precision="bf16", graphs=True, check_every_step=True)
    msg = str({k: v for k, v in res.items() if not k.startswith("log_")})
    assert res["log_gpu"] == res["log_oracle"]
    assert res["params"] <= 2e-2, msg
    assert res["loss"] <= 1e-2 and res["out"] <= 5e-2, msg
    assert res["grads"] <= 0.25, msg
