"""The training-recipe calls of the library against the oracle (oracle/fdg.py), through the C ABI: the
learning-rate schedule driving the updates, running batch-norm statistics, the inference forward and its top-1
count, the drain after the last batch, and save / load of a run in flight."""
import ctypes as C

import numpy as np
import pytest
import torch

import fdg_synth as S
from oracle import fdg as ofdg
from oracle import nets as onets

pytestmark = pytest.mark.gpu

ARCHS = {
    "resnet": dict(family="resnet6n2", n_per_stage=2, widths=(8, 16, 32), stem_width=8, in_h=16, in_w=16, in_c=3,
                   num_classes=10, batch=6),
    "wrn": dict(family="wrn", n_per_stage=1, widths=(16, 24, 40), stem_width=8, in_h=16, in_w=16, in_c=3, num_classes=12,
                batch=6),
    "tc": dict(family="resnet6n2", n_per_stage=1, widths=(16, 32, 64), stem_width=16, in_h=32, in_w=32, in_c=3,
               num_classes=10, batch=8),
}


def _relfro(a, b):
    return float(np.linalg.norm(np.asarray(a, dtype=np.float64) - b) / max(np.linalg.norm(b), 1e-30))


def _pair(B, arch_kw, K, splits, precision="fp32", graphs=False, **kw):
    cfg = dict(beta=0.5, lr=0.05, momentum=0.9, weight_decay=5e-4)
    cfg.update(kw)
    orc = ofdg.FDGOracle(onets.Arch(**arch_kw), ofdg.FDGConfig(K=K, split_after_block=tuple(splits), **cfg),
                         storage="bf16" if precision == "bf16" else None)
    g = B.FDG(B.make_arch(**arch_kw), K=K, split_after_block=tuple(splits), graphs=graphs,
              precision=B.FDG_BF16_TC if precision == "bf16" else B.FDG_FP32_CUDACORE, **cfg)
    for k in range(1, K + 1):
        p = S.init_params(0, k, orc.param_spec(k), jitter=True)
        orc.set_params(k, p)
        g.set_params(k, p)
    return orc, g


def _batch(a, t, seed=0):
    return S.images(seed, t, a["batch"], a["in_h"], a["in_w"], a["in_c"]), S.labels(seed, t, a["batch"], a["num_classes"])


def _step(g, x, y, loss=None):
    g.step(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), loss)


def test_lr_schedule_function_and_driver():
    from paper_1906_09108_b200 import binding as B
    lib = B.load_library()
    sch = B.make_schedule(4, 0.1, (150, 225, 275), 0.1, 3, 0.01)
    out = C.c_float()
    for it in (1, 12, 13, 600, 601, 900, 901, 1100, 1101, 1200):
        assert lib.fdg_lr_at(C.byref(sch), it, C.byref(out)) == 0
        want = ofdg.learning_rate(it, 4, warmup_epochs=3)
        assert abs(out.value - want) <= 1e-6 * want, it
    assert lib.fdg_lr_at(C.byref(sch), 0, C.byref(out)) == 1
    # the schedule drives the updates: same parameters as the oracle under the same schedule
    a = ARCHS["resnet"]
    kw = dict(iters_per_epoch=3, base_lr=0.08, milestones=(2, 3), gamma=0.1, warmup_epochs=1, warmup_lr=0.01)
    orc, g = _pair(B, a, 2, (2,))
    orc.set_schedule(**kw)
    g.set_lr_schedule(B.make_schedule(**kw))
    for t in range(1, 13):
        x, y = _batch(a, t)
        orc.step(x, y)
        _step(g, x, y)
    g.sync()
    for k in (1, 2):
        assert _relfro(g.get_params(k), orc.get_params(k)) <= 1e-4
    g.close()


@pytest.mark.parametrize("name,K,splits,precision,graphs", [
    ("resnet", 1, (), "fp32", False), ("resnet", 3, (2, 4), "fp32", False), ("wrn", 2, (1,), "fp32", False),
    ("tc", 2, (1,), "bf16", True), ("wrn", 2, (2,), "bf16", False)])
def test_running_statistics_and_inference(name, K, splits, precision, graphs):
    """After a few training iterations the running statistics of every batch norm match the oracle's (every
    forward path is exercised: statistics from the reduction kernel and from convolution epilogues, projection
    shortcuts, the pre-activation norms and the head norm of the wide networks), and the inference forward
    gives the oracle's logits and top-1 count."""
    from paper_1906_09108_b200 import binding as B
    a = ARCHS[name]
    if name == "wrn" and precision == "bf16":
        a = dict(a, widths=(16, 32, 64), stem_width=16)
    orc, g = _pair(B, a, K, splits, precision, graphs, lr=0.02)
    steps = 2 * K + (10 if graphs else 3)
    for t in range(1, steps + 1):
        x, y = _batch(a, t)
        orc.step(x, y)
        _step(g, x, y)
    g.sync()
    tol = 2e-2 if precision == "bf16" else 1e-4
    for k in range(1, K + 1):
        want = orc.get_running(k)
        got = g.get_running(k)
        assert got.shape == want.shape
        if want.size:
            assert _relfro(got, want) <= tol, (k, _relfro(got, want))
    # inference with the library's own trained weights and statistics on both sides
    for k in range(1, K + 1):
        orc.set_params(k, g.get_params(k).astype(np.float64))
        orc.set_running(k, g.get_running(k).astype(np.float64))
    correct = torch.zeros(1, dtype=torch.int32, device="cuda")
    want_correct = 0
    for t in (101, 102):
        x, y = _batch(a, t)
        logits = torch.empty((a["batch"], a["num_classes"]), device="cuda")
        g.eval(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), logits, correct)
        torch.cuda.synchronize()
        want = orc.eval_logits(x)
        err = np.abs(logits.cpu().numpy() - want).max() / np.abs(want).max()
        assert err <= (2e-2 if precision == "bf16" else 1e-4), err
        mine = logits.cpu().numpy()
        assert int((mine.argmax(axis=1) == y).sum()) == int(correct.item()) - want_correct     # the count is its own logits' arg-max
        want_correct = int(correct.item())
        if precision == "fp32":                                  # no logit pair of the oracle is closer than the error bar
            assert int((want.argmax(axis=1) == y).sum()) == int((mine.argmax(axis=1) == y).sum())
    # training goes on afterwards: nothing in flight was touched by the inference passes
    ref = [g.get_params(k) for k in range(1, K + 1)]
    g.close()
    orc2, g2 = _pair(B, a, K, splits, precision, graphs, lr=0.02)
    for t in range(1, steps + 1):
        x, y = _batch(a, t)
        if t == steps - 1:
            g2.eval(torch.from_numpy(x).cuda())
        _step(g2, x, y)
    g2.sync()
    for k in range(1, K + 1):
        assert np.array_equal(g2.get_params(k), ref[k - 1])
    g2.close()


@pytest.mark.parametrize("K,splits,graphs", [(1, (), False), (3, (2, 4), False), (4, (1, 3, 5), True)])
def test_drain(K, splits, graphs):
    """fdg_drain against the oracle's drain: schedule rows of the 2K-2 extra iterations, losses, parameters and
    momentum afterwards; then a fresh pipeline starts at iteration 1."""
    from paper_1906_09108_b200 import binding as B
    a = ARCHS["resnet"]
    orc, g = _pair(B, a, K, splits, graphs=graphs, lr=0.02)
    T = 2 * K + (12 if graphs else 2)
    for t in range(1, T + 1):
        x, y = _batch(a, t)
        orc.step(x, y)
        _step(g, x, y)
    n_rows = len(orc.log)
    losses = torch.full((max(2 * K - 2, 1),), float("nan"), device="cuda")
    g.drain(losses)
    orc.drain()
    want_losses = []                                   # the oracle's drain does not return them: recompute from its log
    rows_o = [(r["t"], r["k"], r["tau_f"], r["tau_b"], r["ver_f"], r["ver_b"]) for r in orc.log]
    rows_g = [(r["t"], r["k"], r["tau_f"], r["tau_b"], r["ver_f"], r["ver_b"]) for r in g.schedule_log()]
    assert rows_g == rows_o and len(rows_o) == n_rows + (2 * K - 2) * K
    got_losses = losses.cpu().numpy()
    for i in range(2 * K - 2):                         # the top module handles batch T+i+1-K+1 in drain iteration i
        assert np.isfinite(got_losses[i]) == (T + i + 1 - K + 1 <= T)
    for k in range(1, K + 1):
        assert _relfro(g.get_params(k), orc.get_params(k)) <= 1e-4
        assert _relfro(g.get_momentum(k), orc.get_momentum(k)) <= 1e-4
    for t in range(1, 4):
        x, y = _batch(a, 50 + t)
        orc.step(x, y)
        _step(g, x, y)
    g.sync()
    assert g.schedule_log()[-1]["t"] == 3
    for k in range(1, K + 1):
        assert _relfro(g.get_params(k), orc.get_params(k)) <= 1e-4
    g.close()


@pytest.mark.parametrize("precision,graphs", [("fp32", False), ("bf16", True)])
def test_saved_state_continues_bit_for_bit(precision, graphs):
    """Save in flight, run on; load into a second context with another history, run the same inputs: the
    parameters, momentum, running statistics, losses and schedule rows agree bit for bit."""
    from paper_1906_09108_b200 import binding as B
    a = ARCHS["tc"] if precision == "bf16" else ARCHS["resnet"]
    K, splits = 3, (1, 2)
    _, g = _pair(B, a, K, splits, precision, graphs)
    loss = torch.zeros(1, device="cuda")
    n0 = 2 * K + (9 if graphs else 2)
    for t in range(1, n0 + 1):
        _step(g, *_batch(a, t))
    blob = g.save_state()

    def go_on(ctx):
        ls = []
        for t in range(n0 + 1, n0 + 8):
            _step(ctx, *_batch(a, t), loss)
            ctx.sync()
            ls.append(float(loss.item()))
        ctx.drain()
        return ls, [ctx.get_params(k) for k in range(1, K + 1)] + [ctx.get_momentum(k) for k in range(1, K + 1)] + \
            [ctx.get_running(k) for k in range(1, K + 1)]

    la, outs_a = go_on(g)
    g.close()
    _, h = _pair(B, a, K, splits, precision, graphs)
    for t in range(1, 4):
        _step(h, *_batch(a, 70 + t))                   # a different past, overwritten by the load
    h.load_state(blob)
    lb, outs_b = go_on(h)
    assert la == lb
    for x, y in zip(outs_a, outs_b):
        assert np.array_equal(x, y)
    # a state of another configuration is refused
    _, other = _pair(B, a, 2, (1,), precision, graphs)
    with pytest.raises(B.FDGError):
        other.load_state(blob)
    other.close()
    h.close()
