"""Pins of the training-recipe parts of the oracle (oracle/fdg.py): the learning-rate schedule of the
experiments section, running batch-norm statistics and the inference forward, the drain after the last batch,
and the checkpoint of the in-flight state -- each against something other than the oracle itself (torch's
schedulers, torch's own batch-norm buffers and inference mode, back-propagation by autograd, an
uninterrupted run)."""
import numpy as np
import pytest
import torch

from oracle import fdg
from tests import torch_ref
from tests.test_oracle_fdg import all_params, batch, make, relerr, tiny_arch


def test_learning_rate_schedule_matches_torch_schedulers():
    """Divide by 10 at epochs 150, 225, 275 (torch MultiStepLR stepped once per epoch); with warm-up the first
    3 epochs run at 0.01 (experiments section)."""
    ipe = 4
    p = torch.nn.Parameter(torch.zeros(1))
    opt = torch.optim.SGD([p], lr=0.1)
    sched = torch.optim.lr_scheduler.MultiStepLR(opt, milestones=[150, 225, 275], gamma=0.1)
    it = 0
    for epoch in range(300):
        for _ in range(ipe):
            it += 1
            want = opt.param_groups[0]["lr"]
            assert abs(fdg.learning_rate(it, ipe) - want) <= 1e-12 * want, (epoch, it)
            got_w = fdg.learning_rate(it, ipe, warmup_epochs=3)
            assert got_w == (0.01 if epoch < 3 else fdg.learning_rate(it, ipe))
        opt.step()
        sched.step()
    assert fdg.learning_rate(1, 391) == 0.1 and abs(fdg.learning_rate(391 * 275 + 1, 391) - 1e-4) < 1e-15


def test_schedule_drives_the_update_per_iteration():
    """With a schedule set, iteration t updates with learning_rate(t): the same run with the rate set by hand
    before every step gives the same parameters bit for bit."""
    arch = tiny_arch(n=1)
    kw = dict(iters_per_epoch=2, base_lr=0.1, milestones=(2, 3), gamma=0.1, warmup_epochs=1, warmup_lr=0.01)
    a, b = make(arch, 2, [1], beta=0.5), make(arch, 2, [1], beta=0.5)
    a.set_schedule(**kw)
    for t in range(1, 10):
        b.set_lr(fdg.learning_rate(t, **kw))
        a.step(*batch(arch, t))
        b.step(*batch(arch, t))
    assert np.array_equal(all_params(a), all_params(b))
    assert a.lr == pytest.approx(0.001)


@pytest.mark.parametrize("family", ["resnet6n2", "wrn"])
def test_running_statistics_and_inference_match_torch(family):
    """K = 1 is plain training: after every step the running mean / variance of every batch norm must equal
    the buffers torch.nn.functional.batch_norm maintains itself (momentum 0.1, unbiased variance), and the
    inference forward must equal torch's inference mode on the same weights and buffers."""
    arch = tiny_arch(family, n=1)
    o = make(arch, 1, [], lr=0.05, momentum=0.9, weight_decay=5e-4)
    theta = torch.tensor(all_params(o), requires_grad=True)
    opt = torch.optim.SGD([theta], lr=0.05, momentum=0.9, weight_decay=5e-4)
    buffers = []
    for t in range(1, 5):
        x, y = batch(arch, t)
        o.step(x, y)
        opt.zero_grad()
        torch_ref.network_loss(arch, theta, torch.tensor(x), torch.tensor(y), buffers).backward()
        opt.step()
        flat = np.concatenate([np.concatenate([rm.numpy(), rv.numpy()]) for rm, rv in buffers])
        assert relerr(o.get_running(1), flat) < 1e-12
    assert not np.allclose(o.get_running(1)[:4], 0.0)            # they did move
    x, y = batch(arch, 9)
    with torch.no_grad():
        want = torch_ref.network_logits(arch, theta, torch.tensor(x), buffers, training=False).numpy()
    got = o.eval_logits(x)
    assert relerr(got, want) < 1e-9
    assert o.top1(x, y) == int((want.argmax(axis=1) == y).sum())
    # round trip of the flat vector
    r = o.get_running(1)
    o.set_running(1, r * 2.0)
    assert np.array_equal(o.get_running(1), r * 2.0)


@pytest.mark.parametrize("K,splits", [(1, []), (2, [2]), (3, [1, 3]), (4, [1, 3, 5])])
def test_drain_backpropagates_every_batch_exactly_once(K, splits):
    """After T iterations module k still holds 2(K-k) batches.  The drain lets them through: every module ends
    with T updates and nothing in flight, and (weights frozen, lr = 0) the gradient module k forms for a batch
    that is only back-propagated during the drain is still beta^(K-k) times that batch's back-propagation
    gradient (Eq. 16 / Eq. 17), recomputed by autograd."""
    beta, T = 0.6, 2 * K + 1
    arch = tiny_arch(n=2)
    o = make(arch, K, splits, beta=beta, lr=0.0)
    theta = all_params(o)
    sizes = [o.param_count(k) for k in range(1, K + 1)]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    bp = {}
    for t in range(1, T + 1):
        x, y = batch(arch, t)
        th = torch.tensor(theta, requires_grad=True)
        (g,) = torch.autograd.grad(torch_ref.network_loss(arch, th, torch.tensor(x), torch.tensor(y)), th)
        bp[t] = g.numpy()
        o.step(x, y)
    held = [len(m.saved) for m in o.modules]
    assert held == [2 * (K - k) for k in range(1, K)] + [0]
    done = [m.updates for m in o.modules]                         # module k has back-propagated batches 1 .. T-2K+k+1
    assert done == [T - 2 * K + k + 1 for k in range(1, K + 1)]
    seen = []
    inner = o._update

    def recording_update(k, ghat):
        seen.append((k, ghat.copy()))
        inner(k, ghat)

    o._update = recording_update
    n_log = len(o.log)
    o.drain()
    assert [m.updates for m in o.modules] == [T] * K
    assert all(not m.saved for m in o.modules) and o.t == 0
    assert len(seen) == sum(T - d for d in done)                   # one update per (module, batch) still owed
    rows = [r for r in o.log[n_log:] if r["tau_b"] > 0]
    assert len(rows) == len(seen)
    for (k, ghat), r in zip(seen, rows):
        assert r["k"] == k and done[k - 1] < r["tau_b"] <= T
        assert relerr(ghat, beta ** (K - k) * bp[r["tau_b"]][offs[k - 1]:offs[k]]) < 1e-9
    assert all(r["tau_f"] <= T for r in o.log)                     # no batch beyond the last one was invented
    # the pipeline starts afresh
    o._update = inner
    o.step(*batch(arch, 1))
    assert o.log[-K]["tau_f"] == 1 and o.log[-K]["t"] == 1


@pytest.mark.parametrize("storage", [None, "bf16"])
def test_restored_state_continues_bit_for_bit(storage):
    arch = tiny_arch(n=1)
    cfg = fdg.FDGConfig(K=3, split_after_block=(1, 2), beta=0.5, lr=0.05)
    import fdg_synth as S

    def fresh():
        o = fdg.FDGOracle(arch, cfg, storage=storage)
        for k in range(1, 4):
            o.set_params(k, S.init_params(3, k, o.param_spec(k), jitter=True))
        return o

    a = fresh()
    for t in range(1, 8):
        a.step(*batch(arch, t))
    snap = a.state()
    for t in range(8, 13):
        la = a.step(*batch(arch, t))
    a.drain()
    b = fresh()
    b.step(*batch(arch, 40))                                       # some other history, overwritten by the restore
    b.load_state(snap)
    for t in range(8, 13):
        lb = b.step(*batch(arch, t))
    b.drain()
    assert la == lb
    for k in range(1, 4):
        assert np.array_equal(a.get_params(k), b.get_params(k))
        assert np.array_equal(a.get_momentum(k), b.get_momentum(k))
        assert np.array_equal(a.get_running(k), b.get_running(k))
    assert a.log == b.log
