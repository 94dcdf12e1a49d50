"""Error paths of the library, exercised without making any kernel misbehave: bad inputs the kernels detect
and survive (a non-finite loss, a label out of range), and status words raised from the host the way a
kernel would raise them (fdg_debug_raise_flag), and a bounded wait that is made to run out on a barrier nothing
sets (fdg_debug_wait_probe); all checked through what fdg_sync and fdg_step report."""
import numpy as np
import pytest
import torch

import fdg_synth as S

pytestmark = pytest.mark.gpu

ARCH = dict(family="resnet6n2", n_per_stage=1, widths=(8, 16, 32), stem_width=8, in_h=16, in_w=16, in_c=3,
            num_classes=10, batch=8)


def _make(B, K, splits, **kw):
    g = B.FDG(B.make_arch(**ARCH), K=K, split_after_block=splits, beta=0.5, lr=0.05, **kw)
    for k in range(1, K + 1):
        g.set_params(k, S.init_params(0, k, g.param_layout(k)))
    return g


def _batch(t):
    return (torch.from_numpy(S.images(0, t, 8, 16, 16, 3)).cuda(), torch.from_numpy(S.labels(0, t, 8, 10)).cuda())


def _status(g, fn, *args):
    from paper_1906_09108_b200 import binding as B
    try:
        fn(*args)
        return B.FDG_OK
    except B.FDGError as e:
        return e.status


@pytest.mark.parametrize("precision", ["fp32", "bf16"])
def test_nonfinite_loss_is_reported_once_and_the_context_carries_on(precision):
    from paper_1906_09108_b200 import binding as B
    g = _make(B, 1, (), precision=B.FDG_BF16_TC if precision == "bf16" else B.FDG_FP32_CUDACORE)
    loss = torch.zeros(1, device="cuda")
    x, y = _batch(1)
    g.step(x, y, loss)
    g.sync()
    assert np.isfinite(loss.item())
    # A NaN in the classifier's bias makes the loss NaN.  (A NaN pixel would not: the ReLU kernels take
    # max(x, 0) with the hardware's maximum, which returns the other operand for a NaN, so the first ReLU
    # behind a poisoned batch norm turns it into zeros.)
    good = S.init_params(0, 1, g.param_layout(1))
    poisoned = good.copy()
    poisoned[-1] = np.nan
    g.set_params(1, poisoned)
    g.step(x, y, loss)
    assert _status(g, g.sync) == 6                                  # FDG_ERR_NONFINITE
    assert "NaN" in g.lib.fdg_last_error(g.ctx).decode()
    assert _status(g, g.sync) == B.FDG_OK                           # reported once, then cleared
    # the update that followed spread the NaN further: a cold restart (parameters, momentum) recovers
    g.set_params(1, good)
    g.set_momentum(1, np.zeros(g.param_count(1), dtype=np.float32))
    g.step(x, y, loss)
    assert _status(g, g.sync) == B.FDG_OK and np.isfinite(loss.item())
    g.close()


def test_label_out_of_range_is_reported_and_treated_as_class_zero():
    from paper_1906_09108_b200 import binding as B
    g = _make(B, 2, (1,))
    x, y = _batch(1)
    bad = y.clone()
    bad[3] = ARCH["num_classes"]
    g.step(x, bad)                                                   # module 2 meets these labels at t = 2
    assert _status(g, g.sync) == B.FDG_OK
    g.step(*_batch(2))
    assert _status(g, g.sync) == 1                                   # FDG_ERR_INVALID_ARG
    assert "label" in g.lib.fdg_last_error(g.ctx).decode()
    g.step(*_batch(3))
    assert _status(g, g.sync) == B.FDG_OK
    g.close()


def test_raised_status_words_reach_the_caller():
    """The three device status words, raised from the host as a kernel would raise them.  The time-out of a
    tensor-core kernel's bounded wait is latched: the kernel left early, so the context refuses to go on."""
    from paper_1906_09108_b200 import binding as B
    g = _make(B, 2, (1,))
    g.step(*_batch(1))
    g.sync()
    for which, status in ((0, 6), (1, 1)):
        assert g.lib.fdg_debug_raise_flag(g.ctx, which) == B.FDG_OK
        assert _status(g, g.sync) == status
        assert _status(g, g.sync) == B.FDG_OK
        g.step(*_batch(2 + which))
    assert g.lib.fdg_debug_raise_flag(g.ctx, 3) == 1
    assert g.lib.fdg_debug_raise_flag(g.ctx, 2) == B.FDG_OK
    assert _status(g, g.sync) == 7                                   # FDG_ERR_TIMEOUT
    assert "waiting" in g.lib.fdg_last_error(g.ctx).decode()
    assert _status(g, g.sync) == 7                                   # latched
    assert _status(g, g.step, *_batch(9)) == 7
    g.close()


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """A one-warp kernel waits, with the bounded wait of the tensor-core kernels, on a barrier nothing arrives
    at; after a few thousand polls it gives up, raises the time-out word and returns (nothing is in flight, no
    tensor memory held).  The context latches FDG_ERR_TIMEOUT; the device and a new context carry on."""
    import torch
    from paper_1906_09108_b200 import binding as B
    g = _make(B, 2, (1,))
    g.step(*_batch(1))
    assert _status(g, g.sync) == B.FDG_OK
    assert g.lib.fdg_debug_wait_probe(g.ctx, None, 0) == 1            # limits outside 1..2^20 are refused
    assert g.lib.fdg_debug_wait_probe(g.ctx, None, (1 << 20) + 1) == 1
    assert _status(g, g.sync) == B.FDG_OK
    assert g.lib.fdg_debug_wait_probe(g.ctx, torch.cuda.current_stream().cuda_stream, 4096) == B.FDG_OK
    assert _status(g, g.sync) == 7                                   # FDG_ERR_TIMEOUT
    assert "waiting" in g.lib.fdg_last_error(g.ctx).decode()
    assert _status(g, g.step, *_batch(2)) == 7                       # latched
    g.close()
    torch.cuda.synchronize()                                         # no CUDA error was left behind
    g2 = _make(B, 2, (1,))
    loss = torch.zeros(1, device="cuda")
    g2.step(*_batch(1))
    g2.step(*_batch(2), loss)
    assert _status(g2, g2.sync) == B.FDG_OK and np.isfinite(loss.item())
    g2.close()


@pytest.mark.parametrize("precision", ["fp32", "bf16"])
def test_guard_regions_stay_clean_and_a_damaged_one_is_named(precision):
    """Every workspace buffer is followed by 256 guard bytes.  After real work (stream issue and graph replay) they
    all still hold their pattern; one byte changed from the host, standing in for a kernel that ran past its
    buffer, is reported with the index of that region, and a restored byte clears the report."""
    from paper_1906_09108_b200 import binding as B
    g = _make(B, 2, (1,), precision=B.FDG_BF16_TC if precision == "bf16" else B.FDG_FP32_CUDACORE, graphs=True)
    offs = g.guard_offsets()
    assert len(offs) > 20 and offs == sorted(offs) and all(o % 256 == 0 for o in offs)
    assert offs[-1] + 256 <= g.workspace_bytes
    assert g.check_guards() == -1
    for t in range(1, 12):
        g.step(*_batch(t))
    g.sync()
    assert g.check_guards() == -1
    for idx in (len(offs) // 2, 3):
        at = g.workspace_skip + offs[idx] + 17
        old = int(g.workspace[at].item())
        g.workspace[at] = old ^ 0x5A
        assert g.check_guards() == idx
        g.workspace[at] = old
        assert g.check_guards() == -1
    g.step(*_batch(12))
    assert _status(g, g.sync) == B.FDG_OK
    g.close()
