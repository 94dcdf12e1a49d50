"""CPU-only checks of the C-ABI library: it builds for sm_100a, loads, exports every
symbol include/fdg.h declares, and its host-side argument checks answer without a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_1906_09108_b200 import binding as B
from paper_1906_09108_b200 import build as fdg_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fdg_build.build()
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "fdg.h")).read() + open(os.path.join(ROOT, "include", "fdg_ops.h")).read()
    declared = set(re.findall(r"\b(fdg_[a-z_0-9]+)\s*\(", header))
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert lib.fdg_status_string(0) == b"ok"
    assert len({lib.fdg_status_string(i) for i in range(8)}) == 8


def _cfg(K, splits, **kw):
    arr = (C.c_int * max(len(splits), 1))(*splits)
    d = dict(beta=0.5, lr=0.1, momentum=0.9, weight_decay=5e-4, order=0, weight_reading=0, precision=0, serial=0,
             graphs=0)
    d.update(kw)
    cfg = B.fdg_config(K, C.cast(arr, C.POINTER(C.c_int)), d["beta"], d["lr"], d["momentum"], d["weight_decay"],
                       d["order"], d["weight_reading"], d["precision"], d["serial"], d["graphs"])
    cfg._keep = arr
    return cfg


def test_workspace_bytes_and_argument_checks(lib):
    n = C.c_size_t()
    arch = B.make_arch(n_per_stage=18, batch=128)
    cfg = _cfg(4, (13, 27, 41))
    assert lib.fdg_workspace_bytes(C.byref(arch), C.byref(cfg), C.byref(n)) == 0
    fp32_bytes = n.value
    assert 1 << 30 < fp32_bytes < 16 << 30                 # a few GiB of activation FIFO
    # deeper FIFO when the forward runs first
    cfg2 = _cfg(4, (13, 27, 41), order=1)
    assert lib.fdg_workspace_bytes(C.byref(arch), C.byref(cfg2), C.byref(n)) == 0 and n.value > fp32_bytes
    bad = [
        _cfg(4, (13, 27)),                 # reads a third split from the array: 0 -> not ascending
        _cfg(2, (54,)),                    # split after the last block
        _cfg(2, (0,)),
        _cfg(3, (20, 10)),
        _cfg(2, (10,), beta=0.0),
        _cfg(2, (10,), beta=1.5),
        _cfg(2, (10,), momentum=1.0),
        _cfg(2, (10,), order=7),
        _cfg(0, ()),
    ]
    for c in bad:
        assert lib.fdg_workspace_bytes(C.byref(arch), C.byref(c), C.byref(n)) == 1
    assert lib.fdg_workspace_bytes(None, C.byref(cfg), C.byref(n)) == 1
    assert lib.fdg_workspace_bytes(C.byref(arch), C.byref(cfg), None) == 1
    small = B.make_arch(n_per_stage=1, in_h=2, in_w=2)
    assert lib.fdg_workspace_bytes(C.byref(small), C.byref(_cfg(1, ())), C.byref(n)) == 1
    # null handles are rejected, not dereferenced
    assert lib.fdg_destroy(None) == 1
    assert lib.fdg_step(None, None, None, None, None) == 1
    assert lib.fdg_sync(None, None) == 1
    assert lib.fdg_set_lr(None, 0.1) == 1
    assert lib.fdg_last_error(None) == b"null context"
    ctx = C.c_void_p()
    assert lib.fdg_create(C.byref(arch), C.byref(cfg), None, 0, None, C.byref(ctx)) == 1 and not ctx.value
    # a workspace that is there but one byte short is refused before anything touches it (the pointer is never
    # dereferenced on this path, so any aligned address will do)
    assert lib.fdg_workspace_bytes(C.byref(arch), C.byref(cfg), C.byref(n)) == 0
    assert lib.fdg_create(C.byref(arch), C.byref(cfg), C.c_void_p(1 << 20), n.value - 1, None, C.byref(ctx)) == 2
    assert not ctx.value
    assert lib.fdg_create(C.byref(arch), C.byref(cfg), C.c_void_p((1 << 20) + 8), n.value, None, C.byref(ctx)) == 1   # misaligned
    assert lib.fdg_debug_raise_flag(None, 0) == 1
    assert lib.fdg_debug_guard_count(None, C.byref(n)) == 1 and lib.fdg_debug_check_guards(None, None) == 1
    # operator level: argument checks that answer without a GPU
    s = B.fdg_conv_shape(2, 8, 8, 512, 512, 3, 1, 1)
    assert lib.fdg_conv_wgrad_static(0, C.byref(s), C.c_void_p(256), C.c_void_p(256), C.c_void_p(256), None) == 2
    assert lib.fdg_conv_wgrad_static(0, C.byref(s), None, C.c_void_p(256), C.c_void_p(256), None) == 1
    assert lib.fdg_bn_scratch_bytes(64, C.byref(n)) == 0 and n.value >= 74 * 3 * 64 * 4
    assert lib.fdg_bn_scratch_bytes(0, C.byref(n)) == 1
    assert lib.fdg_bn_stats(0, C.c_void_p(256), 16, 64, 1e-5, C.c_void_p(256), C.c_void_p(256), 16, None) == 2
