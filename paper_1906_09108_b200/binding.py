"""ctypes binding of libfdg: the same entry points as include/fdg.h, argument
marshalling only.  Every step of the FDG path runs inside the CUDA library; there
is no fallback -- if the library is missing or fails to load, importing raises.

PyTorch appears here only as the owner of device memory and streams.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfdg.so")

FDG_OK = 0
STATUS_NAMES = {0: "FDG_OK", 1: "FDG_ERR_INVALID_ARG", 2: "FDG_ERR_WORKSPACE_TOO_SMALL", 3: "FDG_ERR_CUDA",
                4: "FDG_ERR_STATE", 5: "FDG_ERR_UNSUPPORTED", 6: "FDG_ERR_NONFINITE", 7: "FDG_ERR_TIMEOUT"}
FDG_RESNET_6N2, FDG_WRN = 0, 1
FDG_SHORTCUT_PROJECTION, FDG_SHORTCUT_ZERO_PAD = 0, 1
FDG_BACKWARD_FIRST, FDG_FORWARD_FIRST = 0, 1
FDG_STASHED, FDG_CURRENT = 0, 1
FDG_FP32_CUDACORE, FDG_BF16_TC = 0, 1
PARAM_KINDS = {0: "conv", 1: "bn_gamma", 2: "bn_beta", 3: "fc_w", 4: "fc_b"}

EXPORTS = ["fdg_workspace_bytes", "fdg_create", "fdg_destroy", "fdg_param_count", "fdg_param_layout",
           "fdg_set_params", "fdg_set_momentum", "fdg_get_params", "fdg_get_grads", "fdg_get_momentum",
           "fdg_set_lr", "fdg_step", "fdg_step_host", "fdg_sync", "fdg_profile_enable", "fdg_profile_read", "fdg_profile_read_modules", "fdg_get_module_output", "fdg_get_input_grad",
           "fdg_boundary_elems", "fdg_get_saved_tensor", "fdg_get_schedule_log", "fdg_launch_count", "fdg_status_string",
           "fdg_last_error", "fdg_conv_forward", "fdg_conv_dgrad", "fdg_conv_flip_weights",
           "fdg_conv_wgrad_scratch_bytes", "fdg_conv_wgrad", "fdg_conv_wgrad_static", "fdg_conv_path",
           "fdg_get_saved_tensor_of", "fdg_capture_bytes", "fdg_capture_begin", "fdg_capture_end", "fdg_get_captured",
           "fdg_bn_scratch_bytes", "fdg_bn_stats", "fdg_bn_apply", "fdg_bn_backward", "fdg_shrink", "fdg_sgd_update",
           "fdg_ingest", "fdg_head", "fdg_debug_raise_flag", "fdg_debug_wait_probe", "fdg_debug_guard_count", "fdg_debug_guard_offset",
           "fdg_debug_check_guards", "fdg_probe_mma_rate", "fdg_bn_stats_from_partials", "fdg_lr_at", "fdg_set_lr_schedule", "fdg_bn_running_count",
           "fdg_get_bn_running", "fdg_set_bn_running", "fdg_eval", "fdg_drain", "fdg_state_bytes", "fdg_save_state",
           "fdg_load_state"]


class fdg_arch(C.Structure):
    _fields_ = [("family", C.c_int), ("n_stages", C.c_int), ("blocks", C.c_int * 4), ("widths", C.c_int * 4),
                ("stem_width", C.c_int), ("shortcut", C.c_int), ("in_h", C.c_int), ("in_w", C.c_int), ("in_c", C.c_int),
                ("num_classes", C.c_int), ("batch", C.c_int), ("bn_eps", C.c_float)]


class fdg_config(C.Structure):
    _fields_ = [("K", C.c_int), ("split_after_block", C.POINTER(C.c_int)), ("beta", C.c_float), ("lr", C.c_float),
                ("momentum", C.c_float), ("weight_decay", C.c_float), ("order", C.c_int),
                ("weight_reading", C.c_int), ("precision", C.c_int), ("serial", C.c_int), ("graphs", C.c_int)]


class fdg_param_entry(C.Structure):
    _fields_ = [("kind", C.c_int), ("unit", C.c_int), ("dims", C.c_int * 4), ("offset", C.c_size_t),
                ("count", C.c_size_t)]


class fdg_sched_entry(C.Structure):
    _fields_ = [("t", C.c_int64), ("k", C.c_int32), ("tau_f", C.c_int64), ("tau_b", C.c_int64),
                ("ver_f", C.c_int64), ("ver_b", C.c_int64), ("slot_f", C.c_int32), ("slot_b", C.c_int32)]


class fdg_conv_shape(C.Structure):
    _fields_ = [("N", C.c_int), ("H", C.c_int), ("W", C.c_int), ("Ci", C.c_int), ("Co", C.c_int), ("R", C.c_int),
                ("stride", C.c_int), ("pad", C.c_int)]


class fdg_lr_schedule(C.Structure):
    _fields_ = [("iters_per_epoch", C.c_int64), ("base_lr", C.c_float), ("n_milestones", C.c_int),
                ("milestones", C.c_int * 8), ("gamma", C.c_float), ("warmup_epochs", C.c_int), ("warmup_lr", C.c_float)]


def make_schedule(iters_per_epoch, base_lr=0.1, milestones=(150, 225, 275), gamma=0.1, warmup_epochs=0, warmup_lr=0.01):
    ms = list(milestones) + [0] * (8 - len(milestones))
    return fdg_lr_schedule(iters_per_epoch, base_lr, len(milestones), (C.c_int * 8)(*ms), gamma, warmup_epochs, warmup_lr)


class fdg_conv_extra(C.Structure):
    _fields_ = [("share", C.c_int), ("wgrad_cta_cap", C.c_int), ("dy_spread", C.c_void_p), ("reduce", C.c_int),
                ("next_mask", C.c_void_p), ("next_x", C.c_void_p), ("next_stats", C.c_void_p), ("partial", C.c_void_p),
                ("partial_floats", C.c_size_t), ("nparts", C.c_int)]


FDG_CONV_PARTIAL_ROWS = 256


class fdg_kernel_stat(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_uint64), ("total_ms", C.c_double), ("bytes", C.c_double),
                ("flops", C.c_double)]


def _ptr(t):
    return None if t is None else t.data_ptr()


def load_library(path=LIB_PATH):
    if not os.path.exists(path):
        raise ImportError("libfdg.so is not built (%s); run `python -m paper_1906_09108_b200.build`" % path)
    lib = C.CDLL(path)
    vp, sz, i64 = C.c_void_p, C.c_size_t, C.c_int64
    P = C.POINTER
    sig = {
        "fdg_workspace_bytes": [P(fdg_arch), P(fdg_config), P(sz)],
        "fdg_create": [P(fdg_arch), P(fdg_config), vp, sz, P(vp), P(vp)],
        "fdg_destroy": [vp],
        "fdg_param_count": [vp, C.c_int, P(sz)],
        "fdg_param_layout": [vp, C.c_int, P(fdg_param_entry), sz, P(sz)],
        "fdg_set_params": [vp, C.c_int, vp, sz],
        "fdg_set_momentum": [vp, C.c_int, vp, sz],
        "fdg_get_params": [vp, C.c_int, vp, sz],
        "fdg_get_grads": [vp, C.c_int, vp, sz],
        "fdg_get_momentum": [vp, C.c_int, vp, sz],
        "fdg_set_lr": [vp, C.c_float],
        "fdg_step": [vp, vp, vp, vp, vp],
        "fdg_step_host": [vp, vp, vp, vp, vp],
        "fdg_sync": [vp, vp],
        "fdg_profile_enable": [vp, C.c_int],
        "fdg_profile_read": [vp, P(fdg_kernel_stat), sz, P(sz)],
        "fdg_profile_read_modules": [vp, P(C.c_double), sz, P(sz)],
        "fdg_get_module_output": [vp, C.c_int, vp, sz, P(i64)],
        "fdg_get_input_grad": [vp, C.c_int, vp, sz, P(i64)],
        "fdg_boundary_elems": [vp, C.c_int, P(sz), P(sz)],
        "fdg_get_saved_tensor": [vp, C.c_int, C.c_int, C.c_int, vp, sz, P(sz), P(i64)],
        "fdg_get_schedule_log": [vp, P(fdg_sched_entry), sz, P(sz)],
        "fdg_launch_count": [vp, P(C.c_uint64)],
        "fdg_conv_forward": [C.c_int, P(fdg_conv_shape), vp, vp, vp, vp, P(fdg_conv_extra), vp, vp],
        "fdg_conv_dgrad": [C.c_int, P(fdg_conv_shape), vp, vp, vp, vp, vp, vp, P(fdg_conv_extra), vp, vp],
        "fdg_conv_flip_weights": [P(fdg_conv_shape), vp, vp, vp],
        "fdg_probe_mma_rate": [C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp],
        "fdg_bn_stats_from_partials": [vp, C.c_int, C.c_size_t, C.c_int, C.c_float, vp, vp],
        "fdg_conv_wgrad_scratch_bytes": [C.c_int, P(fdg_conv_shape), P(sz)],
        "fdg_conv_wgrad": [C.c_int, P(fdg_conv_shape), vp, vp, vp, vp, sz, P(fdg_conv_extra), vp, vp],
        "fdg_get_saved_tensor_of": [vp, C.c_int, C.c_int, C.c_int, i64, vp, sz, P(sz), P(i64)],
        "fdg_debug_raise_flag": [vp, C.c_int],
        "fdg_debug_wait_probe": [vp, vp, C.c_uint],
        "fdg_debug_guard_count": [vp, C.POINTER(C.c_size_t)],
        "fdg_debug_guard_offset": [vp, C.c_size_t, C.POINTER(C.c_size_t)],
        "fdg_debug_check_guards": [vp, C.POINTER(C.c_longlong)],
        "fdg_lr_at": [P(fdg_lr_schedule), i64, P(C.c_float)],
        "fdg_set_lr_schedule": [vp, P(fdg_lr_schedule)],
        "fdg_bn_running_count": [vp, C.c_int, P(sz)],
        "fdg_get_bn_running": [vp, C.c_int, vp, sz],
        "fdg_set_bn_running": [vp, C.c_int, vp, sz],
        "fdg_eval": [vp, vp, vp, vp, vp, vp],
        "fdg_drain": [vp, vp, vp],
        "fdg_state_bytes": [vp, P(sz)],
        "fdg_save_state": [vp, vp, sz],
        "fdg_load_state": [vp, vp, sz],
        "fdg_capture_bytes": [vp, C.c_int, P(sz)],
        "fdg_capture_begin": [vp, C.c_int, vp, sz],
        "fdg_capture_end": [vp, C.c_int],
        "fdg_get_captured": [vp, C.c_int, C.c_int, C.c_int, vp, sz, P(sz), P(i64)],
        "fdg_bn_scratch_bytes": [C.c_int, P(sz)],
        "fdg_bn_stats": [C.c_int, vp, sz, C.c_int, C.c_float, vp, vp, sz, vp],
        "fdg_bn_apply": [C.c_int, vp, vp, vp, vp, vp, vp, vp, vp, C.c_int, vp, sz, C.c_int, C.c_float, vp, C.c_int,
                         C.c_int, vp],
        "fdg_bn_backward": [C.c_int, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, C.c_int, vp,
                            C.c_int, C.c_int, vp, sz, vp],
        "fdg_shrink": [C.c_int, vp, vp, C.c_float, sz, vp],
        "fdg_sgd_update": [vp, vp, vp, vp, vp, sz, C.c_float, C.c_float, C.c_float, vp],
        "fdg_ingest": [C.c_int, vp, vp, sz, C.c_int, C.c_int, vp, vp, C.c_int, vp],
        "fdg_head": [C.c_int, vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp, vp, vp, vp, vp, vp],
        "fdg_conv_wgrad_static": [C.c_int, P(fdg_conv_shape), vp, vp, vp, vp],
        "fdg_conv_path": [C.c_int, P(fdg_conv_shape), C.c_int, P(C.c_int)],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.fdg_status_string.argtypes = [C.c_int]
    lib.fdg_status_string.restype = C.c_char_p
    lib.fdg_last_error.argtypes = [vp]
    lib.fdg_last_error.restype = C.c_char_p
    return lib


class FDGError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, status), message))
        self.status = status


def make_arch(family="resnet6n2", n_per_stage=1, widths=(16, 32, 64), stem_width=16, in_h=32, in_w=32, in_c=3,
              num_classes=10, batch=128, bn_eps=1e-5, blocks=None, shortcut="projection"):
    """`blocks`: residual blocks per stage; None: n_per_stage in each of len(widths) stages."""
    fam = {"resnet6n2": FDG_RESNET_6N2, "wrn": FDG_WRN}[family]
    sc = {"projection": FDG_SHORTCUT_PROJECTION, "zero_pad": FDG_SHORTCUT_ZERO_PAD}[shortcut]
    ns = len(widths)
    bl = list(blocks) if blocks is not None else [n_per_stage] * ns
    assert len(bl) == ns and 1 <= ns <= 4
    pad = [0] * (4 - ns)
    return fdg_arch(fam, ns, (C.c_int * 4)(*(bl + pad)), (C.c_int * 4)(*(list(widths) + pad)), stem_width, sc, in_h, in_w,
                    in_c, num_classes, batch, bn_eps)


class FDG:
    """Owner of one fdg_ctx and of the torch tensor that backs its workspace.  Each
    method is one C-ABI call (plus host<->device staging of its arguments)."""

    def __init__(self, arch, K=2, split_after_block=(1,), beta=1.0, lr=0.1, momentum=0.9, weight_decay=5e-4,
                 order=FDG_BACKWARD_FIRST, weight_reading=FDG_STASHED, precision=FDG_FP32_CUDACORE, serial=False,
                 graphs=False, device="cuda:0"):
        import torch
        self.torch = torch
        self.lib = load_library()
        self.arch = arch
        self.K = K
        self._splits = (C.c_int * max(len(split_after_block), 1))(*split_after_block)
        self.cfg = fdg_config(K, C.cast(self._splits, C.POINTER(C.c_int)), beta, lr, momentum, weight_decay, order,
                              weight_reading, precision, int(serial), int(graphs))
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        n = C.c_size_t()
        self._check(self.lib.fdg_workspace_bytes(C.byref(self.arch), C.byref(self.cfg), C.byref(n)), None)
        self.workspace_bytes = n.value
        self.workspace = torch.empty(n.value + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.workspace_skip = base - self.workspace.data_ptr()     # bytes of `workspace` before the library's base
        ctx = C.c_void_p()
        self._check(self.lib.fdg_create(C.byref(self.arch), C.byref(self.cfg), base, n.value, None, C.byref(ctx)), None)
        self.ctx = ctx

    def _check(self, status, ctx):
        if status != FDG_OK:
            msg = self.lib.fdg_last_error(ctx).decode() if ctx else self.lib.fdg_status_string(status).decode()
            raise FDGError(status, msg)

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.fdg_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- parameters -----------------------------------------------------------
    def param_count(self, k):
        n = C.c_size_t()
        self._check(self.lib.fdg_param_count(self.ctx, k, C.byref(n)), self.ctx)
        return n.value

    def param_layout(self, k):
        """[(name, kind, shape)] in flat order, the same table the oracle builds."""
        n = C.c_size_t()
        self._check(self.lib.fdg_param_layout(self.ctx, k, None, 0, C.byref(n)), self.ctx)
        arr = (fdg_param_entry * n.value)()
        self._check(self.lib.fdg_param_layout(self.ctx, k, arr, n.value, C.byref(n)), self.ctx)
        out = []
        for e in arr:
            kind = PARAM_KINDS[e.kind]
            dims = tuple(e.dims)
            shape = dims if kind == "conv" else (dims[:2] if kind == "fc_w" else dims[:1])
            unit = "stem" if e.unit == 0 else ("head" if e.unit < 0 else "block%d" % e.unit)
            out.append(("%s@%d" % (unit, e.offset), kind, shape))
        return out

    def _host_vec(self, fn, k):
        out = np.empty(self.param_count(k), dtype=np.float32)
        self._check(fn(self.ctx, k, out.ctypes.data, out.size), self.ctx)
        return out

    def set_params(self, k, flat):
        flat = np.ascontiguousarray(flat, dtype=np.float32)
        self._check(self.lib.fdg_set_params(self.ctx, k, flat.ctypes.data, flat.size), self.ctx)

    def set_momentum(self, k, flat):
        flat = np.ascontiguousarray(flat, dtype=np.float32)
        self._check(self.lib.fdg_set_momentum(self.ctx, k, flat.ctypes.data, flat.size), self.ctx)

    def get_params(self, k):
        return self._host_vec(self.lib.fdg_get_params, k)

    def get_grads(self, k):
        return self._host_vec(self.lib.fdg_get_grads, k)

    def get_momentum(self, k):
        return self._host_vec(self.lib.fdg_get_momentum, k)

    def set_lr(self, lr):
        self._check(self.lib.fdg_set_lr(self.ctx, lr), self.ctx)

    def set_lr_schedule(self, schedule):
        """schedule: fdg_lr_schedule (see make_schedule) or None to switch it off."""
        self._schedule = schedule
        self._check(self.lib.fdg_set_lr_schedule(self.ctx, C.byref(schedule) if schedule is not None else None), self.ctx)

    def get_running(self, k):
        n = C.c_size_t()
        self._check(self.lib.fdg_bn_running_count(self.ctx, k, C.byref(n)), self.ctx)
        out = np.empty(n.value, dtype=np.float32)
        if n.value:
            self._check(self.lib.fdg_get_bn_running(self.ctx, k, out.ctypes.data, out.size), self.ctx)
        return out

    def set_running(self, k, flat):
        flat = np.ascontiguousarray(flat, dtype=np.float32)
        if flat.size:
            self._check(self.lib.fdg_set_bn_running(self.ctx, k, flat.ctypes.data, flat.size), self.ctx)

    def eval(self, images_dev, labels_dev=None, logits_dev=None, correct_dev=None, stream=None):
        """Inference forward of one batch; correct_dev (int32 CUDA tensor of one element) is incremented."""
        st = self.torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._check(self.lib.fdg_eval(self.ctx, st, images_dev.data_ptr(), _ptr(labels_dev), _ptr(logits_dev),
                                      _ptr(correct_dev)), self.ctx)

    def drain(self, losses_dev=None, stream=None):
        st = self.torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._check(self.lib.fdg_drain(self.ctx, st, _ptr(losses_dev)), self.ctx)

    def save_state(self):
        """The run's state as a pinned-size CPU uint8 tensor (fdg_save_state to host memory)."""
        n = C.c_size_t()
        self._check(self.lib.fdg_state_bytes(self.ctx, C.byref(n)), self.ctx)
        blob = self.torch.empty(n.value, dtype=self.torch.uint8)
        self._check(self.lib.fdg_save_state(self.ctx, blob.data_ptr(), n.value), self.ctx)
        return blob

    def load_state(self, blob):
        self._check(self.lib.fdg_load_state(self.ctx, blob.data_ptr(), blob.numel()), self.ctx)

    # ---- stepping -------------------------------------------------------------
    def step(self, images_dev, labels_dev, loss_dev=None, stream=None):
        """images_dev: float32 CUDA tensor [B,H,W,C]; labels_dev: int32 CUDA tensor [B]."""
        st = self.torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._check(self.lib.fdg_step(self.ctx, st, images_dev.data_ptr(), labels_dev.data_ptr(),
                                      loss_dev.data_ptr() if loss_dev is not None else None), self.ctx)

    def step_host(self, images_host, labels_host, loss_host=None, stream=None):
        """images_host / labels_host / loss_host: CPU tensors (pinned for asynchronous copies)."""
        st = self.torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._check(self.lib.fdg_step_host(self.ctx, st, images_host.data_ptr(), labels_host.data_ptr(),
                                           loss_host.data_ptr() if loss_host is not None else None), self.ctx)

    def guard_offsets(self):
        """Byte offsets (from the workspace base given to fdg_create) of the guard regions behind the buffers."""
        n, off, out = C.c_size_t(), C.c_size_t(), []
        self._check(self.lib.fdg_debug_guard_count(self.ctx, C.byref(n)), self.ctx)
        for i in range(n.value):
            self._check(self.lib.fdg_debug_guard_offset(self.ctx, i, C.byref(off)), self.ctx)
            out.append(off.value)
        return out

    def check_guards(self):
        """-1, or the index of the first guard region that was overwritten."""
        bad = C.c_longlong()
        self._check(self.lib.fdg_debug_check_guards(self.ctx, C.byref(bad)), self.ctx)
        return bad.value

    def profile_enable(self, on=True):
        self._check(self.lib.fdg_profile_enable(self.ctx, int(on)), self.ctx)

    def profile_read(self):
        n = C.c_size_t()
        arr = (fdg_kernel_stat * 32)()
        self._check(self.lib.fdg_profile_read(self.ctx, arr, 32, C.byref(n)), self.ctx)
        return [dict(name=e.name.decode(), launches=e.launches, total_ms=e.total_ms, bytes=e.bytes, flops=e.flops)
                for e in arr[:n.value]]

    def profile_read_modules(self):
        """Busy milliseconds of each module's passes since the last read (profiler on)."""
        arr = (C.c_double * self.K)()
        n = C.c_size_t()
        self._check(self.lib.fdg_profile_read_modules(self.ctx, arr, self.K, C.byref(n)), self.ctx)
        return list(arr)

    def sync(self, stream=None):
        st = self.torch.cuda.current_stream().cuda_stream if stream is None else stream
        self._check(self.lib.fdg_sync(self.ctx, st), self.ctx)

    # ---- inspection -----------------------------------------------------------
    def boundary_elems(self, k):
        a, b = C.c_size_t(), C.c_size_t()
        self._check(self.lib.fdg_boundary_elems(self.ctx, k, C.byref(a), C.byref(b)), self.ctx)
        return a.value, b.value

    def module_output(self, k):
        n = self.boundary_elems(k)[0]
        out = np.empty(n, dtype=np.float32)
        b = C.c_int64()
        self._check(self.lib.fdg_get_module_output(self.ctx, k, out.ctypes.data, n, C.byref(b)), self.ctx)
        return b.value, out

    def input_grad(self, k):
        n = self.boundary_elems(k)[1]
        out = np.empty(n, dtype=np.float32)
        b = C.c_int64()
        self._check(self.lib.fdg_get_input_grad(self.ctx, k, out.ctypes.data, n, C.byref(b)), self.ctx)
        return b.value, out

    def saved_tensor(self, k, unit, which):
        """(batch, flat fp32 array) of one tensor in module k's newest activation-FIFO slot."""
        n, b = C.c_size_t(), C.c_int64()
        self._check(self.lib.fdg_get_saved_tensor(self.ctx, k, unit, which, None, 0, C.byref(n), None), self.ctx)
        out = np.empty(n.value, dtype=np.float32)
        self._check(self.lib.fdg_get_saved_tensor(self.ctx, k, unit, which, out.ctypes.data, n.value, None,
                                                  C.byref(b)), self.ctx)
        return b.value, out

    def saved_tensor_of(self, k, unit, which, batch):
        """The same for the slot that holds `batch` (one still in flight in module k)."""
        n, b = C.c_size_t(), C.c_int64()
        self._check(self.lib.fdg_get_saved_tensor_of(self.ctx, k, unit, which, batch, None, 0, C.byref(n), None), self.ctx)
        out = np.empty(n.value, dtype=np.float32)
        self._check(self.lib.fdg_get_saved_tensor_of(self.ctx, k, unit, which, batch, out.ctypes.data, n.value, None,
                                                     C.byref(b)), self.ctx)
        return b.value, out

    def capture_begin(self, k):
        """Keeps a copy of every gradient tensor of module k's backward passes (torch owns the buffer)."""
        n = C.c_size_t()
        self._check(self.lib.fdg_capture_bytes(self.ctx, k, C.byref(n)), self.ctx)
        buf = self.torch.empty(n.value + 256, dtype=self.torch.uint8, device=self.device)
        base = (buf.data_ptr() + 255) // 256 * 256
        self._check(self.lib.fdg_capture_begin(self.ctx, k, base, n.value), self.ctx)
        self._capture = getattr(self, "_capture", {})
        self._capture[k] = buf

    def capture_end(self, k):
        self._check(self.lib.fdg_capture_end(self.ctx, k), self.ctx)
        self._capture.pop(k, None)

    def captured(self, k, unit, which):
        """(batch, flat fp32 array) of one gradient tensor of module k's most recent captured backward."""
        n, b = C.c_size_t(), C.c_int64()
        self._check(self.lib.fdg_get_captured(self.ctx, k, unit, which, None, 0, C.byref(n), None), self.ctx)
        out = np.empty(n.value, dtype=np.float32)
        self._check(self.lib.fdg_get_captured(self.ctx, k, unit, which, out.ctypes.data, n.value, None, C.byref(b)),
                    self.ctx)
        return b.value, out

    def schedule_log(self):
        n = C.c_size_t()
        self._check(self.lib.fdg_get_schedule_log(self.ctx, None, 0, C.byref(n)), self.ctx)
        arr = (fdg_sched_entry * max(n.value, 1))()
        self._check(self.lib.fdg_get_schedule_log(self.ctx, arr, n.value, C.byref(n)), self.ctx)
        return [dict(t=e.t, k=e.k, tau_f=e.tau_f, tau_b=e.tau_b, ver_f=e.ver_f, ver_b=e.ver_b, slot_f=e.slot_f,
                     slot_b=e.slot_b) for e in arr[:n.value]]

    def launch_count(self):
        n = C.c_uint64()
        self._check(self.lib.fdg_launch_count(self.ctx, C.byref(n)), self.ctx)
        return n.value


# ---- operator level (include/fdg_ops.h): thin wrappers over torch CUDA tensors -----------

class ConvOps:
    """fdg_conv_* on torch CUDA tensors of the precision's storage type (float32 / bfloat16)."""

    def __init__(self, precision):
        import torch
        self.torch = torch
        self.lib = load_library()
        self.precision = precision
        self.dtype = torch.bfloat16 if precision == FDG_BF16_TC else torch.float32
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def _stream(self):
        return self.torch.cuda.current_stream().cuda_stream

    def _chk(self, rc):
        if rc != FDG_OK:
            raise FDGError(rc, self.lib.fdg_status_string(rc).decode())

    def out_hw(self, s):
        return (s.H + 2 * s.pad - s.R) // s.stride + 1, (s.W + 2 * s.pad - s.R) // s.stride + 1

    def path(self, s, op):
        v = C.c_int()
        self._chk(self.lib.fdg_conv_path(self.precision, C.byref(s), op, C.byref(v)))
        return bool(v.value)

    def _extra(self, s, share=0, wgrad_cta_cap=0, spread=False, reduce=0, next_mask=None, next_x=None, next_stats=None,
               C_red=0):
        """fdg_conv_extra plus the torch tensors it points to (kept alive by the caller)."""
        ex = fdg_conv_extra()
        ex.share, ex.wgrad_cta_cap, ex.reduce = share, wgrad_cta_cap, reduce
        keep = []
        if spread:
            up = self.torch.empty((s.N, s.H, s.W, s.Co), dtype=self.dtype, device="cuda")
            ex.dy_spread = up.data_ptr()
            keep.append(up)
        if reduce:
            part = self.torch.full((FDG_CONV_PARTIAL_ROWS, 2 * C_red), float("nan"), dtype=self.torch.float32, device="cuda")
            ex.partial, ex.partial_floats = part.data_ptr(), part.numel()
            ex.next_mask, ex.next_x, ex.next_stats = _ptr(next_mask), _ptr(next_x), _ptr(next_stats)
            keep.append(part)
        return ex, keep

    def forward(self, s, x, w, res=None, share=0, reduce=False):
        """y, or (y, partial rows [nparts, 2*Co]) with reduce=True."""
        p, q = self.out_hw(s)
        y = self.torch.empty((s.N, p, q, s.Co), dtype=self.dtype, device="cuda")
        ex, keep = self._extra(s, share=share, reduce=1 if reduce else 0, C_red=s.Co)
        self._chk(self.lib.fdg_conv_forward(self.precision, C.byref(s), _ptr(x), _ptr(w), _ptr(y), _ptr(res),
                                            C.byref(ex), _ptr(self.status), self._stream()))
        return (y, keep[-1][:ex.nparts]) if reduce else y

    def flip_weights(self, s, w):
        out = self.torch.empty(s.Ci * s.R * s.R * s.Co, dtype=self.torch.bfloat16, device="cuda")
        self._chk(self.lib.fdg_conv_flip_weights(C.byref(s), _ptr(w), _ptr(out), self._stream()))
        return out

    def dgrad(self, s, dy, w, w_flipped=None, res=None, res_mask=None, share=0, spread=False, next_bn=None):
        """dx, or (dx, partial rows [nparts, 2*Ci]) with next_bn = (mask, x, stats) of the batch norm dx feeds."""
        dx = self.torch.empty((s.N, s.H, s.W, s.Ci), dtype=self.dtype, device="cuda")
        nm, nx, ns = next_bn if next_bn else (None, None, None)
        ex, keep = self._extra(s, share=share, spread=spread, reduce=2 if next_bn else 0, next_mask=nm, next_x=nx,
                               next_stats=ns, C_red=s.Ci)
        self._chk(self.lib.fdg_conv_dgrad(self.precision, C.byref(s), _ptr(dy), _ptr(w), _ptr(w_flipped), _ptr(dx),
                                          _ptr(res), _ptr(res_mask), C.byref(ex), _ptr(self.status), self._stream()))
        return (dx, keep[-1][:ex.nparts]) if next_bn else dx

    def wgrad(self, s, x, dy, cta_cap=0, spread=False):
        n = C.c_size_t()
        self._chk(self.lib.fdg_conv_wgrad_scratch_bytes(self.precision, C.byref(s), C.byref(n)))
        scratch = self.torch.empty(max(n.value, 16), dtype=self.torch.uint8, device="cuda")
        dw = self.torch.empty((s.Co, s.R, s.R, s.Ci), dtype=self.torch.float32, device="cuda")
        ex, keep = self._extra(s, wgrad_cta_cap=cta_cap, spread=spread)
        self._chk(self.lib.fdg_conv_wgrad(self.precision, C.byref(s), _ptr(x), _ptr(dy), _ptr(dw), _ptr(scratch),
                                          n.value, C.byref(ex), _ptr(self.status), self._stream()))
        return dw

    def wgrad_static(self, s, x, dy):
        """fdg_conv_wgrad_static: the weight gradient with the library's built-in scratch buffer
        (only the result tensor is allocated here, by torch, before the call)."""
        dw = self.torch.empty((s.Co, s.R, s.R, s.Ci), dtype=self.torch.float32, device="cuda")
        self._chk(self.lib.fdg_conv_wgrad_static(self.precision, C.byref(s), _ptr(x), _ptr(dy), _ptr(dw),
                                                 self._stream()))
        return dw

    def timed_out(self):
        return bool(self.status.item())


class EwOps:
    """The memory-bound operator-level calls (fdg_bn_*, fdg_shrink, fdg_sgd_update, fdg_ingest, fdg_head) on
    torch CUDA tensors; activations [rows, C] (any leading shape) in the precision's storage type."""

    def __init__(self, precision):
        import torch
        self.torch = torch
        self.lib = load_library()
        self.precision = precision
        self.dtype = torch.bfloat16 if precision == FDG_BF16_TC else torch.float32

    def _stream(self):
        return self.torch.cuda.current_stream().cuda_stream

    def _chk(self, rc):
        if rc != FDG_OK:
            raise FDGError(rc, self.lib.fdg_status_string(rc).decode())

    def _scratch(self, ch):
        n = C.c_size_t()
        self._chk(self.lib.fdg_bn_scratch_bytes(ch, C.byref(n)))
        return self.torch.empty(n.value, dtype=self.torch.uint8, device="cuda"), n.value

    def _f32(self, *shape):
        return self.torch.empty(shape, dtype=self.torch.float32, device="cuda")

    def bn_stats(self, x, eps=1e-5):
        ch = x.shape[-1]
        rows = x.numel() // ch
        stats = self._f32(2 * ch)
        sc, nb = self._scratch(ch)
        self._chk(self.lib.fdg_bn_stats(self.precision, _ptr(x), rows, ch, eps, _ptr(stats), _ptr(sc), nb, self._stream()))
        return stats

    def bn_apply(self, x, stats, gamma, beta, res=None, res_bn=None, relu=True, eps=1e-5, partial=None, block_cap=0):
        """res_bn = (stats, gamma, beta) of the residual's own batch norm.  With `partial` (rows from a fused
        convolution) `stats` is an output."""
        ch = x.shape[-1]
        rows = x.numel() // ch
        y = self.torch.empty_like(x)
        rs, rg, rb = res_bn if res_bn else (None, None, None)
        self._chk(self.lib.fdg_bn_apply(self.precision, _ptr(x), _ptr(stats), _ptr(gamma), _ptr(beta), _ptr(res), _ptr(rs),
                                        _ptr(rg), _ptr(rb), int(relu), _ptr(y), rows, ch, eps, _ptr(partial),
                                        0 if partial is None else partial.shape[0], block_cap, self._stream()))
        return y

    def bn_backward(self, dy, mask, x, stats, gamma, second=None, res=None, partial=None, block_cap=0, sums_only=False):
        """Returns (dx, dgamma, dbeta) or, with second = (x2, stats2, gamma2), (dx, dgamma, dbeta, dx2, dgamma2, dbeta2);
        sums_only: dx is None and only the parameter gradients are formed."""
        ch = x.shape[-1]
        rows = x.numel() // ch
        dx = None if sums_only else self.torch.empty_like(x)
        dg, db = self._f32(ch), self._f32(ch)
        x2, s2, g2 = second if second else (None, None, None)
        dx2 = self.torch.empty_like(x) if (second and not sums_only) else None
        dg2, db2 = (self._f32(ch), self._f32(ch)) if second else (None, None)
        sc, nb = self._scratch(ch)
        self._chk(self.lib.fdg_bn_backward(self.precision, _ptr(dy), _ptr(mask), _ptr(x), _ptr(stats), _ptr(gamma), _ptr(x2),
                                           _ptr(s2), _ptr(g2), _ptr(res), _ptr(dx), _ptr(dx2), _ptr(dg), _ptr(db), _ptr(dg2),
                                           _ptr(db2), rows, ch, _ptr(partial), 0 if partial is None else partial.shape[0],
                                           block_cap, _ptr(sc), nb, self._stream()))
        return (dx, dg, db, dx2, dg2, db2) if second else (dx, dg, db)

    def shrink(self, x, beta):
        out = self.torch.empty_like(x)
        self._chk(self.lib.fdg_shrink(self.precision, _ptr(x), _ptr(out), beta, x.numel(), self._stream()))
        return out

    def sgd_update(self, theta, mom, grad, lr, momentum, weight_decay, bf16_copy=True):
        """In place on theta and mom; returns (next fp32 copy, next bf16 copy or None)."""
        n32 = self.torch.empty_like(theta)
        n16 = self.torch.empty(theta.numel(), dtype=self.torch.bfloat16, device="cuda") if bf16_copy else None
        self._chk(self.lib.fdg_sgd_update(_ptr(theta), _ptr(mom), _ptr(grad), _ptr(n32), _ptr(n16), theta.numel(), lr,
                                          momentum, weight_decay, self._stream()))
        return n32, n16

    def ingest(self, images, c_out, labels):
        rows = images.numel() // images.shape[-1]
        out = self.torch.empty(tuple(images.shape[:-1]) + (c_out,), dtype=self.dtype, device="cuda")
        lab = self.torch.empty_like(labels)
        self._chk(self.lib.fdg_ingest(self.precision, _ptr(images), _ptr(out), rows, images.shape[-1], c_out, _ptr(labels),
                                      _ptr(lab), labels.numel(), self._stream()))
        return out, lab

    def head(self, x, w, b, labels):
        """x [B, HW.., F].  Returns dict(pooled, dlogits, loss_n, dx, dw, db, loss, flags)."""
        bsz, feat = x.shape[0], x.shape[-1]
        hw = x.numel() // (bsz * feat)
        classes = w.shape[0]
        o = dict(pooled=self._f32(bsz, feat), dlogits=self._f32(bsz, classes), loss_n=self._f32(bsz),
                 dx=self.torch.empty_like(x), dw=self._f32(classes, feat), db=self._f32(classes), loss=self._f32(1),
                 flags=self.torch.zeros(4, dtype=self.torch.int32, device="cuda"))
        self._chk(self.lib.fdg_head(self.precision, _ptr(x), _ptr(w), _ptr(b), _ptr(labels), bsz, hw, feat, classes,
                                    _ptr(o["pooled"]), _ptr(o["dlogits"]), _ptr(o["loss_n"]), _ptr(o["dx"]), _ptr(o["dw"]),
                                    _ptr(o["db"]), _ptr(o["loss"]), _ptr(o["flags"]), self._stream()))
        return o
