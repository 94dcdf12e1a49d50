"""Seeded synthetic inputs for FDG training, shared by the CPU oracle's tests
and by the CUDA path's tests and benchmark.

This module holds none of the method's arithmetic: it only draws numbers.  The
paper trains on CIFAR-10/100 images after per-channel normalisation (zero mean,
unit variance, 32x32x3) with integer class labels; the stand-ins are i.i.d.
N(0,1) pixels and labels uniform over the classes.  Every draw is keyed by
(seed, purpose, index) through numpy's counter-based Philox generator, so any
batch or parameter vector can be regenerated independently of call order.
"""
import numpy as np

_IMAGES, _LABELS, _PARAMS = 1, 2, 3


def _rng(seed, purpose, index):
    return np.random.Generator(np.random.Philox(key=[(int(seed) << 8) | purpose, int(index)]))


def images(seed, t, batch, h, w, c):
    """Batch t (1-based) of images, float32 [batch, h, w, c], i.i.d. N(0,1)."""
    return _rng(seed, _IMAGES, t).standard_normal((batch, h, w, c), dtype=np.float32)


def labels(seed, t, batch, num_classes):
    """Batch t of labels, int32 [batch], uniform over the classes."""
    return _rng(seed, _LABELS, t).integers(0, num_classes, size=batch, dtype=np.int32)


def init_params(seed, module, spec, jitter=False):
    """Initial flat float32 parameter vector of one module.

    `spec` is the module's parameter table [(name, kind, shape)] in flat order.
    conv: normal, std sqrt(2/fan_in), fan_in = R*S*C_in.  fc_w / fc_b: uniform
    in +-1/sqrt(features).  bn_gamma = 1 and bn_beta = 0, or, with jitter=True,
    gamma ~ U(0.5, 1.5) and beta ~ N(0, 0.1) so that tests exercise both.
    """
    rng = _rng(seed, _PARAMS, module)
    parts = []
    fc_bound = 1.0
    for _, kind, shape in spec:
        n = int(np.prod(shape))
        if kind == "conv":
            fan_in = shape[1] * shape[2] * shape[3]
            a = rng.standard_normal(n, dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
        elif kind == "bn_gamma":
            a = (rng.uniform(0.5, 1.5, n) if jitter else np.ones(n)).astype(np.float32)
        elif kind == "bn_beta":
            a = (rng.standard_normal(n) * 0.1 if jitter else np.zeros(n)).astype(np.float32)
        elif kind == "fc_w":
            fc_bound = 1.0 / np.sqrt(shape[1])
            a = rng.uniform(-fc_bound, fc_bound, n).astype(np.float32)
        elif kind == "fc_b":
            a = rng.uniform(-fc_bound, fc_bound, n).astype(np.float32)
        else:
            raise ValueError(kind)
        parts.append(a)
    return np.concatenate(parts) if parts else np.zeros(0, np.float32)
