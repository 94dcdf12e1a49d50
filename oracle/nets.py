"""CPU oracle, part 2: the residual networks the paper trains, cut into units.

TEST INFRASTRUCTURE ONLY (see oracle/layers.py).

The paper splits the layer indices {1..L} into K contiguous groups q(k)
(Section 3.1, first paragraph).  Here the network is an ordered list of units
-- stem, residual blocks 1..3n, head -- and a split point is a block index, so
module 1 owns the stem and module K owns the head.  Each unit offers a forward
that returns what its backward will need (the "saved computation graph" of
Fig. 1(b)) and a backward that is the chain rule of Eq. 8 / Eq. 9 through its
layers.

The paper defines no architecture; these are the standard definitions of the
networks it cites (Tables 3-6):
  * "resnet6n2": post-activation basic blocks, stages of n blocks (three stages of n for the
       6n+2 networks; four stages of two at widths 64..512 for the CIFAR ResNet-18),
       block(x) = ReLU( BN(conv3x3(ReLU(BN(conv3x3_s(x))))) + sc(x) ),
       sc = identity, or, when the shape changes, BN(conv1x1_s(x)) ("projection") or the
       parameter-free x taken at every second pixel with zero channels added on both sides
       ("zero_pad", the other standard choice for the 6n+2 networks; the printed parameter
       counts cannot tell the two apart);
       stem = ReLU(BN(conv3x3(image))); head = GAP -> FC -> softmax-CE.
  * "wrn": pre-activation basic blocks,
       o = ReLU(BN(x)); block(x) = conv3x3(ReLU(BN(conv3x3_s(o)))) + sc,
       sc = x, or conv1x1_s(o) when the shape changes;
       stem = conv3x3(image); head = ReLU(BN(.)) -> GAP -> FC -> softmax-CE.

Storage precision.  Every unit carries two maps, `q` (applied to each activation or
gradient tensor the path keeps between two of its steps) and `qw` (applied to
convolution weights before they are used).  Both are the identity by default, which
is the mathematics above and nothing else.  `set_storage(units, "bf16")` makes them
round to bfloat16, reproducing a path that holds those tensors in bfloat16 while it
accumulates, normalises and reduces in higher precision: the ReLU gates are then
decided on the same rounded values on both sides.  Sums that are formed and consumed
inside one step (a ReLU derivative times its incoming gradient, a residual sum before
its ReLU) are not rounded.

Parameter order inside a unit (and therefore inside a module's flat vector) is
the order of `param_spec()`; convolution weights are [C_out, R, S, C_in].
"""
from dataclasses import dataclass, field
from typing import Tuple
import numpy as np

from . import layers as L


@dataclass
class Arch:
    family: str = "resnet6n2"          # "resnet6n2" | "wrn"
    n_per_stage: int = 1
    widths: Tuple[int, int, int] = (16, 32, 64)
    stem_width: int = 16
    in_h: int = 32
    in_w: int = 32
    in_c: int = 3
    num_classes: int = 10
    batch: int = 128
    bn_eps: float = 1e-5
    blocks: Tuple[int, ...] = None     # residual blocks per stage; None: n_per_stage in each of len(widths) stages
    shortcut: str = "projection"       # "projection" | "zero_pad" (resnet6n2 only)

    def stage_blocks(self):
        return tuple(self.blocks) if self.blocks is not None else (self.n_per_stage,) * len(self.widths)


# ----------------------------------------------------------------------------
# units
# ----------------------------------------------------------------------------
class Stem:
    def __init__(self, arch):
        self.ci, self.co, self.eps = arch.in_c, arch.stem_width, arch.bn_eps
        self.with_bn = arch.family == "resnet6n2"
        self.name = "stem"
        self.q = self.qw = L.identity

    def param_spec(self):
        spec = [("conv.w", "conv", (self.co, 3, 3, self.ci))]
        if self.with_bn:
            spec += [("bn.g", "bn_gamma", (self.co,)), ("bn.b", "bn_beta", (self.co,))]
        return spec

    def bn_spec(self):
        """[(name, channels)] of the unit's batch norms, in the order their running statistics are kept."""
        return [("bn", self.co)] if self.with_bn else []

    def forward(self, x, p, running=None):
        q = self.q
        c = q(L.conv2d_forward(x, self.qw(p["conv.w"]), 1, 1))
        if not self.with_bn:
            return c, dict(x=x)
        if running is not None:
            L.batchnorm_running_update(running["bn"], c)
        b, sv = L.batchnorm_forward(c, p["bn.g"], p["bn.b"], self.eps)
        y = q(L.relu_forward(b))
        return y, dict(x=x, sv=sv, y=y)

    def forward_eval(self, x, p, running):
        q = self.q
        c = q(L.conv2d_forward(x, self.qw(p["conv.w"]), 1, 1))
        if not self.with_bn:
            return c
        return q(L.relu_forward(L.batchnorm_eval(c, p["bn.g"], p["bn.b"], running["bn"], self.eps)))

    def backward(self, dy, ctx, p):
        g = {}
        if self.with_bn:
            db = L.relu_backward(dy, ctx["y"])
            dc, g["bn.g"], g["bn.b"] = L.batchnorm_backward(db, ctx["sv"], p["bn.g"])
            dc = self.q(dc)
        else:
            dc = dy
        dx, g["conv.w"] = L.conv2d_backward(dc, ctx["x"], self.qw(p["conv.w"]), 1, 1)
        return self.q(dx), g


class BasicBlock:
    """Post-activation block of the 6n+2 networks."""

    def __init__(self, arch, ci, co, stride, index):
        self.ci, self.co, self.stride, self.eps = ci, co, stride, arch.bn_eps
        changes = (ci != co) or (stride != 1)
        self.proj = changes and arch.shortcut == "projection"
        self.zero_pad = changes and arch.shortcut == "zero_pad"
        assert not self.zero_pad or (co >= ci and (co - ci) % 2 == 0)
        self.name = "block%d" % index
        self.q = self.qw = L.identity

    def _pad_shortcut(self, x):
        """x at every stride-th pixel, (co - ci)/2 zero channels in front and behind."""
        lo = (self.co - self.ci) // 2
        xs = x[:, ::self.stride, ::self.stride, :]
        out = np.zeros(xs.shape[:3] + (self.co,), dtype=x.dtype)
        out[..., lo:lo + self.ci] = xs
        return out

    def _pad_shortcut_backward(self, dsc, x_shape):
        lo = (self.co - self.ci) // 2
        dx = np.zeros(x_shape, dtype=dsc.dtype)
        dx[:, ::self.stride, ::self.stride, :] = dsc[..., lo:lo + self.ci]
        return dx

    def param_spec(self):
        spec = [("conv1.w", "conv", (self.co, 3, 3, self.ci)),
                ("bn1.g", "bn_gamma", (self.co,)), ("bn1.b", "bn_beta", (self.co,)),
                ("conv2.w", "conv", (self.co, 3, 3, self.co)),
                ("bn2.g", "bn_gamma", (self.co,)), ("bn2.b", "bn_beta", (self.co,))]
        if self.proj:
            spec += [("sc.w", "conv", (self.co, 1, 1, self.ci)),
                     ("scbn.g", "bn_gamma", (self.co,)), ("scbn.b", "bn_beta", (self.co,))]
        return spec

    def bn_spec(self):
        return [("bn1", self.co), ("bn2", self.co)] + ([("scbn", self.co)] if self.proj else [])

    def forward(self, x, p, running=None):
        q, qw = self.q, self.qw
        c1 = q(L.conv2d_forward(x, qw(p["conv1.w"]), self.stride, 1))
        b1, sv1 = L.batchnorm_forward(c1, p["bn1.g"], p["bn1.b"], self.eps)
        a1 = q(L.relu_forward(b1))
        c2 = q(L.conv2d_forward(a1, qw(p["conv2.w"]), 1, 1))
        b2, sv2 = L.batchnorm_forward(c2, p["bn2.g"], p["bn2.b"], self.eps)
        ctx = dict(x=x, sv1=sv1, a1=a1, sv2=sv2)
        if running is not None:
            L.batchnorm_running_update(running["bn1"], c1)
            L.batchnorm_running_update(running["bn2"], c2)
        if self.proj:
            cs = q(L.conv2d_forward(x, qw(p["sc.w"]), self.stride, 0))
            sc, ctx["svs"] = L.batchnorm_forward(cs, p["scbn.g"], p["scbn.b"], self.eps)
            if running is not None:
                L.batchnorm_running_update(running["scbn"], cs)
        elif self.zero_pad:
            sc = self._pad_shortcut(x)
        else:
            sc = x
        y = q(L.relu_forward(b2 + sc))
        ctx["y"] = y
        return y, ctx

    def forward_eval(self, x, p, running):
        q, qw = self.q, self.qw
        c1 = q(L.conv2d_forward(x, qw(p["conv1.w"]), self.stride, 1))
        a1 = q(L.relu_forward(L.batchnorm_eval(c1, p["bn1.g"], p["bn1.b"], running["bn1"], self.eps)))
        c2 = q(L.conv2d_forward(a1, qw(p["conv2.w"]), 1, 1))
        b2 = L.batchnorm_eval(c2, p["bn2.g"], p["bn2.b"], running["bn2"], self.eps)
        if self.proj:
            cs = q(L.conv2d_forward(x, qw(p["sc.w"]), self.stride, 0))
            sc = L.batchnorm_eval(cs, p["scbn.g"], p["scbn.b"], running["scbn"], self.eps)
        elif self.zero_pad:
            sc = self._pad_shortcut(x)
        else:
            sc = x
        return q(L.relu_forward(b2 + sc))

    def backward(self, dy, ctx, p):
        g = {}
        q, qw = self.q, self.qw
        dsum = L.relu_backward(dy, ctx["y"])          # gradient of b2 + sc
        dc2, g["bn2.g"], g["bn2.b"] = L.batchnorm_backward(dsum, ctx["sv2"], p["bn2.g"])
        dc2 = q(dc2)
        da1, g["conv2.w"] = L.conv2d_backward(dc2, ctx["a1"], qw(p["conv2.w"]), 1, 1)
        db1 = L.relu_backward(q(da1), ctx["a1"])
        dc1, g["bn1.g"], g["bn1.b"] = L.batchnorm_backward(db1, ctx["sv1"], p["bn1.g"])
        dc1 = q(dc1)
        dx, g["conv1.w"] = L.conv2d_backward(dc1, ctx["x"], qw(p["conv1.w"]), self.stride, 1)
        if self.proj:
            dcs, g["scbn.g"], g["scbn.b"] = L.batchnorm_backward(dsum, ctx["svs"], p["scbn.g"])
            dcs = q(dcs)
            dxs, g["sc.w"] = L.conv2d_backward(dcs, ctx["x"], qw(p["sc.w"]), self.stride, 0)
            dx = dx + q(dxs)
        elif self.zero_pad:
            dx = dx + self._pad_shortcut_backward(dsum, dx.shape)
        else:
            dx = dx + dsum
        return q(dx), g


class PreActBlock:
    """Pre-activation block of the wide residual networks."""

    def __init__(self, arch, ci, co, stride, index):
        self.ci, self.co, self.stride, self.eps = ci, co, stride, arch.bn_eps
        self.proj = (ci != co) or (stride != 1)
        self.name = "block%d" % index
        self.q = self.qw = L.identity

    def param_spec(self):
        spec = [("bn1.g", "bn_gamma", (self.ci,)), ("bn1.b", "bn_beta", (self.ci,)),
                ("conv1.w", "conv", (self.co, 3, 3, self.ci)),
                ("bn2.g", "bn_gamma", (self.co,)), ("bn2.b", "bn_beta", (self.co,)),
                ("conv2.w", "conv", (self.co, 3, 3, self.co))]
        if self.proj:
            spec += [("sc.w", "conv", (self.co, 1, 1, self.ci))]
        return spec

    def bn_spec(self):
        return [("bn1", self.ci), ("bn2", self.co)]

    def forward_eval(self, x, p, running):
        q, qw = self.q, self.qw
        o = q(L.relu_forward(L.batchnorm_eval(x, p["bn1.g"], p["bn1.b"], running["bn1"], self.eps)))
        c1 = q(L.conv2d_forward(o, qw(p["conv1.w"]), self.stride, 1))
        a2 = q(L.relu_forward(L.batchnorm_eval(c1, p["bn2.g"], p["bn2.b"], running["bn2"], self.eps)))
        c2 = L.conv2d_forward(a2, qw(p["conv2.w"]), 1, 1)
        sc = q(L.conv2d_forward(o, qw(p["sc.w"]), self.stride, 0)) if self.proj else x
        return q(c2 + sc)

    def forward(self, x, p, running=None):
        q, qw = self.q, self.qw
        if running is not None:
            L.batchnorm_running_update(running["bn1"], x)
        b1, sv1 = L.batchnorm_forward(x, p["bn1.g"], p["bn1.b"], self.eps)
        o = q(L.relu_forward(b1))
        c1 = q(L.conv2d_forward(o, qw(p["conv1.w"]), self.stride, 1))
        if running is not None:
            L.batchnorm_running_update(running["bn2"], c1)
        b2, sv2 = L.batchnorm_forward(c1, p["bn2.g"], p["bn2.b"], self.eps)
        a2 = q(L.relu_forward(b2))
        c2 = L.conv2d_forward(a2, qw(p["conv2.w"]), 1, 1)
        if self.proj:
            sc = q(L.conv2d_forward(o, qw(p["sc.w"]), self.stride, 0))
        else:
            sc = x
        y = q(c2 + sc)
        return y, dict(sv1=sv1, o=o, sv2=sv2, a2=a2)

    def backward(self, dy, ctx, p):
        g = {}
        q, qw = self.q, self.qw
        da2, g["conv2.w"] = L.conv2d_backward(dy, ctx["a2"], qw(p["conv2.w"]), 1, 1)
        db2 = L.relu_backward(q(da2), ctx["a2"])
        dc1, g["bn2.g"], g["bn2.b"] = L.batchnorm_backward(db2, ctx["sv2"], p["bn2.g"])
        dc1 = q(dc1)
        do, g["conv1.w"] = L.conv2d_backward(dc1, ctx["o"], qw(p["conv1.w"]), self.stride, 1)
        if self.proj:
            dos, g["sc.w"] = L.conv2d_backward(dy, ctx["o"], qw(p["sc.w"]), self.stride, 0)
            do = do + q(dos)
        db1 = L.relu_backward(q(do), ctx["o"])
        dx, g["bn1.g"], g["bn1.b"] = L.batchnorm_backward(db1, ctx["sv1"], p["bn1.g"])
        if not self.proj:
            dx = dx + dy
        return q(dx), g


class Head:
    """Classifier and loss.  The paper's f is abstract (Eq. 1); the task is
    classification, so f is the mean softmax cross-entropy over the batch."""

    def __init__(self, arch, feat):
        self.feat, self.classes, self.eps = feat, arch.num_classes, arch.bn_eps
        self.with_bn = arch.family == "wrn"
        self.name = "head"
        self.q = self.qw = L.identity

    def param_spec(self):
        spec = []
        if self.with_bn:
            spec += [("bn.g", "bn_gamma", (self.feat,)), ("bn.b", "bn_beta", (self.feat,))]
        spec += [("fc.w", "fc_w", (self.classes, self.feat)), ("fc.b", "fc_b", (self.classes,))]
        return spec

    def bn_spec(self):
        return [("bn", self.feat)] if self.with_bn else []

    def logits_eval(self, x, p, running):
        if self.with_bn:
            x = self.q(L.relu_forward(L.batchnorm_eval(x, p["bn.g"], p["bn.b"], running["bn"], self.eps)))
        return L.fc_forward(L.gap_forward(x), p["fc.w"], p["fc.b"])

    def forward_loss(self, x, labels, p, running=None):
        ctx = dict(shape=x.shape)
        if self.with_bn:
            if running is not None:
                L.batchnorm_running_update(running["bn"], x)
            b, ctx["sv"] = L.batchnorm_forward(x, p["bn.g"], p["bn.b"], self.eps)
            x = self.q(L.relu_forward(b))
            ctx["a"] = x
        pooled = L.gap_forward(x)
        logits = L.fc_forward(pooled, p["fc.w"], p["fc.b"])
        loss, probs = L.softmax_xent_forward(logits, labels)
        ctx.update(pooled=pooled, probs=probs, labels=labels, logits=logits)
        return loss, ctx

    def backward(self, ctx, p):
        g = {}
        dlogits = L.softmax_xent_backward(ctx["probs"], ctx["labels"])
        dpooled, g["fc.w"], g["fc.b"] = L.fc_backward(dlogits, ctx["pooled"], p["fc.w"])
        dx = self.q(L.gap_backward(dpooled, ctx["shape"]))
        if self.with_bn:
            db = L.relu_backward(dx, ctx["a"])
            dx, g["bn.g"], g["bn.b"] = L.batchnorm_backward(db, ctx["sv"], p["bn.g"])
            dx = self.q(dx)
        return dx, g


# ----------------------------------------------------------------------------
# network = stem + 3n blocks + head, and its partition into K modules
# ----------------------------------------------------------------------------
def build_units(arch):
    units = [Stem(arch)]
    block_cls = BasicBlock if arch.family == "resnet6n2" else PreActBlock
    assert arch.shortcut in ("projection", "zero_pad") and (arch.shortcut == "projection" or arch.family == "resnet6n2")
    ci = arch.stem_width
    index = 0
    for stage, n_blocks in enumerate(arch.stage_blocks()):
        for j in range(n_blocks):
            index += 1
            stride = 2 if (stage > 0 and j == 0) else 1
            units.append(block_cls(arch, ci, arch.widths[stage], stride, index))
            ci = arch.widths[stage]
    units.append(Head(arch, ci))
    return units


def set_storage(units, storage):
    """storage None: exact arithmetic in the working dtype.  "bf16": activations,
    gradients and convolution weights are rounded to bfloat16 wherever they are kept."""
    assert storage in (None, "bf16"), storage
    f = L.round_bf16 if storage == "bf16" else L.identity
    for u in units:
        u.q = u.qw = f


def split_units(units, split_after_block):
    """Partition [stem, block1..blockN, head] at the given block indices
    (ascending, 1-based): the paper's q(1)..q(K) with module 1 holding the stem
    and module K the head."""
    n_blocks = len(units) - 2
    cuts = list(split_after_block)
    assert all(1 <= c < n_blocks for c in cuts) and cuts == sorted(set(cuts)), cuts
    bounds = [0] + [c + 1 for c in cuts] + [len(units)]
    return [units[bounds[k]:bounds[k + 1]] for k in range(len(bounds) - 1)]


def module_param_spec(module_units):
    """[(qualified name, kind, shape)] in flat-vector order."""
    spec = []
    for u in module_units:
        for name, kind, shape in u.param_spec():
            spec.append((u.name + "." + name, kind, shape))
    return spec


def module_bn_spec(module_units):
    """[(qualified name, channels)] of a module's batch norms; a module's flat vector of running statistics is,
    for each of them in this order, the running mean then the running variance."""
    return [(u.name + "." + name, ch) for u in module_units for name, ch in u.bn_spec()]


def spec_size(spec):
    return int(sum(int(np.prod(s)) for _, _, s in spec))


def unflatten(flat, spec):
    """Views into `flat`, keyed by qualified name."""
    out, off = {}, 0
    for name, _, shape in spec:
        n = int(np.prod(shape))
        out[name] = flat[off:off + n].reshape(shape)
        off += n
    assert off == flat.size
    return out


def flatten(named, spec, dtype):
    return np.concatenate([np.asarray(named[name], dtype=dtype).reshape(-1) for name, _, _ in spec]) \
        if spec else np.zeros(0, dtype=dtype)


def unit_params(named, unit):
    """The sub-dictionary of one unit with the unit prefix stripped."""
    pre = unit.name + "."
    return {k[len(pre):]: v for k, v in named.items() if k.startswith(pre)}
