"""CPU oracle, part 3: the FDG iteration (Algorithm I) over K modules.

TEST INFRASTRUCTURE ONLY (see oracle/layers.py).

One call of `step` is one iteration t of Algorithm I for every module k=1..K:

  * forward  (Section 3.1, "forward"): module k forwards batch tau_f = t-k+1,
    received from module k-1 at the end of iteration t-1 (module 1 reads the
    images handed to this call, which are batch t).
  * backward (Section 3.1, "backward", Eq. 10, with shrinking Eq. 15): module k
    back-propagates batch tau_b = t-2K+k+1 from the gradient module k+1 sent at
    the end of iteration t-1, multiplied by beta (modules k<K only; the top
    module's gradient comes from the loss and is not shrunk, paragraph after
    Eq. 15).  The Jacobians are taken at the activations saved by the forward
    of that same batch (the paragraph after Eq. 10 requires forward and backward of a
    batch to meet the same activations).
  * update (Eq. 11) with the SGD-momentum / weight-decay optimiser of the
    experiments section.
  * communication (Section 3.1, "communication"; Fig. 1(a): "right before the
    iteration ends"): outputs go into mailboxes that become visible at t+1, so
    the order in which the modules are visited inside an iteration is
    irrelevant ("Parallel for k").

Readings taken where the paper leaves a choice:
  order           "backward_first" is Algorithm I; "forward_first" is the
                  FDG-forward variant of Appendix A.  Module K has delay 0 and
                  always runs forward -> loss -> backward -> update.
  weight_reading  "stashed": the delayed backward uses the weights the forward
                  of that batch used (superscripts of Eq. 10 / Eq. 13);
                  "current": it uses the weights as they are now.
  pipeline fill   a step whose batch index is < 1 is skipped, update included.
  optimiser       g = ghat + wd*theta ; v = mu*v + g (v = g the first time) ;
                  theta = theta - lr*v.  beta never scales the wd term.

The rest of the training recipe of the experiments section, which the paper names but does not
spell out, each with the reading taken:
  learning rate   `learning_rate`: the step schedule (divide by 10 at epochs 150, 225, 275) with the
                  optional warm-up at 0.01 for the first 3 epochs, one value per iteration.
  test accuracy   running batch-norm statistics are kept by every forward (oracle/layers.py,
                  batchnorm_running_update) and `eval_logits` / `top1` run the network in inference
                  mode with the current weights of all modules.
  end of training `drain`: the paper stops after T iterations and leaves 2(K-k) batches of module k
                  without their gradient; drain runs the 2K-2 further iterations of Algorithm I in
                  which no new batch enters, so that every batch is back-propagated by every module.
  checkpoint      `state` / `load_state`: everything in flight (saved contexts, mailboxes, label
                  queue, running statistics, momentum, counters), so that a restored run continues
                  bit for bit.
"""
import copy
from dataclasses import dataclass
from typing import Tuple
import numpy as np

from . import nets

BACKWARD_FIRST = "backward_first"
FORWARD_FIRST = "forward_first"
STASHED = "stashed"
CURRENT = "current"


@dataclass
class FDGConfig:
    K: int = 2
    split_after_block: Tuple[int, ...] = (1,)
    beta: float = 1.0
    lr: float = 0.1
    momentum: float = 0.9
    weight_decay: float = 5e-4
    order: str = BACKWARD_FIRST
    weight_reading: str = STASHED


def learning_rate(iteration, iters_per_epoch, base_lr=0.1, milestones=(150, 225, 275), gamma=0.1,
                  warmup_epochs=0, warmup_lr=0.01):
    """Learning rate of iteration `iteration` (from 1), experiments section: start at base_lr, divide by
    10 at each milestone epoch; for the deep networks and K = 3, 4 the first 3 epochs run at 0.01
    (warm-up).  Epoch e (from 0) holds iterations e*iters_per_epoch+1 .. (e+1)*iters_per_epoch."""
    epoch = (iteration - 1) // iters_per_epoch
    if epoch < warmup_epochs:
        return warmup_lr
    lr = base_lr
    for m in milestones:
        if epoch >= m:
            lr = lr * gamma
    return lr


def forward_batch(t, k):
    """Batch forwarded by module k (1-based) at iteration t: t-k+1."""
    return t - k + 1


def backward_batch(t, k, K):
    """Batch back-propagated by module k at iteration t: t-2K+k+1."""
    return t - 2 * K + k + 1


class _Module:
    def __init__(self, units, dtype):
        self.units = units
        self.spec = nets.module_param_spec(units)
        n = nets.spec_size(self.spec)
        self.theta = np.zeros(n, dtype=dtype)
        self.v = np.zeros(n, dtype=dtype)
        self.updates = 0                 # u_k: how many updates theta has received
        self.saved = {}                  # batch index -> saved context
        self.last_grad = None            # last ghat_theta (shrunk, before wd), flat
        self.bn_spec = nets.module_bn_spec(units)
        # running statistics per unit: {unit name: {bn name: [mean, var]}}, started at mean 0 / variance 1
        self.running = {u.name: {name: [np.zeros(ch, dtype=dtype), np.ones(ch, dtype=dtype)] for name, ch in u.bn_spec()}
                        for u in units}


class FDGOracle:
    def __init__(self, arch, cfg, dtype=np.float64, storage=None):
        assert cfg.K == len(cfg.split_after_block) + 1
        self.arch, self.cfg, self.dtype = arch, cfg, np.dtype(dtype)
        self.K = cfg.K
        units = nets.build_units(arch)
        nets.set_storage(units, storage)          # None: exact; "bf16": see oracle/nets.py
        self.q = units[0].q
        parts = nets.split_units(units, cfg.split_after_block)
        self.modules = [_Module(u, self.dtype) for u in parts]
        self.lr = cfg.lr
        self.t = 0
        # mailboxes: what was sent at the end of the previous iteration
        self.act_in = [None] * (self.K + 2)     # act_in[k]  = (batch, tensor) for module k
        self.grad_in = [None] * (self.K + 2)    # grad_in[k] = (batch, tensor) for module k
        self.labels = {}                        # batch -> labels, until module K uses them
        self.images = {}
        self.module_output = [None] * (self.K + 1)   # [k] = (batch, tensor) last produced
        self.input_grad = [None] * (self.K + 1)      # [k] = (batch, tensor) last produced
        self.loss = None                             # (batch, value) last produced
        self.log = []                                # schedule log, one row per (t, k)
        self.schedule = None                         # keyword arguments of learning_rate, or None: lr stays as set
        self.last_batch = None                       # set by drain(): no batch beyond it exists

    # -- parameters ----------------------------------------------------------
    def param_spec(self, k):
        return self.modules[k - 1].spec

    def param_count(self, k):
        return self.modules[k - 1].theta.size

    def set_params(self, k, flat):
        m = self.modules[k - 1]
        assert flat.size == m.theta.size
        m.theta[:] = flat

    def get_params(self, k):
        return self.modules[k - 1].theta.copy()

    def get_momentum(self, k):
        return self.modules[k - 1].v.copy()

    def get_grads(self, k):
        g = self.modules[k - 1].last_grad
        return None if g is None else g.copy()

    def set_lr(self, lr):
        self.lr = lr

    def set_schedule(self, **kw):
        """From the next step on, iteration t runs at learning_rate(t, **kw)."""
        self.schedule = kw

    def get_running(self, k):
        """Flat running statistics of module k: for each batch norm in module order, mean then variance."""
        m = self.modules[k - 1]
        parts = []
        for u in m.units:
            for name, _ in u.bn_spec():
                parts += [m.running[u.name][name][0], m.running[u.name][name][1]]
        return np.concatenate(parts) if parts else np.zeros(0, dtype=self.dtype)

    def set_running(self, k, flat):
        m, off = self.modules[k - 1], 0
        for u in m.units:
            for name, ch in u.bn_spec():
                m.running[u.name][name][0][:] = flat[off:off + ch]
                m.running[u.name][name][1][:] = flat[off + ch:off + 2 * ch]
                off += 2 * ch
        assert off == flat.size

    # -- inference -------------------------------------------------------------
    def eval_logits(self, images):
        """The whole network in inference mode: current weights of every module, running statistics."""
        x = self.q(np.asarray(images, dtype=self.dtype))
        for m in self.modules:
            named = nets.unflatten(m.theta, m.spec)
            for u in m.units:
                p = nets.unit_params(named, u)
                if isinstance(u, nets.Head):
                    return u.logits_eval(x, p, m.running[u.name])
                x = u.forward_eval(x, p, m.running[u.name])

    def top1(self, images, labels):
        """Number of samples whose largest logit is at the label (ties: the lowest class index wins)."""
        return int((np.argmax(self.eval_logits(images), axis=1) == np.asarray(labels)).sum())

    # -- checkpoint ------------------------------------------------------------
    _STATE = ("modules", "lr", "t", "act_in", "grad_in", "labels", "images", "module_output", "input_grad", "loss",
              "log", "schedule", "last_batch")

    def state(self):
        """Everything a continued run depends on, copied."""
        return copy.deepcopy({name: getattr(self, name) for name in self._STATE})

    def load_state(self, state):
        for name, value in copy.deepcopy(state).items():
            setattr(self, name, value)
        for m in self.modules:                      # the units' rounding maps are functions: keep this oracle's
            for u in m.units:
                u.q = u.qw = self.q

    # -- pieces of one module-step -------------------------------------------
    def _forward(self, k, tau, x):
        """Forward of batch tau with the module's current weights; saves context."""
        m = self.modules[k - 1]
        theta_used = m.theta.copy()
        named = nets.unflatten(theta_used, m.spec)
        ctxs = []
        for u in m.units:
            if isinstance(u, nets.Head):
                loss, c = u.forward_loss(x, self.labels.pop(tau), nets.unit_params(named, u), m.running[u.name])
                ctxs.append(c)
                x = None
                self.loss = (tau, float(loss))
            else:
                x, c = u.forward(x, nets.unit_params(named, u), m.running[u.name])
                ctxs.append(c)
        m.saved[tau] = dict(batch=tau, ctxs=ctxs, theta=theta_used, version=m.updates)
        return x

    def _backward(self, k, tau, g):
        """Chain rule through module k for batch tau; returns (grad wrt module input,
        flat parameter gradient, weight version used)."""
        m = self.modules[k - 1]
        saved = m.saved.pop(tau)
        assert saved["batch"] == tau                      # same-batch rule
        if self.cfg.weight_reading == STASHED:
            theta, version = saved["theta"], saved["version"]
        else:
            theta, version = m.theta, m.updates
        named = nets.unflatten(theta, m.spec)
        grads = {}
        for u, c in zip(reversed(m.units), reversed(saved["ctxs"])):
            p = nets.unit_params(named, u)
            if isinstance(u, nets.Head):
                g, gu = u.backward(c, p)
            else:
                g, gu = u.backward(g, c, p)
            for name, val in gu.items():
                grads[u.name + "." + name] = val
        return g, nets.flatten(grads, m.spec, self.dtype), version

    def _update(self, k, ghat):
        m = self.modules[k - 1]
        c = self.cfg
        dt = self.dtype.type
        g = ghat + dt(c.weight_decay) * m.theta
        m.v = g.copy() if m.updates == 0 else dt(c.momentum) * m.v + g
        m.theta = m.theta - dt(self.lr) * m.v
        m.updates += 1
        m.last_grad = ghat

    # -- one iteration of Algorithm I ----------------------------------------
    def step(self, images, labels):
        """Iteration t (t counts calls from 1).  `images` [B,H,W,C], `labels` [B]
        are batch t.  Returns the loss produced in this iteration (batch t-K+1)
        or None while the pipeline fills."""
        self.t += 1
        t, K = self.t, self.K
        if self.schedule is not None:
            self.lr = learning_rate(t, **self.schedule)
        if images is not None:
            self.images[t] = self.q(np.asarray(images, dtype=self.dtype))
            self.labels[t] = np.asarray(labels).astype(np.int64)
        new_act = [None] * (K + 2)
        new_grad = [None] * (K + 2)
        loss_out = None

        for k in range(1, K + 1):
            tau_f = forward_batch(t, k)
            tau_b = backward_batch(t, k, K)
            row = dict(t=t, k=k, tau_f=-1, tau_b=-1, ver_f=-1, ver_b=-1)

            def do_forward():
                if tau_f < 1 or (self.last_batch is not None and tau_f > self.last_batch):
                    return
                if k == 1:
                    x = self.images.pop(tau_f)
                else:
                    b, x = self.act_in[k]
                    assert b == tau_f
                row["tau_f"], row["ver_f"] = tau_f, self.modules[k - 1].updates
                y = self._forward(k, tau_f, x)
                if k < K:
                    new_act[k + 1] = (tau_f, y)
                    self.module_output[k] = (tau_f, y)

            def do_backward_update():
                if tau_b < 1 or (self.last_batch is not None and tau_b > self.last_batch):
                    return
                if k < K:
                    b, g = self.grad_in[k]
                    assert b == tau_b
                    g = self.q(self.dtype.type(self.cfg.beta) * g)   # Eq. 15
                else:
                    g = None                                       # from the loss
                gin, ghat, ver = self._backward(k, tau_b, g)
                row["tau_b"], row["ver_b"] = tau_b, ver
                self._update(k, ghat)                              # Eq. 11
                self.input_grad[k] = (tau_b, gin)
                if k > 1:
                    new_grad[k - 1] = (tau_b, gin)

            if k == K:
                do_forward()
                if row["tau_f"] >= 1:
                    loss_out = self.loss[1]
                do_backward_update()
            elif self.cfg.order == BACKWARD_FIRST:
                do_backward_update()
                do_forward()
            else:
                do_forward()
                do_backward_update()
            self.log.append(row)

        # communication, visible from iteration t+1 on
        self.act_in, self.grad_in = new_act, new_grad
        return loss_out

    def drain(self):
        """Runs the 2K-2 iterations of Algorithm I that follow the last batch, with no new batch entering:
        module k still forwards the batches its upstream sent (up to the last one) and back-propagates the
        2(K-k) batches it holds.  Afterwards every module has applied one update per batch, nothing is in
        flight, and the iteration counter restarts at 0 with the trained weights (a fresh pipeline)."""
        self.last_batch = self.t
        for _ in range(2 * self.K - 2):
            self.step(None, None)
        assert all(not m.saved for m in self.modules) and not self.labels and not self.images
        self.t = 0
        self.last_batch = None
        self.act_in = [None] * (self.K + 2)
        self.grad_in = [None] * (self.K + 2)
