"""Runs the CUDA library and the CPU oracle side by side on the same seeded inputs
and compares them step by step.  Used by the GPU parity tests and the smoke check."""
import numpy as np

import fdg_synth as S
from oracle import fdg as ofdg
from oracle import nets as onets


def relmax(a, b):
    """max|a-b| / max|b| (b = oracle)."""
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30))


def relfro(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-30))


def run_pair(arch_kw, K, splits, steps, beta=0.5, lr=0.1, momentum=0.9, weight_decay=5e-4,
             order="backward_first", weight_reading="stashed", precision="fp32", serial=False, seed=0,
             jitter=True, oracle_dtype=np.float64, check_every_step=True, graphs=False, plain=None):
    """Returns a dict of worst-case errors and the two schedule logs.

    In bf16 mode every error is measured twice: against the oracle with bfloat16 storage (keys "out", "gin",
    "loss", "grads", "params": the same tensors rounded on both sides, so every ReLU gate is decided on the
    same values) and against the plain float64 oracle, which rounds nothing (the same keys with "_plain"):
    the second figure includes what keeping activations, gradients and weights in bfloat16 costs.
    `plain=False` skips the second oracle (deep networks, where it doubles a long CPU run)."""
    import torch
    from paper_1906_09108_b200 import binding as B

    arch_o = onets.Arch(**arch_kw)
    cfg_o = ofdg.FDGConfig(K=K, split_after_block=tuple(splits), beta=beta, lr=lr, momentum=momentum,
                           weight_decay=weight_decay, order=order, weight_reading=weight_reading)
    # In bf16 mode the library keeps activations, gradients and convolution weights in
    # bfloat16; the oracle then rounds the same tensors, so that both sides decide every
    # ReLU gate on the same values (everything else stays float64 in the oracle).
    orc = ofdg.FDGOracle(arch_o, cfg_o, dtype=oracle_dtype, storage="bf16" if precision == "bf16" else None)
    if plain is None:
        plain = precision == "bf16"
    orc_plain = ofdg.FDGOracle(arch_o, cfg_o, dtype=oracle_dtype, storage=None) if plain else None
    g = B.FDG(B.make_arch(**arch_kw), K=K, split_after_block=tuple(splits), beta=beta, lr=lr, momentum=momentum,
              weight_decay=weight_decay,
              order=B.FDG_BACKWARD_FIRST if order == "backward_first" else B.FDG_FORWARD_FIRST,
              weight_reading=B.FDG_STASHED if weight_reading == "stashed" else B.FDG_CURRENT,
              precision=B.FDG_FP32_CUDACORE if precision == "fp32" else B.FDG_BF16_TC, serial=serial, graphs=graphs)
    for k in range(1, K + 1):
        spec_o = [(kind, tuple(shape)) for _, kind, shape in orc.param_spec(k)]
        spec_g = [(kind, tuple(shape)) for _, kind, shape in g.param_layout(k)]
        assert spec_o == spec_g, "parameter layouts differ in module %d" % k
        p = S.init_params(seed, k, orc.param_spec(k), jitter=jitter)
        orc.set_params(k, p)
        if orc_plain is not None:
            orc_plain.set_params(k, p)
        g.set_params(k, p)
    a = arch_o
    res = dict(out=0.0, gin=0.0, loss=0.0, grads=0.0, steps=steps)
    if orc_plain is not None:
        res.update(out_plain=0.0, gin_plain=0.0, loss_plain=0.0, grads_plain=0.0)
    res["grads_by_step"] = []          # (t, k, error): where a failure started, for the assertion message
    res["worst_tensors"] = []          # the three worst parameter tensors at the worst (t, k)
    layouts = {k: g.param_layout(k) for k in range(1, K + 1)}
    loss_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    for t in range(1, steps + 1):
        x = S.images(seed, t, a.batch, a.in_h, a.in_w, a.in_c)
        y = S.labels(seed, t, a.batch, a.num_classes)
        lo = orc.step(x, y)
        lo_plain = orc_plain.step(x, y) if orc_plain is not None else None
        g.step(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), loss_dev)
        if not (check_every_step or t == steps):
            continue
        g.sync()
        if lo is not None:
            res["loss"] = max(res["loss"], abs(float(loss_dev.item()) - lo) / max(abs(lo), 1e-30))
            if lo_plain is not None:
                res["loss_plain"] = max(res["loss_plain"], abs(float(loss_dev.item()) - lo_plain) / max(abs(lo_plain), 1e-30))
        for k in range(1, K + 1):
            if k < K and orc.module_output[k] is not None:
                b, out = g.module_output(k)
                bo, oo = orc.module_output[k]
                assert b == bo, ("module output batch", t, k, b, bo)
                res["out"] = max(res["out"], relmax(out, oo.reshape(-1)))
                if orc_plain is not None:
                    res["out_plain"] = max(res["out_plain"], relmax(out, orc_plain.module_output[k][1].reshape(-1)))
            if k >= 2 and orc.input_grad[k] is not None:
                b, gi = g.input_grad(k)
                bo, go = orc.input_grad[k]
                assert b == bo, ("input grad batch", t, k, b, bo)
                res["gin"] = max(res["gin"], relmax(gi, go.reshape(-1)))
                if orc_plain is not None:
                    res["gin_plain"] = max(res["gin_plain"], relmax(gi, orc_plain.input_grad[k][1].reshape(-1)))
            go = orc.get_grads(k)
            if go is not None:
                gg = g.get_grads(k)
                if orc_plain is not None:
                    res["grads_plain"] = max(res["grads_plain"], relfro(gg, orc_plain.get_grads(k)))
                err = relfro(gg, go)
                res["grads_by_step"].append((t, k, float("%.3g" % err)))
                if err > res["grads"]:
                    res["grads"] = err
                    per = []
                    for name, _, shape in layouts[k]:
                        off, n = int(name.split("@")[1]), int(np.prod(shape))
                        per.append((round(relfro(gg[off:off + n], go[off:off + n]), 4), t, k, name, tuple(shape)))
                    res["worst_tensors"] = sorted(per, reverse=True)[:3]
    g.sync()
    res["params"] = max(relfro(g.get_params(k), orc.get_params(k)) for k in range(1, K + 1))
    res["momentum"] = max(relfro(g.get_momentum(k), orc.get_momentum(k)) for k in range(1, K + 1))
    if orc_plain is not None:
        res["params_plain"] = max(relfro(g.get_params(k), orc_plain.get_params(k)) for k in range(1, K + 1))
    res["log_gpu"] = [(r["t"], r["k"], r["tau_f"], r["tau_b"], r["ver_f"], r["ver_b"]) for r in g.schedule_log()]
    res["log_oracle"] = [(r["t"], r["k"], r["tau_f"], r["tau_b"], r["ver_f"], r["ver_b"]) for r in orc.log]
    res["launches"] = g.launch_count()
    assert g.check_guards() == -1          # no kernel wrote past the end of a workspace buffer
    g.close()
    return res
