"""FDG training throughput on B200: `python bench.py --gpus N --steps K --warmup W`.

Workload: ResNet-110 (6n+2, n=18, 16/32/64 channels), K=4 modules split after blocks
13/27/41, batch 128, 32x32x3 synthetic N(0,1) images, 10 uniform classes, beta 0.2,
lr 0.01, momentum 0.9, weight decay 5e-4, one CUDA stream per module.  A step is one
call of fdg_step: one iteration of Algorithm I for all four modules (ingest, shrink,
backward, update, forward, handoff).  The pipeline is filled before timing.

Prints ONE JSON line (rank 0).  `value` = images/s with the 16 input batches resident in
HBM; `e2e` = the same through fdg_step_host from pinned host memory with the loss read
back every step; `roofline` = the dominant kernel class timed alone (serial context, CUDA
events on its stream) against the measured peak; `cpu_baseline` = the CPU oracle on a
bounded sample.  `--impl reference` times the oracle alone on the host cores.
With N > 1 (torchrun) every rank runs an independent replica: the path has no
inter-GPU step, so there is no collective on the data path.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

ARCH = dict(family="resnet6n2", n_per_stage=18, widths=(16, 32, 64), stem_width=16, in_h=32, in_w=32, in_c=3,
            num_classes=10, batch=128)
K_MODULES = 4
SPLITS = (13, 27, 41)
BETA, LR, MOM, WD = 0.2, 0.01, 0.9, 5e-4

# The other workloads of the paper's tables that the library is measured on (--workload); the
# default, and the only one the bench line's metric is quoted on, is resnet110_k4.


def profiled_traffic(summary="conv_halo_kernel_fprop_stage1.md", source="conv_halo.cuh"):
    """DRAM bytes per launch of the dominant kernel from its committed ncu summary (the line
    `traffic_bytes_per_launch: N`), or None when the summary is missing or was taken on another version of the
    kernel's source (the line `kernel_source_sha16: H` holds the first 16 hex digits of the source's SHA-256)."""
    import hashlib
    import re
    try:
        text = open(os.path.join(ROOT, "profiles", summary)).read()
        src = open(os.path.join(ROOT, "paper_1906_09108_b200", "csrc", source), "rb").read()
    except OSError:
        return None
    t = re.search(r"^traffic_bytes_per_launch:\s*(\d+)", text, re.M)
    h = re.search(r"^kernel_source_sha16:\s*([0-9a-f]{16})", text, re.M)
    if not t or not h or h.group(1) != hashlib.sha256(src).hexdigest()[:16]:
        return None
    return int(t.group(1))


WORKLOADS = {
    "tiny_k2": dict(arch=dict(family="resnet6n2", n_per_stage=1, widths=(8, 16, 32), stem_width=8, in_h=16, in_w=16,
                              in_c=3, num_classes=10, batch=8), K=2, splits=(1,), beta=0.2, lr=0.1,
                    name="tiny 6n+2 (n=1, 8/16/32 channels, 16x16) K=2 batch 8"),
    "resnet56_k2": dict(arch=dict(family="resnet6n2", n_per_stage=9, widths=(16, 32, 64), stem_width=16, in_h=32, in_w=32,
                                  in_c=3, num_classes=10, batch=128), K=2, splits=(13,), beta=0.5, lr=0.1,
                        name="ResNet-56 (6n+2, n=9) K=2 batch 128, 32x32x3 synthetic N(0,1), 10 classes"),
    "resnet110_k4": None,
    "wrn28_10_k2": dict(arch=dict(family="wrn", n_per_stage=4, widths=(160, 320, 640), stem_width=16, in_h=32, in_w=32,
                                  in_c=3, num_classes=100, batch=128), K=2, splits=(6,), beta=0.6, lr=0.1,
                        name="WRN-28-10 K=2 batch 128, 32x32x3 synthetic N(0,1), 100 classes"),
    "resnet18_k2": dict(arch=dict(family="resnet6n2", blocks=(2, 2, 2, 2), widths=(64, 128, 256, 512), stem_width=64, in_h=32,
                                  in_w=32, in_c=3, num_classes=10, batch=128), K=2, splits=(4,), beta=0.5, lr=0.1,
                        name="CIFAR ResNet-18 (4 stages of 2 basic blocks, 64..512 channels) K=2 batch 128, 32x32x3 synthetic N(0,1)"),
    "resnet1202_k4": dict(arch=dict(family="resnet6n2", n_per_stage=200, widths=(16, 32, 64), stem_width=16, in_h=32,
                                    in_w=32, in_c=3, num_classes=10, batch=64), K=4, splits=(150, 300, 450), beta=0.5,
                          lr=0.01, name="ResNet-1202 (6n+2, n=200) K=4 batch 64, 32x32x3 synthetic N(0,1), 10 classes"),
}


def select_workload(name):
    global ARCH, K_MODULES, SPLITS, BETA, LR, WORKLOAD
    w = WORKLOADS[name]
    if w is None:
        return
    global METRIC
    ARCH, K_MODULES, SPLITS, BETA, LR, WORKLOAD = w["arch"], w["K"], w["splits"], w["beta"], w["lr"], w["name"]
    METRIC = "FDG train images/sec on 1 B200 (%s)" % name
WORKLOAD = "ResNet-110 (6n+2, n=18) K=4 batch 128, 32x32x3 synthetic N(0,1), 10 classes"
METRIC = "FDG train images/sec on 1 B200 (ResNet-110, K=4)"
POOL = 16
ORACLE_SAMPLE_BATCH = 16


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------ oracle arm --
def oracle_images_per_s(steps, warmup, batch=ORACLE_SAMPLE_BATCH):
    """The CPU oracle as it stands, same network / K / hyper-parameters, on a batch-`batch`
    sample of the workload; the pipeline is filled (2K iterations) before warm-up."""
    import torch
    import fdg_synth as S
    from oracle import fdg as ofdg
    from oracle import nets as onets
    arch = dict(ARCH, batch=batch)
    o = ofdg.FDGOracle(onets.Arch(**arch), ofdg.FDGConfig(K=K_MODULES, split_after_block=SPLITS, beta=BETA, lr=LR,
                                                         momentum=MOM, weight_decay=WD))
    for k in range(1, K_MODULES + 1):
        o.set_params(k, S.init_params(0, k, o.param_spec(k)))
    t = 0

    def one():
        nonlocal t
        t += 1
        o.step(S.images(0, t, batch, ARCH["in_h"], ARCH["in_w"], 3), S.labels(0, t, batch, ARCH["num_classes"]))

    for _ in range(2 * K_MODULES + warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = time.perf_counter() - t0
    return batch * steps / dt, dt / steps, torch.get_num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = args.steps if args.steps is not None else 4
    warmup = args.warmup if args.warmup is not None else 1
    ips, sec, cores = oracle_images_per_s(steps, warmup)
    sample = ("same network, K and hyper-parameters at batch %d of 128; pipeline filled (2K iterations) before the "
              "warm-up; numpy float64" % ORACLE_SAMPLE_BATCH)
    line = dict(impl="reference", metric=METRIC, value=ips, unit="images/s", n_gpus=args.gpus, steps=steps,
                warmup=warmup, ms_per_step=sec * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", config=dict(workload=WORKLOAD, K=K_MODULES, global_batch=ARCH["batch"]),
                cpu_baseline=dict(value=ips, unit="images/s", cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=ips, unit="images/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# --------------------------------------------------------------------- GPU arm --
def max_over_ranks(ms, world, device="cuda"):
    """The slowest rank's time: what a job of `world` independent replicas takes (all-reduce MAX over the process group;
    `device` is where the group's backend wants its tensors: cuda for NCCL, cpu for gloo)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    tm = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tm, op=dist.ReduceOp.MAX)
    return float(tm.item())


def whole_job_value(world, batch, steps, ms):
    """Images per second of the whole job: every rank processed batch * steps images within `ms` (the slowest rank's)."""
    return world * batch * steps / (ms * 1e-3)


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.file,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


# ------------------------------------------------------------ kernel-level arm --
KERNEL_SHAPES = {     # the 3x3 stride-1 layer shapes of the 6n+2 workloads and of WRN-28-10: (N, H, W, C)
    "stage1": (128, 32, 32, 16), "stage2": (128, 16, 16, 32), "stage3": (128, 8, 8, 64),
    "wrn_stage1": (128, 32, 32, 160), "wrn_stage2": (128, 16, 16, 320), "wrn_stage3": (128, 8, 8, 640)}


# The convolution launches as the module-step issues them: on a quarter of the SMs (four modules side by side),
# several image tiles per CTA, with the reductions fused into their epilogues.
STEP_VARIANTS = {
    "fprop_stats": "forward + batch-norm statistics of its output (conv1, conv2 of a block)",
    "dgrad_bn": "data gradient + the sums of the batch-norm backward it feeds (conv2's data gradient)",
    "dgrad_res_bn": "data gradient + gated residual + those sums (the block-input gradient of an identity block)",
    "wgrad_side": "weight gradient with its pixel split capped at 16 CTAs (side stream)",
}


def kernel_bench(B, which="fprop", stage="stage1", launches=64, reps=5, use_graph=True):
    """Average duration of one convolution kernel launch, timed alone: `launches` calls of the operator-level
    entry point, each on its own input/output pair out of a pool larger than the L2 cache (so every launch
    reads HBM), recorded once into a CUDA graph and replayed; CUDA events around the replay on its stream.
    Returns (microseconds per launch, algorithmic bytes per launch, flops per launch)."""
    import torch
    n, h, w, c = KERNEL_SHAPES[stage]
    ops = B.ConvOps(B.FDG_BF16_TC)
    variant = which if which in STEP_VARIANTS else None
    s = B.fdg_conv_shape(n, h, w, c, c, 3, 1, 1)
    elems = n * h * w * c
    pool = max(8, (300 << 20) // (4 * elems) + 1)                 # in + out pairs summing to > 2 x 126 MB
    xs = [torch.randn((n, h, w, c), device="cuda").to(torch.bfloat16) for _ in range(pool)]
    ys = [torch.empty((n, h, w, c), dtype=torch.bfloat16, device="cuda") for _ in range(pool)]
    wt = (torch.randn((c, 3, 3, c), device="cuda") * 0.1).to(torch.bfloat16)
    wf = ops.flip_weights(s, wt)
    need = B.C.c_size_t()
    ops._chk(ops.lib.fdg_conv_wgrad_scratch_bytes(ops.precision, B.C.byref(s), B.C.byref(need)))
    scratch = torch.empty(max(need.value, 16), dtype=torch.uint8, device="cuda")
    dw = torch.empty((c, 3, 3, c), dtype=torch.float32, device="cuda")
    st = torch.cuda.Stream()

    extra = None
    extra_tensors = 0
    if variant:
        ex, keep = ops._extra(s, share=4, wgrad_cta_cap=16 if variant == "wgrad_side" else 0,
                              reduce={"fprop_stats": 1, "dgrad_bn": 2, "dgrad_res_bn": 2, "wgrad_side": 0}[variant],
                              next_mask=xs[0], next_x=xs[0], next_stats=torch.zeros(2 * c, device="cuda") + 1.0, C_red=c)
        extra = B.C.byref(ex)
        extra_tensors = {"fprop_stats": 0, "dgrad_bn": 2, "dgrad_res_bn": 4, "wgrad_side": 0}[variant]

    def call(i):
        x, y = xs[i % pool], ys[i % pool]
        cs = st.cuda_stream
        if variant in ("dgrad_bn", "dgrad_res_bn"):
            ex.next_mask, ex.next_x = xs[(i + 1) % pool].data_ptr(), xs[(i + 2) % pool].data_ptr()
            res = xs[(i + 3) % pool].data_ptr() if variant == "dgrad_res_bn" else None
            msk = xs[(i + 4) % pool].data_ptr() if variant == "dgrad_res_bn" else None
            rc = ops.lib.fdg_conv_dgrad(ops.precision, B.C.byref(s), x.data_ptr(), wt.data_ptr(), wf.data_ptr(), y.data_ptr(),
                                        res, msk, extra, ops.status.data_ptr(), cs)
        elif variant == "fprop_stats":
            rc = ops.lib.fdg_conv_forward(ops.precision, B.C.byref(s), x.data_ptr(), wt.data_ptr(), y.data_ptr(), None,
                                          extra, ops.status.data_ptr(), cs)
        elif variant == "wgrad_side":
            rc = ops.lib.fdg_conv_wgrad(ops.precision, B.C.byref(s), x.data_ptr(), xs[(i + 1) % pool].data_ptr(),
                                        dw.data_ptr(), scratch.data_ptr(), need.value, extra, ops.status.data_ptr(), cs)
        elif which == "fprop":
            rc = ops.lib.fdg_conv_forward(ops.precision, B.C.byref(s), x.data_ptr(), wt.data_ptr(), y.data_ptr(), None,
                                          None, ops.status.data_ptr(), cs)
        elif which == "dgrad":
            rc = ops.lib.fdg_conv_dgrad(ops.precision, B.C.byref(s), x.data_ptr(), wt.data_ptr(), wf.data_ptr(),
                                        y.data_ptr(), None, None, None, ops.status.data_ptr(), cs)
        else:
            rc = ops.lib.fdg_conv_wgrad(ops.precision, B.C.byref(s), x.data_ptr(), xs[(i + 1) % pool].data_ptr(),
                                        dw.data_ptr(), scratch.data_ptr(), need.value, None, ops.status.data_ptr(), cs)
        ops._chk(rc)

    with torch.cuda.stream(st):
        for i in range(pool):                      # ordinary launches first: tensor maps and attributes get set up
            call(i)
        st.synchronize()
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=st):
                for i in range(launches):
                    call(i)
            replay = graph.replay
        else:                                      # plain launches: what a profiler run uses
            def replay():
                for i in range(launches):
                    call(i)
        replay()
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(reps):
            replay()
        e1.record(st)
        st.synchronize()
    assert not ops.timed_out()
    us = e0.elapsed_time(e1) * 1e3 / (reps * launches)
    wbytes = c * 9 * c * (4 if which in ("wgrad", "wgrad_side") else 2)
    return us, (2 + extra_tensors) * elems * 2 + wbytes, 2.0 * n * h * w * c * 9 * c


EW_KERNELS = ["bn_stats", "bn_apply", "bn_apply_res", "bn_bwd_reduce", "bn_bwd_apply", "shrink", "sgd", "ingest", "head"]


def ew_kernel_bench(B, which, stage="stage1", launches=64, reps=5, use_graph=True):
    """The same measurement for a memory-bound kernel of the module-step through its operator-level entry point:
    `launches` calls, each on its own tensors out of a pool that sums to more than twice the L2 cache, recorded
    into a CUDA graph and replayed; CUDA events around the replay.  Returns (microseconds per launch,
    algorithmic bytes per launch: every operand tensor once)."""
    import torch
    n, h, w, c = KERNEL_SHAPES[stage]
    ew = B.EwOps(B.FDG_BF16_TC)
    lib, prec, C = ew.lib, ew.precision, B.C
    elems, rows = n * h * w * c, n * h * w
    tensors_per_call = {"bn_stats": 1, "bn_apply": 2, "bn_apply_res": 3, "bn_bwd_reduce": 3, "bn_bwd_apply": 4, "shrink": 2,
                        "sgd": 0, "ingest": 0, "head": 2}[which]
    fused_sums = 2 * c <= 256           # the layers whose data gradient leaves the sums as per-CTA partial rows
    if which == "bn_bwd_apply" and not fused_sums:
        tensors_per_call = 7            # wider layers: reduce (3 reads) + apply (3 reads, 1 write) in one call
    st = torch.cuda.Stream()
    bf = torch.bfloat16
    if which == "sgd":                       # one module of the headline workload has ~0.5 M parameters; use 8 M for a
        nparam = 8 << 20                     # transfer that is not all launch latency (24 B per parameter + 2 B copy)
        pool = max(4, (300 << 20) // (26 * nparam) + 1)
        bufs = [[torch.randn(nparam, device="cuda") for _ in range(3)] + [torch.empty(nparam, device="cuda"),
                torch.empty(nparam, dtype=bf, device="cuda")] for _ in range(pool)]
        nbytes = 26 * nparam
    elif which == "ingest":
        rows_i = n * h * w
        pool = max(4, (300 << 20) // (rows_i * (12 + 6)) + 1)
        bufs = [[torch.randn((n, h, w, 3), device="cuda"), torch.empty((n, h, w, 3), dtype=bf, device="cuda")] for _ in range(pool)]
        lab = torch.zeros(n, dtype=torch.int32, device="cuda")
        lab2 = torch.zeros(n, dtype=torch.int32, device="cuda")
        nbytes = rows_i * (12 + 6)
    else:
        nt = min(tensors_per_call, 4)
        pool = max(4, (300 << 20) // (2 * elems * nt) + 1)
        bufs = [[torch.randn((n, h, w, c), device="cuda").to(bf) for _ in range(nt)] for _ in range(pool)]
        nbytes = 2 * elems * tensors_per_call
    gam = torch.ones(c, device="cuda")
    bet = torch.zeros(c, device="cuda")
    stats = torch.cat([torch.zeros(c, device="cuda"), torch.ones(c, device="cuda")])
    dg, db = torch.empty(c, device="cuda"), torch.empty(c, device="cuda")
    need = C.c_size_t()
    ew._chk(lib.fdg_bn_scratch_bytes(c, C.byref(need)))
    scratch = torch.zeros(need.value, dtype=torch.uint8, device="cuda")
    if which == "head":
        classes = 10
        wfc, bfc = torch.randn((classes, c), device="cuda") * 0.1, torch.zeros(classes, device="cuda")
        hl = torch.zeros(n, dtype=torch.int32, device="cuda")
        hb = dict(pooled=torch.empty((n, c), device="cuda"), dlogits=torch.empty((n, classes), device="cuda"),
                  loss_n=torch.empty(n, device="cuda"), dw=torch.empty((classes, c), device="cuda"),
                  db=torch.empty(classes, device="cuda"), loss=torch.empty(1, device="cuda"),
                  flags=torch.zeros(4, dtype=torch.int32, device="cuda"))
    P = lambda t: t.data_ptr()

    def call(i):
        t = bufs[i % pool]
        cs = st.cuda_stream
        if which == "bn_stats":
            rc = lib.fdg_bn_stats(prec, P(t[0]), rows, c, 1e-5, P(stats), P(scratch), need.value, cs)
        elif which == "bn_apply":
            rc = lib.fdg_bn_apply(prec, P(t[0]), P(stats), P(gam), P(bet), None, None, None, None, 1, P(t[1]), rows, c, 1e-5,
                                  None, 0, 0, cs)
        elif which == "bn_apply_res":
            rc = lib.fdg_bn_apply(prec, P(t[0]), P(stats), P(gam), P(bet), P(t[2]), None, None, None, 1, P(t[1]), rows, c,
                                  1e-5, None, 0, 0, cs)
        elif which == "bn_bwd_reduce":
            rc = lib.fdg_bn_backward(prec, P(t[0]), P(t[1]), P(t[2]), P(stats), P(gam), None, None, None, None, None, None,
                                     P(dg), P(db), None, None, rows, c, None, 0, 0, P(scratch), need.value, cs)
        elif which == "bn_bwd_apply":      # the sums come as one row of partials, as after a fused data gradient
            rc = lib.fdg_bn_backward(prec, P(t[0]), P(t[1]), P(t[2]), P(stats), P(gam), None, None, None, None, P(t[3]), None,
                                     P(dg), P(db), None, None, rows, c, P(stats) if fused_sums else None, 1 if fused_sums else 0,
                                     148, P(scratch), need.value, cs)
        elif which == "shrink":
            rc = lib.fdg_shrink(prec, P(t[0]), P(t[1]), 0.2, elems, cs)
        elif which == "sgd":
            rc = lib.fdg_sgd_update(P(t[0]), P(t[1]), P(t[2]), P(t[3]), P(t[4]), t[0].numel(), 1e-3, 0.9, 5e-4, cs)
        elif which == "ingest":
            rc = lib.fdg_ingest(prec, P(t[0]), P(t[1]), n * h * w, 3, 3, P(lab), P(lab2), n, cs)
        else:
            rc = lib.fdg_head(prec, P(t[0]), P(wfc), P(bfc), P(hl), n, h * w, c, classes, P(hb["pooled"]), P(hb["dlogits"]),
                              P(hb["loss_n"]), P(t[1]), P(hb["dw"]), P(hb["db"]), P(hb["loss"]), P(hb["flags"]), cs)
        ew._chk(rc)

    with torch.cuda.stream(st):
        for i in range(pool):
            call(i)
        st.synchronize()
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=st):
                for i in range(launches):
                    call(i)
            replay = graph.replay
        else:
            def replay():
                for i in range(launches):
                    call(i)
        replay()
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(reps):
            replay()
        e1.record(st)
        st.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * launches), nbytes


def run_kernel_bench(args):
    from paper_1906_09108_b200 import binding as B
    peaks = measured_peaks()
    out = {}
    if args.kernel_bench == "ew" or args.kernel_bench in EW_KERNELS:
        kinds = EW_KERNELS if args.kernel_bench == "ew" else [args.kernel_bench]
        stages = [args.kernel_stage] if args.kernel_stage else ["stage1", "wrn_stage1"]
        for which in kinds:
            for stage in stages:
                if which in ("sgd",) and stage != stages[0]:
                    continue
                if which == "head" and not args.kernel_stage:      # the classifier sees the last stage's maps
                    if stage != stages[0]:
                        continue
                    stage = "stage3"
                us, nbytes = ew_kernel_bench(B, which, stage, launches=args.kernel_launches,
                                             reps=1 if args.kernel_launches <= 8 else 5, use_graph=args.kernel_launches > 8)
                name = which + ("+reduce" if which == "bn_bwd_apply" and KERNEL_SHAPES[stage][3] > 128 else "")
                out["%s_%s" % (name, "8Mparams" if which == "sgd" else stage)] = dict(
                    us=us, mbytes=nbytes / 1e6, gbs=nbytes / us / 1e3, hbm_frac=nbytes / us / 1e3 / peaks["hbm_gbs"])
        print(json.dumps(dict(kernel_bench=out, peak_source=peaks["source"], hbm_gbs=peaks["hbm_gbs"])))
        return
    if args.kernel_bench == "mma_rate":
        # cycles per tcgen05.mma (M = 128, K = 16) issued back to back by one thread per SM, for N and for the number
        # of accumulators the instructions rotate over (fdg_probe_mma_rate): the two rates the wide kernels are built on
        import torch
        ops = B.ConvOps(B.FDG_BF16_TC)
        cyc = torch.zeros(2, dtype=torch.int64, device="cuda")
        reps = 200
        table = {}
        for unrolled in (1, 0):
            for accs in (1, 3):
                for n in (16, 64, 128, 160, 256):
                    if n * accs > 512:
                        continue
                    ops._chk(ops.lib.fdg_probe_mma_rate(n, accs, reps, unrolled, cyc.data_ptr(), ops.status.data_ptr(),
                                                        torch.cuda.current_stream().cuda_stream))
                    torch.cuda.synchronize()
                    issued, done = (int(v) for v in cyc.cpu())
                    table["%s_N%d_acc%d" % ("straight" if unrolled else "looped", n, accs)] = dict(
                        issue=round(issued / (reps * 4 * accs), 1), complete=round(done / (reps * 4 * accs), 1))
        assert not ops.timed_out()
        print(json.dumps(dict(mma_rate_cycles_per_instruction=table)))
        return
    which_list = {"all": ["fprop", "dgrad", "wgrad"], "step": list(STEP_VARIANTS)}.get(args.kernel_bench, [args.kernel_bench])
    if args.kernel_bench == "step" and not args.kernel_stage:
        args.kernel_stage = "stage1"
    stages = [args.kernel_stage] if args.kernel_stage else list(KERNEL_SHAPES)
    for which in which_list:
        for stage in stages:
            us, nbytes, flops = kernel_bench(B, which, stage, launches=args.kernel_launches,
                                             reps=1 if args.kernel_launches <= 8 else 5, use_graph=args.kernel_launches > 8)
            out["%s_%s" % (which, stage)] = dict(us=us, gbs=nbytes / us / 1e3, tflops=flops / us / 1e6,
                                                 hbm_frac=nbytes / us / 1e3 / peaks["hbm_gbs"],
                                                 tensor_frac=flops / us / 1e6 / peaks["bf16_tflops"])
    print(json.dumps(dict(kernel_bench=out, peak_source=peaks["source"], hbm_gbs=peaks["hbm_gbs"])))


def make_fdg(B, precision, serial, graphs=False):
    import fdg_synth as S
    g = B.FDG(B.make_arch(**ARCH), K=K_MODULES, split_after_block=SPLITS, beta=BETA, lr=LR, momentum=MOM,
              weight_decay=WD, precision=precision, serial=serial, graphs=graphs)
    for k in range(1, K_MODULES + 1):
        g.set_params(k, S.init_params(0, k, g.param_layout(k)))
    return g


def run_gpu(args):
    import torch
    import torch.distributed as dist
    import fdg_synth as S
    from paper_1906_09108_b200 import binding as B

    steps = args.steps if args.steps is not None else 300
    warmup = args.warmup if args.warmup is not None else 20
    warmup = max(warmup, 3)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    precision = B.FDG_BF16_TC if args.precision == "bf16" else B.FDG_FP32_CUDACORE
    b = ARCH["batch"]

    pool_x = [torch.from_numpy(S.images(rank, t, b, ARCH["in_h"], ARCH["in_w"], 3)).cuda() for t in range(1, POOL + 1)]
    pool_y = [torch.from_numpy(S.labels(rank, t, b, ARCH["num_classes"])).cuda() for t in range(1, POOL + 1)]
    host_x = [torch.from_numpy(S.images(rank, t, b, ARCH["in_h"], ARCH["in_w"], 3)).pin_memory() for t in range(1, POOL + 1)]
    host_y = [torch.from_numpy(S.labels(rank, t, b, ARCH["num_classes"])).pin_memory() for t in range(1, POOL + 1)]
    loss_host = torch.zeros(1, dtype=torch.float32).pin_memory()
    loss_dev = torch.zeros(1, dtype=torch.float32, device="cuda")

    g = make_fdg(B, precision, serial=False, graphs=not args.no_graphs)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(n, step_fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for i in range(n):
            step_fn(i)
        g.sync()
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world)

    dev_step = lambda i: g.step(pool_x[i % POOL], pool_y[i % POOL], loss_dev)
    # the clock sampler needs a moment to start: it runs from before the warm-up, so that its samples cover the timed region
    sampler = ClockSampler(local) if rank == 0 else None
    for i in range(2 * K_MODULES + 2 + (0 if args.no_graphs else 8) + warmup):   # pipeline fill (+ graph recording) + warm-up, untimed
        dev_step(i)
    g.sync()
    n0 = g.launch_count()
    ms = timed(steps, dev_step)
    launches = g.launch_count() - n0
    clocks = sampler.stop() if sampler else None
    value = whole_job_value(world, b, steps, ms)

    if args.device_arm_only:
        g.close()
        if rank == 0:
            print(json.dumps(dict(metric=METRIC, value=value, unit="images/s", n_gpus=world, steps=steps, warmup=warmup,
                                  ms_per_step=ms / steps, gpu_launches=int(launches), clocks=clocks,
                                  note="device arm only; not a bench line")))
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # end to end: host buffers through the C ABI, loss read back every step
    def host_step(i):
        g.step_host(host_x[i % POOL], host_y[i % POOL], loss_host)
    for i in range(3):
        host_step(i)
    g.sync()
    ms_e2e = timed(steps, host_step)
    e2e_value = whole_job_value(world, b, steps, ms_e2e)
    h2d = host_x[0].numel() * 4 + host_y[0].numel() * 4
    final_loss = float(loss_host.item())
    g.close()

    line = None
    if rank == 0:
        # dominant kernel class, timed alone on a serial context of the same workload
        peaks = measured_peaks()
        gs = make_fdg(B, precision, serial=True)
        for i in range(2 * K_MODULES + 3):
            gs.step(pool_x[i % POOL], pool_y[i % POOL])
        gs.sync()
        gs.profile_enable(True)
        prof_steps = min(steps, 10)
        for i in range(prof_steps):
            gs.step(pool_x[i % POOL], pool_y[i % POOL])
        stats = [s for s in gs.profile_read() if s["launches"]]
        gs.close()
        total = sum(s["total_ms"] for s in stats)
        top = max(stats, key=lambda s: s["total_ms"])
        sec = top["total_ms"] * 1e-3
        hbm_frac = top["bytes"] / sec / 1e9 / peaks["hbm_gbs"]
        if args.precision == "bf16":
            # Dominant kernel (largest share of device time in an ncu launch list of this workload): the halo-tile
            # convolution.  Timed alone on its most frequent shape; a 16-channel 3x3 layer has 72 flop per byte,
            # far below the machine balance, so HBM is the roofline that bounds it.
            us, nbytes, flops = kernel_bench(B, "fprop", "stage1")
            roof = dict(bound="hbm", achieved=nbytes / us / 1e3, peak=peaks["hbm_gbs"], unit="GB/s",
                        kernel="conv_halo_kernel, 3x3 stride-1 forward, [128,32,32,16] -> 16 channels",
                        avg_us=us, tflops=flops / us / 1e6,
                        how="64 launches on distinct buffers (pool > 2 x L2) replayed from a CUDA graph, CUDA events "
                            "on the replay stream",
                        # dram__bytes_read.sum + dram__bytes_write.sum of one launch of this kernel on this shape,
                        # from the committed ncu summary; null once the kernel's source has changed since
                        traffic=profiled_traffic())
            # The same kernels in the launch shape the module-step issues them in (a quarter of the SMs, four image
            # tiles per CTA, reductions fused into the epilogue), the two batch-norm apply kernels at the stage-1
            # shape, and the wide-layer convolution against the tensor roofline: each timed alone the same way.
            iso = {}
            for kind in STEP_VARIANTS:
                u2, b2, f2 = kernel_bench(B, kind, "stage1")
                iso[kind + "_stage1"] = dict(us=u2, gbs=b2 / u2 / 1e3, frac_hbm=b2 / u2 / 1e3 / peaks["hbm_gbs"])
            for kind in ("bn_apply_res", "bn_bwd_apply"):
                u2, b2 = ew_kernel_bench(B, kind, "stage1")
                iso[kind + "_stage1"] = dict(us=u2, gbs=b2 / u2 / 1e3, frac_hbm=b2 / u2 / 1e3 / peaks["hbm_gbs"])
            u2, b2, f2 = kernel_bench(B, "fprop", "wrn_stage2", launches=16)
            iso["fprop_wrn_stage2"] = dict(us=u2, tflops=f2 / u2 / 1e6, frac_tensor=f2 / u2 / 1e6 / peaks["bf16_tflops"],
                                           kernel="conv3x3_patch_kernel, [128,16,16,320] -> 320 channels")
            u2, b2, f2 = kernel_bench(B, "wgrad", "wrn_stage2", launches=16)
            iso["wgrad_wrn_stage2"] = dict(us=u2, tflops=f2 / u2 / 1e6, frac_tensor=f2 / u2 / 1e6 / peaks["bf16_tflops"],
                                           kernel="wgrad_wide_kernel + wgrad_wide_sum_kernel, x and dy [128,16,16,320]")
            roof["isolated"] = iso
        elif top["name"].startswith("conv"):
            # fp32 FMA peak: 148 SMs x 128 lanes x 2 flop x max SM clock
            alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12
            roof = dict(bound="alu", achieved=top["flops"] / sec / 1e12, peak=alu_peak, unit="TFLOP/s")
        else:
            roof = dict(bound="hbm", achieved=top["bytes"] / sec / 1e9, peak=peaks["hbm_gbs"], unit="GB/s")
        roof.setdefault("kernel", top["name"])
        roof.setdefault("avg_us", top["total_ms"] * 1e3 / top["launches"])
        roof.setdefault("how", "CUDA events around every launch on its stream, serial context, %d steps" % prof_steps)
        roof.setdefault("traffic", None)
        roof.update(frac=roof["achieved"] / roof["peak"], peak_source=peaks["source"],
                    per_class_note="serial context, CUDA events around every launch: includes the host's launch gaps",
                    per_class={s["name"]: dict(ms_per_step=s["total_ms"] / prof_steps, share=s["total_ms"] / total,
                                               gbs=s["bytes"] / (s["total_ms"] * 1e-3) / 1e9,
                                               tflops=s["flops"] / (s["total_ms"] * 1e-3) / 1e12) for s in stats})
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            ips, sec_o, cores = oracle_images_per_s(2, 0)
            cpu = dict(value=ips, unit="images/s", cores=cores, kind="oracle",
                       sample="same network, K and hyper-parameters at batch %d of 128, 2 iterations timed after "
                              "the pipeline fill (2K iterations); numpy float64" % ORACLE_SAMPLE_BATCH)
        line = dict(metric=METRIC, value=value, unit="images/s", n_gpus=world, steps=steps, warmup=warmup,
                    ms_per_step=ms / steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="bf16" if args.precision == "bf16" else "f32", data="synthetic",
                    config=dict(workload=WORKLOAD, K=K_MODULES, splits=list(SPLITS), global_batch=world * b,
                                beta=BETA, lr=LR, precision=args.precision, streams=K_MODULES,
                                cuda_graphs=not args.no_graphs,
                                parallelism="replicas only" if world > 1 else "single GPU",
                                l2="activation FIFO touched per step (>1 GiB) exceeds the 126 MB L2; "
                                   "16 input batches cycled"),
                    clocks=clocks,
                    e2e=dict(value=e2e_value, unit="images/s", h2d_bytes_per_step=h2d, d2h_bytes_per_step=4,
                             ms_per_step=ms_e2e / steps, final_loss=final_loss),
                    gpu_launches=int(launches), roofline=roof, cpu_baseline=cpu)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="fdg", choices=["fdg", "reference"])
    ap.add_argument("--precision", default="bf16", choices=["fp32", "bf16"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graphs", action="store_true")
    ap.add_argument("--workload", default="resnet110_k4", choices=list(WORKLOADS))
    ap.add_argument("--splits", default=None,
                    help="comma-separated block indices after which the modules end, instead of the workload's own")
    ap.add_argument("--kernel-bench", default=None, choices=["fprop", "dgrad", "wgrad", "all", "ew", "step", "mma_rate"] + EW_KERNELS + list(STEP_VARIANTS),
                    help="time the convolution kernels alone through the operator-level C ABI and exit")
    ap.add_argument("--kernel-launches", type=int, default=64,
                    help="launches per replay; 8 or fewer are issued as plain launches (profiler runs)")
    ap.add_argument("--kernel-stage", default=None, choices=list(KERNEL_SHAPES))
    ap.add_argument("--device-arm-only", action="store_true",
                    help="time the device-resident arm only (no end-to-end arm, no per-kernel roofline, no CPU "
                         "baseline): the short run the ncu launch list is taken from")
    args = ap.parse_args()
    select_workload(args.workload)
    if args.splits:
        global SPLITS
        SPLITS = tuple(int(v) for v in args.splits.split(","))
        assert len(SPLITS) == K_MODULES - 1
    if args.kernel_bench:
        run_kernel_bench(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
