#!/usr/bin/env python
"""Benchmark of the inverse-convolution hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                    [--no-per-config] [--table] [--sweep]

A step is one `invconv_forward` call plus one `invconv_backward` call (grad_y
and grad_w) on one batch of the headline workload (default: `wide48_k5`, the
heaviest benchmark shape); the metric is images per second through forward +
backward.  Inputs are resident in HBM for `value`; `e2e` runs the same step
through `invconv_step_host` from pinned host buffers with the copies inside the
timed region.  Rank 0 prints ONE JSON line; its `per_config` list carries all
ten benchmark shapes (L2-cold and L2-warm times, the three bounds, the binding
one and the fraction reached, the masked convolution).

Multi-GPU (one rank per GPU, launched by torchrun or spawned by `--gpus N`):
the batch axis is sharded -- every rank runs the layer on its own batch of the
workload's size (weak scaling) and grad_w, the only sum over the batch, is
all-reduced with NCCL inside every timed step; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel, one launch, from the ncu captures
# summarised under profiles/ (per workload; None where no capture exists)
NCU_TRAFFIC_BYTES = {"mnist": 1.655e6, "wide48_k5": 3.65e6 + 6.34e6}   # wide48_k5: transposed solve + grad_w (profiles/tensor_wavefront_wide48_k5.md)

METRIC = "invconv_fwd_bwd_images_per_sec"
UNIT = "images/s"
L2_BYTES = 126 * 1024 * 1024
TF32_OVER_BF16 = 1.1 / 2.25          # nominal dense peaks, tf32 : bf16
FFMA_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "kind": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "kind": "fallback"}


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs (read-only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def sample(self):
        if self.nv is None:
            return
        try:
            self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
            try:
                r = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _loop(self):
        while not self._stop.is_set():
            self.sample()
            self._stop.wait(0.01)

    def __enter__(self):
        self.sample()
        self._thread = threading.Thread(target=self._loop, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thread.join()
        self.sample()

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# --------------------------------------------------------------------------- bounds

PATH_NAMES = {1: "generic", 2: "warp", 3: "team", 4: "tensor"}


def bounds(shape, path, cluster, t_step_cycles, sm_mhz, pk):
    """Per-call lower bounds of forward + backward, in microseconds, and which one binds.

    t_hbm: algorithmic bytes over the measured copy bandwidth.  t_cp: 2(H+W-1) dependent steps times the
    measured latency of one step of the mechanism the shape forces (warp shuffle; shared memory + block
    barrier; cluster shared memory + cluster barrier where one SM cannot hold the kernel).  t_alu: flops on
    the fp32 FMA pipe.  t_tensor (tensor-core family only): the solves cost two tensor-core passes per
    product (tf32 + one bf16 pass of twice the depth holding both correction terms = 2 tf32-equivalent
    passes), grad_w one tf32 pass, against tf32 peak = measured bf16 peak x the nominal tf32:bf16 ratio.
    The binding bound is the largest of t_hbm, t_cp and the bound of the arithmetic pipe actually used."""
    E = shape.elements
    w_bytes = 4 * shape.C * shape.C * shape.k * shape.k
    algo_bytes = 20 * E + 3 * w_bytes                  # fwd: y in, x out; bwd: grad_x, x in, grad_y out; w twice in, grad_w out
    t_hbm = algo_bytes / (pk["hbm_gbs"] * 1e3)
    flops = 6.0 * E * shape.C * shape.k * shape.k
    t_alu = flops / (FFMA_TFLOPS * 1e12) * 1e6         # fp32 FMA pipe: 148 SMs x 128 lanes x 2 flop at the maximum SM clock
    clk = (sm_mhz or 1965) * 1e6
    mech = 0 if path == 2 else (2 if cluster > 1 else 1)
    t_cp = 2 * shape.n_diagonals * t_step_cycles[mech] / clk * 1e6
    out = {"t_hbm_us": t_hbm, "t_alu_us": t_alu, "t_cp_us": t_cp, "t_step_cycles": t_step_cycles[mech],
           "step_mechanism": ("shuffle", "smem+barrier", "cluster smem+barrier")[mech],
           "algo_bytes": algo_bytes, "flops": flops}
    cands = [("hbm", t_hbm), ("critical_path", t_cp)]
    if path == 4:
        tf32 = pk["bf16_tflops"] * TF32_OVER_BF16 * 1e12
        out["t_tensor_us"] = (2 * (2.0 / 3.0) * flops + (1.0 / 3.0) * flops) / tf32 * 1e6
        cands.append(("tensor", out["t_tensor_us"]))
    else:
        cands.append(("alu", t_alu))
    name, t = max(cands, key=lambda kv: kv[1])
    out["binding"], out["t_roofline_us"] = name, t
    return out


# --------------------------------------------------------------------------- our arm

class DeviceStep:
    """Rotating sets of device buffers for one workload (larger than twice the L2 in total unless `warm`),
    and the CUDA graphs that replay forward / backward / both over them."""

    def __init__(self, shape, w, y, gx, device, warm=False, storage="f32"):
        import torch
        from paper_2410_14634_b200 import binding
        self.torch, self.b, self.shape, self.device = torch, binding, shape, device
        self.narrow = storage == "bf16"          # activations held as bfloat16 (the storage variant's calls)
        per_set = 4 * (2 if self.narrow else 4) * shape.elements
        self.nsets = 1 if warm else max(3, -(-2 * L2_BYTES // per_set) + 1)
        yd = torch.from_numpy(y).to(device)
        gxd = torch.from_numpy(gx).to(device)
        if self.narrow:
            yd, gxd = yd.to(torch.bfloat16), gxd.to(torch.bfloat16)
        self.w = torch.from_numpy(w).to(device)
        self.y = [yd.clone() for _ in range(self.nsets)]
        self.gx = [gxd.clone() for _ in range(self.nsets)]
        self.x = [torch.empty_like(yd) for _ in range(self.nsets)]
        self.gy = [torch.empty_like(yd) for _ in range(self.nsets)]
        self.gw = torch.empty_like(self.w)
        self.cursor = 0
        self.stream = torch.cuda.Stream(device)
        # make sure x holds valid data in every set (backward-only graphs read it)
        with torch.cuda.stream(self.stream):
            for i in range(self.nsets):
                self.fwd(i)
            if not self.narrow:
                binding.masked_conv_forward(self.x[0], self.w, out=self.gy[0])     # first call outside any graph capture
        self.stream.synchronize()

    def fwd(self, i):
        if self.narrow:
            self.b.invconv_forward_bf16(self.y[i], self.w, out=self.x[i])
        else:
            self.b.invconv_forward(self.y[i], self.w, out=self.x[i])

    def conv(self, i):
        self.b.masked_conv_forward(self.x[i], self.w, out=self.gy[i])

    def bwd(self, i):
        if self.narrow:
            _, gw = self.b.invconv_backward_bf16(self.gx[i], self.x[i], self.w, out_grad_y=self.gy[i], out_grad_w=self.gw)
        else:
            self.b.invconv_backward(self.gx[i], self.x[i], self.w, out_grad_y=self.gy[i], out_grad_w=self.gw)

    def graph(self, what: str, nsteps: int):
        """Capture `nsteps` steps (walking the buffer sets) into one CUDA graph."""
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        before = self.b.invconv_kernel_launch_count()
        with torch.cuda.graph(g, stream=self.stream):
            for s in range(nsteps):
                i = (self.cursor + s) % self.nsets
                if what in ("fwd", "both"):
                    self.fwd(i)
                if what in ("bwd", "both"):
                    self.bwd(i)
                if what == "conv":
                    self.conv(i)
        launches = self.b.invconv_kernel_launch_count() - before
        self.cursor = (self.cursor + nsteps) % self.nsets
        return g, launches

    def time_graphs(self, what: str, steps: int, warmup: int, barrier=None, sampler=None):
        """Device time (ms) of exactly `steps` steps after `warmup` untimed ones, on this object's stream."""
        torch = self.torch
        chunk = min(steps, 128)
        g_main, l_main = self.graph(what, chunk)
        rem = steps % chunk
        g_rem, l_rem = self.graph(what, rem) if rem else (None, 0)
        g_warm, _ = self.graph(what, min(max(warmup, 1), 128))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            for _ in range(-(-max(warmup, 1) // min(max(warmup, 1), 128))):
                g_warm.replay()
        self.stream.synchronize()
        if barrier:
            barrier()
        torch.cuda.synchronize(self.device)
        ctx = sampler if sampler is not None else _Null()
        with ctx:
            with torch.cuda.stream(self.stream):
                e0.record(self.stream)
                for _ in range(steps // chunk):
                    g_main.replay()
                if g_rem is not None:
                    g_rem.replay()
                e1.record(self.stream)
            self.stream.synchronize()
        if barrier:
            barrier()
        torch.cuda.synchronize(self.device)
        launches = (steps // chunk) * l_main + l_rem
        return e0.elapsed_time(e1), launches

    def time_data_parallel(self, steps: int, warmup: int, barrier, sampler):
        """Several ranks: forward, backward and the NCCL all-reduce of grad_w per step, launched eagerly on this
        object's stream (the collective is part of the step); device time (ms) of exactly `steps` steps."""
        torch = self.torch
        from paper_2410_14634_b200 import sharding
        before = self.b.invconv_kernel_launch_count()

        def one(i):
            self.fwd(i)
            self.bwd(i)
            sharding.allreduce_grad_w(self.gw)

        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            for s in range(max(warmup, 1)):
                one(s % self.nsets)
            self.stream.synchronize()
            barrier()
            torch.cuda.synchronize(self.device)
            before = self.b.invconv_kernel_launch_count()
            with sampler:
                e0.record(self.stream)
                for s in range(steps):
                    one((warmup + s) % self.nsets)
                e1.record(self.stream)
                self.stream.synchronize()
            barrier()
            torch.cuda.synchronize(self.device)
        return e0.elapsed_time(e1), self.b.invconv_kernel_launch_count() - before


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def time_e2e(shape, w, y, gx, device, steps, warmup):
    """The step through `invconv_step_host` from pinned host buffers, copies inside the timed region.  Two
    independent sets of host buffers and device scratch alternate on two streams, as an input pipeline would
    run it, so that one step's copies out overlap the next step's copies in; every step still moves all of
    its own bytes.  Also times the same copies alone (no kernels): the floor the host link sets."""
    import torch
    from paper_2410_14634_b200 import binding
    hss = [binding.HostStep(shape.B, shape.C, shape.H, shape.W, shape.k, device) for _ in range(2)]
    for hs in hss:
        hs.y.copy_(torch.from_numpy(y)); hs.w.copy_(torch.from_numpy(w)); hs.grad_x.copy_(torch.from_numpy(gx))
    sts = [torch.cuda.Stream(device) for _ in range(2)]

    def run(fn, n):
        e0, e1, ej = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(sts[0])
        sts[1].wait_event(e0)
        for i in range(n):
            fn(i & 1)
        ej.record(sts[1])
        sts[0].wait_event(ej)
        e1.record(sts[0])
        for st in sts:
            st.synchronize()
        return e0.elapsed_time(e1)

    step = lambda j: hss[j].run(sts[j])
    for i in range(warmup):
        step(i & 1)
    for st in sts:
        st.synchronize()
    ms = run(step, steps)

    # the same bytes with plain copies only
    dev = [[torch.empty_like(t, device=device) for t in (hs.y, hs.grad_x, hs.w)] for hs in hss]

    def copies(j):
        hs = hss[j]
        with torch.cuda.stream(sts[j]):
            for d, h in zip(dev[j], (hs.y, hs.grad_x, hs.w)):
                d.copy_(h, non_blocking=True)
            hs.x.copy_(dev[j][0], non_blocking=True)
            hs.grad_y.copy_(dev[j][1], non_blocking=True)
            hs.grad_w.copy_(dev[j][2], non_blocking=True)

    for i in range(4):
        copies(i & 1)
    for st in sts:
        st.synchronize()
    ms_copy = run(copies, steps)
    return ms, ms_copy, hss[0]


def _oracle_shard(args):
    name, start, count = args
    from oracle import api as oracle
    from paper_2410_14634_b200 import workloads
    _, w, y, gx = workloads.make(name, batch=start + count)
    y, gx = y[start:start + count], gx[start:start + count]
    t0 = time.perf_counter()
    x = oracle.invconv_forward(y, w)
    oracle.invconv_backward(gx, x, w)
    return time.perf_counter() - t0


def cpu_baseline(shape_name, budget_s=10.0):
    """The float64 oracle, as it stands, on the host cores, on a bounded sample of the workload: one core, then
    one process per core over shards of the batch (images are independent; grad_w partial sums would be added)."""
    import multiprocessing as mp
    from oracle import api as oracle
    from paper_2410_14634_b200 import workloads
    shape = workloads.BY_NAME[shape_name]
    # size the sample from a one-image probe so that the whole leg stays near the budget
    s1, w, y, gx = workloads.make(shape_name, batch=1)
    t0 = time.perf_counter()
    x = oracle.invconv_forward(y, w)
    oracle.invconv_backward(gx, x, w)
    per_image = max(time.perf_counter() - t0, 1e-7)
    nb = int(max(1, min(shape.B, budget_s / 2 / per_image)))
    s, w, y, gx = workloads.make(shape_name, batch=nb)
    best = float("inf")
    for _ in range(2):
        t0 = time.perf_counter()
        x = oracle.invconv_forward(y, w)
        oracle.invconv_backward(gx, x, w)
        best = min(best, time.perf_counter() - t0)
    one_core = nb / best
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        cores = os.cpu_count() or 1
    out = {"value": one_core, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{nb} of {shape.B} images of '{shape_name}', fwd+bwd, float64, best of 2",
           "one_core_images_per_s": one_core, "host_cores": cores}
    if cores > 1:
        per = max(1, min(shape.B // cores if shape.B >= cores else 1, int(budget_s / 2 / per_image) or 1))
        jobs = [(shape_name, r * per, per) for r in range(cores)]
        try:
            with mp.get_context("fork").Pool(cores) as pool:
                pool.map(_oracle_shard, [(shape_name, 0, 1)] * cores)          # start the workers, load the library
                t0 = time.perf_counter()
                pool.map(_oracle_shard, jobs)
                dt = time.perf_counter() - t0
            out.update({"value": cores * per / dt, "cores": cores, "all_cores_images_per_s": cores * per / dt,
                        "sample": out["sample"] + f"; all cores: {cores} processes x {per} images, wall clock"})
        except Exception as e:                                                  # report the one-core figure alone
            out["all_cores_error"] = repr(e)
    return out


def run_reference(args, rank):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if rank != 0:
        return
    from oracle import api as oracle
    from paper_2410_14634_b200 import workloads
    shape = workloads.BY_NAME[args.workload]
    s1, w, y, gx = workloads.make(args.workload, batch=1)
    t0 = time.perf_counter()
    x = oracle.invconv_forward(y, w); oracle.invconv_backward(gx, x, w)
    per_image = max(time.perf_counter() - t0, 1e-7)
    total_steps = args.steps + args.warmup
    nb = int(max(1, min(shape.B, 120.0 / total_steps / per_image)))
    s, w, y, gx = workloads.make(args.workload, batch=nb)
    for _ in range(args.warmup):
        x = oracle.invconv_forward(y, w); oracle.invconv_backward(gx, x, w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        x = oracle.invconv_forward(y, w); oracle.invconv_backward(gx, x, w)
    dt = time.perf_counter() - t0
    value = nb * args.steps / dt
    sample = f"{nb} of {shape.B} images of '{args.workload}' per step, fwd+bwd, float64 C oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "B": shape.B, "C": shape.C, "H": shape.H, "W": shape.W, "k": shape.k},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def probe_steps(binding, device):
    return {m: binding.invconv_probe_step_latency(m, 4096, device) for m in (0, 1, 2)}


def per_config_rows(binding, workloads, device, pk, t_step, sm_mhz, steps, warmup):
    """All ten benchmark shapes on one GPU: microseconds per call (L2-cold rotating buffers and L2-warm), images
    per second, the bounds and the fraction of the binding one, and the masked convolution."""
    import torch
    rows = []
    for shape in workloads.SHAPES:
        _, w, y, gx = workloads.make(shape.name)
        path = binding.invconv_path_for(shape.B, shape.C, shape.H, shape.W, shape.k)
        cluster = binding.invconv_cluster_size_for(shape.B, shape.C, shape.H, shape.W, shape.k)
        ds = DeviceStep(shape, w, y, gx, device)
        ms_f, _ = ds.time_graphs("fwd", steps, warmup)
        ms_b, _ = ds.time_graphs("bwd", steps, warmup)
        ms_c, _ = ds.time_graphs("conv", steps, warmup)
        del ds
        dw = DeviceStep(shape, w, y, gx, device, warm=True)
        ms_fw, _ = dw.time_graphs("fwd", steps, warmup)
        ms_bw, _ = dw.time_graphs("bwd", steps, warmup)
        del dw
        torch.cuda.empty_cache()
        tf, tb, tc = ms_f / steps * 1e3, ms_b / steps * 1e3, ms_c / steps * 1e3
        bd = bounds(shape, path, cluster, t_step, sm_mhz, pk)
        row = {"workload": shape.name, "B": shape.B, "C": shape.C, "H": shape.H, "W": shape.W, "k": shape.k,
               "path": PATH_NAMES.get(path, str(path)), "cluster": cluster,
               "t_fwd_us": round(tf, 2), "t_bwd_us": round(tb, 2),
               "t_fwd_warm_us": round(ms_fw / steps * 1e3, 2), "t_bwd_warm_us": round(ms_bw / steps * 1e3, 2),
               "images_per_s": round(shape.B / ((tf + tb) * 1e-6)),
               "t_hbm_us": round(bd["t_hbm_us"], 3), "t_alu_us": round(bd["t_alu_us"], 3),
               "t_cp_us": round(bd["t_cp_us"], 3), "binding": bd["binding"],
               "frac": round(bd["t_roofline_us"] / (tf + tb), 4),
               "frac_of_ffma_bound": round(bd["t_alu_us"] / (tf + tb), 4),
               "t_masked_conv_us": round(tc, 2),
               "masked_conv_hbm_frac": round(8.0 * shape.elements / (tc * 1e-6) / 1e9 / pk["hbm_gbs"], 4)}
        if "t_tensor_us" in bd:
            row["t_tensor_us"] = round(bd["t_tensor_us"], 3)
        dims = (shape.B, shape.C, shape.H, shape.W, shape.k)
        if binding.invconv_bf16_in_kernel(*dims, backward=False):
            # the storage variant where the wavefront kernel itself reads and writes bfloat16 (half the activation bytes)
            d16 = DeviceStep(shape, w, y, gx, device, storage="bf16")
            ms_f16, _ = d16.time_graphs("fwd", steps, warmup)
            ms_b16, _ = d16.time_graphs("bwd", steps, warmup)
            del d16
            torch.cuda.empty_cache()
            row["bf16_storage"] = {"t_fwd_us": round(ms_f16 / steps * 1e3, 2), "t_bwd_us": round(ms_b16 / steps * 1e3, 2),
                                   "t_hbm_us": round(bd["t_hbm_us"] / 2, 3),
                                   "backward_in_kernel": bool(binding.invconv_bf16_in_kernel(*dims, backward=True))}
        rows.append(row)
    return rows


def run_ours(args, rank, world):
    import torch
    from paper_2410_14634_b200 import binding, workloads, sharding
    binding.lib()                                            # no fallback: fail here if the library is missing
    local = int(os.environ.get("LOCAL_RANK", "0"))
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    dist = None
    if world > 1 or args.collective:
        import torch.distributed as dist
        if not dist.is_initialized():
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29533")
            os.environ.setdefault("RANK", "0")
            os.environ.setdefault("WORLD_SIZE", "1")
            dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()

    shape, w, y, gx = workloads.make(args.workload)
    pk = peaks()
    ds = DeviceStep(shape, w, y, gx, device)
    sampler = ClockSampler(local)
    if dist is not None:
        ms, launches = ds.time_data_parallel(args.steps, args.warmup, barrier, sampler)
        launch_mode = "eager launches; NCCL all-reduce of grad_w inside every step"
    else:
        ms, launches = ds.time_graphs("both", args.steps, args.warmup, barrier=barrier, sampler=sampler)
        launch_mode = "CUDA graphs of <=128 steps replayed on one stream"
    ms = sharding.max_over_ranks(ms, device)
    value = world * shape.B * args.steps / (ms * 1e-3)
    assert binding.invconv_get_status(device=device) == 0

    # end to end from pinned host memory: every rank runs it at the same time, the slowest rank counts
    e2e_steps = max(2, min(args.steps, 100))
    barrier()
    ms_e, ms_copy, hs = time_e2e(shape, w, y, gx, device, e2e_steps, min(max(args.warmup, 3), 10))
    ms_e = sharding.max_over_ranks(ms_e, device)

    out = None
    if rank == 0:
        clocks = sampler.summary()
        # per-kernel durations over the same rotating buffers
        ksteps = max(3, min(args.steps, 500))
        ms_f, lf = ds.time_graphs("fwd", ksteps, min(args.warmup, 20))
        ms_b, lb = ds.time_graphs("bwd", ksteps, min(args.warmup, 20))
        t_fwd_us, t_bwd_us = ms_f / ksteps * 1e3, ms_b / ksteps * 1e3
        t_step = probe_steps(binding, device)
        path = binding.invconv_path_for(shape.B, shape.C, shape.H, shape.W, shape.k)
        cluster = binding.invconv_cluster_size_for(shape.B, shape.C, shape.H, shape.W, shape.k)
        bd = bounds(shape, path, cluster, t_step, clocks["sm_max_mhz"], pk)
        E = shape.elements
        wb = 4 * shape.C * shape.C * shape.k * shape.k
        # dominant launch group = the backward call (grad_y solve + grad_w correlation)
        if path == 4 or bd["t_alu_us"] > bd["t_hbm_us"]:          # a dense contraction: judged on its arithmetic pipe
            dom_flops = 4.0 * E * shape.C * shape.k * shape.k
            achieved = dom_flops / (t_bwd_us * 1e-6) / 1e12
            peak = pk["bf16_tflops"] * TF32_OVER_BF16 if path == 4 else FFMA_TFLOPS
            roof = {"bound": "tensor" if path == 4 else "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                    "kernel": "backward call (grad_y solve + grad_w correlation)",
                    "algorithmic_flops_per_launch": dom_flops,
                    "peak_kind": (f"tf32 = {pk['kind']} bf16 burst x nominal 1.1/2.25" if path == 4
                                  else "fp32 FMA pipe, 148 SMs x 128 lanes x 2 x 1.965 GHz (derived)"),
                    "achieved_over_ffma_peak": achieved / FFMA_TFLOPS,
                    "note": f"the binding bound of this shape is {bd['binding']} (see north_star_roofline)"}
        else:
            dom_bytes = 12 * E + 2 * wb
            achieved = dom_bytes / (t_bwd_us * 1e-6) / 1e9
            roof = {"bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / pk["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                    "kernel": "backward call (grad_y + grad_w)", "algorithmic_bytes_per_launch": dom_bytes,
                    "peak_kind": f"of {pk['kind']}",
                    "note": f"the binding bound of this shape is {bd['binding']} (see north_star_roofline)"}
        cpu = cpu_baseline(args.workload)
        rows = [] if args.no_per_config else per_config_rows(binding, workloads, device, pk, t_step,
                                                             clocks["sm_max_mhz"], args.per_config_steps, 5)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "B": shape.B, "C": shape.C, "H": shape.H, "W": shape.W,
                       "k": shape.k, "per_rank_batch": shape.B,
                       "parallelism": f"batch sharded over {world} rank(s)" + (", grad_w all-reduced (NCCL)" if dist is not None else ""),
                       "l2": f"rotating {ds.nsets} buffer sets ({ds.nsets * 16 * E / 2**20:.0f} MiB > 2x L2)",
                       "launch": launch_mode, "kernel_path": PATH_NAMES.get(path, str(path)), "cluster": cluster},
            "us_per_layer": {"forward": t_fwd_us, "backward": t_bwd_us, "sum": t_fwd_us + t_bwd_us},
            "roofline": roof,
            "north_star_roofline": {**{k: bd[k] for k in bd if k not in ("algo_bytes", "flops")},
                                    "t_achieved_us": t_fwd_us + t_bwd_us,
                                    "frac": bd["t_roofline_us"] / (t_fwd_us + t_bwd_us),
                                    "frac_of_ffma_bound": bd["t_alu_us"] / (t_fwd_us + t_bwd_us)},
            "cpu_baseline": cpu,
            "e2e": {"value": world * shape.B * e2e_steps / (ms_e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": hs.h2d_bytes, "d2h_bytes_per_step": hs.d2h_bytes,
                    "ms_per_step": ms_e / e2e_steps, "steps": e2e_steps,
                    "copies_only_ms_per_step": ms_copy / e2e_steps,
                    "pipeline": "two host-buffer sets alternating on two streams"},
            "gpu_launches": launches,
            "clocks": clocks,
            "per_config": rows,
        }
    barrier()
    if dist is not None:
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out))


def run_table(args):
    """Every benchmark shape on one GPU, one JSON object per shape (human-readable form of `per_config`)."""
    import torch
    from paper_2410_14634_b200 import binding, workloads
    device = torch.device("cuda:0")
    pk = peaks()
    t_step = probe_steps(binding, device)
    for r in per_config_rows(binding, workloads, device, pk, t_step, 1965, args.steps, args.warmup):
        print(json.dumps(r))


def run_sweep(args):
    """The paper's ablation axes at three channels (kernel size, image side, batch size): microseconds per call,
    and per diagonal, against the O(m k^2) model of Table 1 (human-readable, one JSON object per shape)."""
    import torch
    from paper_2410_14634_b200 import binding, workloads
    device = torch.device("cuda:0")
    cases = [("k", 32, 3, 32, k) for k in (2, 3, 5, 7, 9, 11)]
    cases += [("side", 32, 3, m, 3) for m in (16, 32, 64, 128, 256)]
    cases += [("batch", b, 3, 32, 3) for b in (1, 4, 16, 64, 128, 256)]
    for axis, Bn, C, m, k in cases:
        w, y, gx = workloads.make_custom(900 + Bn + m + k, Bn, C, m, m, k, sigma=0.02)
        shape = workloads.Shape(f"sweep_{axis}_B{Bn}_m{m}_k{k}", 0, Bn, C, m, m, k, 0.02, 0.8, 1.2, 0)
        ds = DeviceStep(shape, w, y, gx, device)
        path = binding.invconv_path_for(Bn, C, m, m, k)
        steps = max(3, min(args.steps, 200 if path != binding.PATH_GENERIC else 10))
        ms_f, _ = ds.time_graphs("fwd", steps, min(args.warmup, 5))
        ms_b, _ = ds.time_graphs("bwd", steps, min(args.warmup, 5))
        tf, tb = ms_f / steps * 1e3, ms_b / steps * 1e3
        print(json.dumps({"axis": axis, "B": Bn, "C": C, "side": m, "k": k, "path": path, "t_fwd_us": round(tf, 2),
                          "t_bwd_us": round(tb, 2), "fwd_ns_per_diagonal": round(tf * 1e3 / (2 * m - 1), 1),
                          "images_per_s": round(Bn / ((tf + tb) * 1e-6))}), flush=True)
        del ds
        torch.cuda.empty_cache()


def spawn_ranks(args):
    """`--gpus N` without a launcher: start the N ranks (one per GPU) with torch.distributed.run."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 400), os.path.abspath(__file__)]
    cmd += [a for a in sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="wide48_k5")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-config", action="store_true", help="skip the per-shape list (headline workload only)")
    ap.add_argument("--per-config-steps", type=int, default=50, help="timed calls per shape of the per_config list")
    ap.add_argument("--collective", action="store_true",
                    help="run the data-parallel step (NCCL all-reduce of grad_w) even on one rank")
    ap.add_argument("--table", action="store_true", help="time every benchmark shape on one GPU")
    ap.add_argument("--sweep", action="store_true", help="time the ablation axes (kernel size, image side, batch) at C=3")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1 and not (args.table or args.sweep):
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(world_env or "1")
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.table:
        run_table(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    run_ours(args, rank, world)


if __name__ == "__main__":
    main()
