#!/usr/bin/env python
"""Benchmark of the inverse-convolution hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference] [--table]

A step is one `invconv_forward` call plus one `invconv_backward` call (grad_y
and grad_w) on one batch of the named workload; the metric is images per second
through forward + backward.  Inputs are resident in HBM for `value`; `e2e` runs
the same step through `invconv_step_host` from pinned host buffers with the
copies inside the timed region.  Rank 0 prints ONE JSON line.

Multi-GPU (`torchrun`, one rank per GPU): images are independent, so every rank
runs the layer on its own batch (replicas, weak scaling, no data-path
collective); time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum of the dominant (backward) kernel, one launch, from the ncu
# capture summarised in profiles/ (per workload; None where no capture exists)
NCU_TRAFFIC_BYTES = {"mnist": 1.655e6, "wide48_k3": None}

METRIC = "invconv_fwd_bwd_images_per_sec"
UNIT = "images/s"
L2_BYTES = 126 * 1024 * 1024


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


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

def bounds(shape, t_step_cycles, sm_mhz, hbm_gbs):
    """The three per-call lower bounds of forward + backward, in microseconds."""
    E = shape.elements
    w_bytes = 4 * shape.C * shape.C * shape.k * shape.k
    algo_bytes = 20 * E + 3 * w_bytes                  # fwd: y in, x out; bwd: grad_x, x in, grad_y out; w twice in, grad_w out
    t_hbm = algo_bytes / (hbm_gbs * 1e3)
    flops = 6.0 * E * shape.C * shape.k * shape.k
    t_alu = flops / (148 * 128 * 2 * 1.965e9) * 1e6    # fp32 FMA pipe: 148 SMs x 128 lanes x 2 flop at the maximum SM clock
    clk = (sm_mhz or 1965) * 1e6
    t_cp = 2 * shape.n_diagonals * t_step_cycles / clk * 1e6
    return {"t_hbm_us": t_hbm, "t_alu_us": t_alu, "t_cp_us": t_cp, "algo_bytes": algo_bytes, "flops": flops}


# --------------------------------------------------------------------------- our arm

class DeviceStep:
    """Rotating sets of device buffers for one workload, larger than twice the L2 in total, and the
    CUDA graphs that replay forward / backward / both over them."""

    def __init__(self, shape, w, y, gx, device):
        import torch
        from paper_2410_14634_b200 import binding
        self.torch, self.b, self.shape, self.device = torch, binding, shape, device
        per_set = 4 * 4 * shape.elements
        self.nsets = max(3, -(-2 * L2_BYTES // per_set) + 1)
        yd = torch.from_numpy(y).to(device)
        gxd = torch.from_numpy(gx).to(device)
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
                binding.invconv_forward(self.y[i], self.w, out=self.x[i])
        self.stream.synchronize()

    def fwd(self, i):
        self.b.invconv_forward(self.y[i], self.w, out=self.x[i])

    def conv(self, i):
        self.b.masked_conv_forward(self.x[i], self.w, out=self.gy[i])

    def bwd(self, i):
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


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def time_e2e(shape, w, y, gx, device, steps, warmup):
    """The step through `invconv_step_host` from pinned host buffers, copies inside the timed region.  Two
    independent sets of host buffers and device scratch alternate on two streams, as an input pipeline would
    run it, so that one step's copies out overlap the next step's copies in; every step still moves all of
    its own bytes."""
    import torch
    from paper_2410_14634_b200 import binding
    hss = [binding.HostStep(shape.B, shape.C, shape.H, shape.W, shape.k, device) for _ in range(2)]
    for hs in hss:
        hs.y.copy_(torch.from_numpy(y)); hs.w.copy_(torch.from_numpy(w)); hs.grad_x.copy_(torch.from_numpy(gx))
    sts = [torch.cuda.Stream(device) for _ in range(2)]
    for i in range(warmup):
        hss[i & 1].run(sts[i & 1])
    for st in sts:
        st.synchronize()
    e0, e1, ej = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    e0.record(sts[0])
    sts[1].wait_event(e0)
    for i in range(steps):
        hss[i & 1].run(sts[i & 1])
    ej.record(sts[1])
    sts[0].wait_event(ej)
    e1.record(sts[0])
    for st in sts:
        st.synchronize()
    return e0.elapsed_time(e1), hss[0]


def cpu_baseline(shape_name, budget_s=12.0):
    """The float64 oracle, as it stands, on one host core, on a bounded sample of the workload."""
    from oracle import api as oracle
    from paper_2410_14634_b200 import workloads
    shape = workloads.BY_NAME[shape_name]
    # size the sample from a one-image probe so that the whole leg stays near the budget
    s1, w, y, gx = workloads.make(shape_name, batch=1)
    t0 = time.perf_counter()
    x = oracle.invconv_forward(y, w)
    oracle.invconv_backward(gx, x, w)
    per_image = max(time.perf_counter() - t0, 1e-7)
    nb = int(max(1, min(shape.B, budget_s / 3 / per_image)))
    s, w, y, gx = workloads.make(shape_name, batch=nb)
    best = float("inf")
    for _ in range(3):
        t0 = time.perf_counter()
        x = oracle.invconv_forward(y, w)
        oracle.invconv_backward(gx, x, w)
        best = min(best, time.perf_counter() - t0)
    return {"value": nb / best, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{nb} of {shape.B} images of '{shape_name}', fwd+bwd, float64, best of 3",
            "ms_per_step_full_batch": best / nb * shape.B * 1e3}


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


def run_ours(args, rank, world):
    import torch
    from paper_2410_14634_b200 import binding, workloads
    binding.lib()                                            # no fallback: fail here if the library is missing
    local = int(os.environ.get("LOCAL_RANK", "0"))
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()

    shape, w, y, gx = workloads.make(args.workload)
    hbm_gbs, peak_kind = peaks()
    ds = DeviceStep(shape, w, y, gx, device)
    sampler = ClockSampler(local)
    ms, launches = ds.time_graphs("both", args.steps, args.warmup, barrier=barrier, sampler=sampler)
    from paper_2410_14634_b200 import sharding
    ms = sharding.max_over_ranks(ms, device)
    value = world * shape.B * args.steps / (ms * 1e-3)
    assert binding.invconv_get_status(device=device) == 0

    # end to end from pinned host memory: every rank runs it at the same time, the slowest rank counts
    e2e_steps = max(2, min(args.steps, 200))
    barrier()
    ms_e, hs = time_e2e(shape, w, y, gx, device, e2e_steps, min(max(args.warmup, 3), 20))
    ms_e = sharding.max_over_ranks(ms_e, device)

    out = None
    if rank == 0:
        # per-kernel durations over the same rotating buffers
        ksteps = min(args.steps, 2000)
        ms_f, lf = ds.time_graphs("fwd", ksteps, min(args.warmup, 50))
        ms_b, lb = ds.time_graphs("bwd", ksteps, min(args.warmup, 50))
        t_fwd_us, t_bwd_us = ms_f / ksteps * 1e3, ms_b / ksteps * 1e3
        clocks = sampler.summary()
        mech = 0 if binding.invconv_path_for(shape.B, shape.C, shape.H, shape.W, shape.k) == binding.PATH_WARP else 1
        t_step_cycles = binding.invconv_probe_step_latency(mech, 4096, device)
        bd = bounds(shape, t_step_cycles, clocks["sm_max_mhz"], hbm_gbs)
        t_roof = max(bd["t_hbm_us"], bd["t_alu_us"], bd["t_cp_us"])
        binding_name = max((("hbm", bd["t_hbm_us"]), ("alu", bd["t_alu_us"]), ("critical_path", bd["t_cp_us"])),
                           key=lambda kv: kv[1])[0]
        # dominant kernel = the backward launch (reads grad_x and x, writes grad_y: 12 B per element, plus w and grad_w)
        E = shape.elements
        wb = 4 * shape.C * shape.C * shape.k * shape.k
        dom_bytes = 12 * E + 2 * wb
        achieved = dom_bytes / (t_bwd_us * 1e-6) / 1e9
        cpu = cpu_baseline(args.workload)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "B": shape.B, "C": shape.C, "H": shape.H, "W": shape.W,
                       "k": shape.k, "per_rank_batch": shape.B, "parallelism": f"replicas x{world}",
                       "l2": f"rotating {ds.nsets} buffer sets ({ds.nsets * 16 * E / 2**20:.0f} MiB > 2x L2)",
                       "launch": "CUDA graphs of <=128 steps replayed on one stream",
                       "kernel_path": binding.invconv_path_for(shape.B, shape.C, shape.H, shape.W, shape.k)},
            "us_per_layer": {"forward": t_fwd_us, "backward": t_bwd_us, "sum": t_fwd_us + t_bwd_us},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s",
                         "frac": achieved / hbm_gbs, "traffic": NCU_TRAFFIC_BYTES.get(args.workload), "kernel": "backward (grad_y + grad_w)",
                         "algorithmic_bytes_per_launch": dom_bytes, "peak_kind": f"of {peak_kind}"},
            "north_star_roofline": {"t_hbm_us": bd["t_hbm_us"], "t_alu_us": bd["t_alu_us"], "t_cp_us": bd["t_cp_us"],
                                    "t_step_cycles": t_step_cycles, "step_mechanism": mech, "binding": binding_name,
                                    "t_roofline_us": t_roof, "t_achieved_us": t_fwd_us + t_bwd_us,
                                    "frac": t_roof / (t_fwd_us + t_bwd_us)},
            "cpu_baseline": cpu,
            "e2e": {"value": world * shape.B * e2e_steps / (ms_e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": hs.h2d_bytes, "d2h_bytes_per_step": hs.d2h_bytes,
                    "ms_per_step": ms_e / e2e_steps, "steps": e2e_steps,
                    "pipeline": "two host-buffer sets alternating on two streams"},
            "gpu_launches": launches,
            "clocks": clocks,
        }
    barrier()
    if dist is not None:
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out))


def run_table(args):
    """Every benchmark shape on one GPU: microseconds per call and fraction of its roofline (human-readable)."""
    import torch
    from paper_2410_14634_b200 import binding, workloads
    device = torch.device("cuda:0")
    hbm_gbs, _ = peaks()
    rows = []
    for shape in workloads.SHAPES:
        _, w, y, gx = workloads.make(shape.name)
        ds = DeviceStep(shape, w, y, gx, device)
        steps = args.steps
        ms_f, _ = ds.time_graphs("fwd", steps, args.warmup)
        ms_b, _ = ds.time_graphs("bwd", steps, args.warmup)
        path = binding.invconv_path_for(shape.B, shape.C, shape.H, shape.W, shape.k)
        cyc = binding.invconv_probe_step_latency(0 if path == binding.PATH_WARP else 1, 4096, device)
        bd = bounds(shape, cyc, 1965, hbm_gbs)
        t = (ms_f + ms_b) / steps * 1e3
        roof = max(bd["t_hbm_us"], bd["t_alu_us"], bd["t_cp_us"])
        ms_c, _ = ds.time_graphs("conv", steps, args.warmup)
        rows.append({"shape": shape.name, "path": path, "t_fwd_us": ms_f / steps * 1e3, "t_bwd_us": ms_b / steps * 1e3,
                     "t_masked_conv_us": ms_c / steps * 1e3,
                     "masked_conv_hbm_frac": (8.0 * shape.elements / (ms_c / steps * 1e-3) / 1e9) / hbm_gbs,
                     "images_per_s": shape.B / (t * 1e-6), **{k: bd[k] for k in ("t_hbm_us", "t_alu_us", "t_cp_us")},
                     "frac_of_roofline": roof / t})
        del ds
        torch.cuda.empty_cache()
    for r in rows:
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--workload", default="mnist")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--table", action="store_true", help="time every benchmark shape on one GPU")
    ap.add_argument("--sweep", action="store_true", help="time the ablation axes (kernel size, image side, batch) at C=3")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
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
