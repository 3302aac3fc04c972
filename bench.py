#!/usr/bin/env python
"""Benchmark of the training hot path on B200.

    python bench.py --gpus N --steps K --warmup W [--workload vgga|conv|dnn] [--impl reference]

A step is one pass of the whole hot path over one minibatch of seeded synthetic
input.  Default workload: the full VGG-A training step at minibatch 256
(forward, backward, SGD update: every row of the hot path -- conv forward /
backward-data / weight-gradient, FC forward / backward, update, pooling, loss).
`--workload conv` times the three passes + update of the VGG-A mid-network conv
layer (3x3, N=256, C=K=256, 56x56); `--workload dnn` the 7-layer DNN step.

One JSON line is printed by rank 0.  `value` is whole-job throughput with inputs
resident in HBM; `e2e` is the same metric through the user-level call with a
pinned host minibatch copied in and the loss read back every step; `roofline`
describes the dominant kernel (event-timed inside an instrumented repeat of the
same steps); `cpu_baseline` is the fp64 oracle timed on the host cores on a
bounded sample.  With N > 1 (torchrun) every rank runs an independent replica on
its own minibatch shard: the path has no exchange step on one node without the
paper's multinode gradient exchange, so there is no data-path collective.

`--impl reference` times the oracle (there is no reference implementation to
install: the paper's code was never published).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "conv fwd/bwd-data/bwd-wgt TFLOP/s and VGG-A images/sec at 1 B200 (% TF32 peak)"
TF32_OVER_BF16_NOMINAL = 1.1 / 2.25      # nominal dense TF32 / bf16 tensor peaks
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu (captured at minibatch 32 and scaled to the
# full minibatch: weight bytes once, activation bytes x 8); the captures are summarised under profiles/
NCU_DRAM_BYTES_PER_LAUNCH = {
    "vgga": {"tc_fprop_kernel": 531.4e6, "tc_wgrad_kernel": 930.7e6},
    "conv": {"tc_fprop_kernel": (163.8e6 + 283.9e6) / 2 * 8, "tc_wgrad_kernel": 209.9e6 * 8},
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(source="measured", hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])))
    return dict(source="fallback", hbm_gbs=FALLBACK_HBM_GBS, bf16_burst=FALLBACK_BF16_TFLOPS, bf16_sustained=1400.0)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"], samples=0)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    power_w_max=max(power) if power else None, reasons=sorted(reasons), samples=len(sm))


# ---------------------------------------------------------------------------
# Workloads (CUDA arm)
# ---------------------------------------------------------------------------
class VggWorkload:
    name = "configs[4]: full VGG-A training step (fwd+bwd+SGD), N=256, 3x224x224, He-normal weights, 1000 classes"
    unit = "images/s"

    def __init__(self, rank: int, minibatch: int = 0):
        import torch
        from paper_1602_06709_b200 import inputs, networks
        self.torch = torch
        self.N = minibatch or 256
        self.net = networks.VggA(self.N)
        x = inputs.uniform(inputs.tensor_id("cfg5", "x", rank), (self.N, 224, 224, 3), 0.0, 1.0)
        lab = inputs.labels(inputs.tensor_id("cfg5", "labels", rank), self.N, 1000)
        self.x_host = torch.from_numpy(x).pin_memory()
        self.lab_host = torch.from_numpy(lab).pin_memory()
        self.net.x.copy_(self.x_host)
        self.net.labels.copy_(self.lab_host)
        self.units_per_step = self.N
        self.conv_flops = 3 * sum(self.net.conv_flops_fwd) - self.net.conv_flops_fwd[0]   # conv1 skips bwd-data
        self.fc_flops = 3 * sum(self.net.fc_flops_fwd)
        self.h2d = self.x_host.numel() * 4 + self.lab_host.numel() * 4
        self.d2h = 4

    def step(self):
        self.net.run_step()        # the captured CUDA graph when use_graph() was called, else launch by launch

    def step_eager(self):
        self.net.step()

    def use_graph(self):
        self.net.capture_step()
        return self.net.graph_launches

    def e2e_step(self):
        # the next minibatch (here: the same pinned buffers) is copied while this step computes
        return self.net.step_from_host(self.x_host, self.lab_host, self.x_host, self.lab_host)

    def describe(self):
        return dict(minibatch=self.N, conv_flop_per_step=self.conv_flops, fc_flop_per_step=self.fc_flops,
                    params=self.net.store.n_real())


class ConvWorkload:
    name = "configs[1]: VGG-A mid conv layer 3x3 s1 p1, N=256 C=K=256 56x56: fwd + bwd_data + bwd_weights + SGD update"
    unit = "TFLOP/s"

    def __init__(self, rank: int, minibatch: int = 0, layer=None):
        import torch
        from paper_1602_06709_b200 import binding as B
        from paper_1602_06709_b200 import inputs
        self.torch, self.B = torch, B
        c = dict(inputs.CFG2)
        if minibatch:
            c["N"] = minibatch
        if layer:       # profiler captures of another 3x3 pad-1 layer shape (--layer C,K,H with --kernels-only)
            c["C"], c["K"], c["H"] = layer
            c["W"] = c["H"]
        self.N = c["N"]
        self.d = B.conv_desc(c["N"], c["C"], c["K"], c["H"], c["W"], c["R"], c["S"], 1, 1)
        x, w, dy = inputs.conv_inputs("cfg2", f"conv{rank}", c["N"], c["C"], c["H"], c["W"], c["K"], 3, 3, c["H"], c["W"],
                                      "train")
        self.x_host = torch.from_numpy(x).pin_memory()
        self.dy_host = torch.from_numpy(dy).pin_memory()
        self.x = torch.empty_like(self.x_host, device="cuda"); self.x.copy_(self.x_host)
        self.dy = torch.empty_like(self.dy_host, device="cuda"); self.dy.copy_(self.dy_host)
        self.w = torch.from_numpy(w).cuda()
        self.bias = torch.zeros(c["K"], device="cuda")
        self.y = torch.empty_like(self.dy); self.dx = torch.empty_like(self.x); self.dw = torch.empty_like(self.w)
        ws = max(B.conv_workspace_bytes(self.d, i) for i in range(3))
        self.ws = torch.empty(max(ws, 256), dtype=torch.uint8, device="cuda")
        self.flops_pass = 2 * c["N"] * c["K"] * c["H"] * c["W"] * c["C"] * 9
        self.units_per_step = 3 * self.flops_pass / 1e12      # TFLOP per step
        self.h2d = (self.x_host.numel() + self.dy_host.numel()) * 4
        self.d2h = self.dw.numel() * 4
        self.dw_host = torch.empty_like(self.dw, device="cpu").pin_memory()

    def step(self):
        B = self.B
        B.conv_fwd(self.d, self.x, self.w, self.bias, self.y, B.ACT_RELU, self.ws)
        B.conv_bwd_weights(self.d, self.x, self.dy, self.dw, None, True, self.ws)
        B.conv_bwd_data(self.d, self.dy, self.w, self.x, self.dx, self.ws)
        B.sgd_update(self.w, self.dw, 1e-6)

    step_eager = step

    def e2e_step(self):
        self.x.copy_(self.x_host, non_blocking=True)
        self.dy.copy_(self.dy_host, non_blocking=True)
        self.step()
        self.dw_host.copy_(self.dw, non_blocking=False)
        return float(self.dw_host[0, 0, 0, 0])

    def describe(self):
        return dict(minibatch=self.N, flop_per_pass=self.flops_pass)


class DnnWorkload:
    name = "configs[3]: 7-layer DNN 440-5x2048-8192, sigmoid, minibatch 1024: fwd + bwd + SGD update"
    unit = "frames/s"

    def __init__(self, rank: int, minibatch: int = 0):
        import torch
        from paper_1602_06709_b200 import inputs, networks
        self.torch = torch
        self.N = minibatch or inputs.CFG4_N
        self.net = networks.Dnn(self.N)
        x = inputs.normal(inputs.tensor_id("cfg4", "x", rank), (self.N, 440), 1.0)
        lab = inputs.labels(inputs.tensor_id("cfg4", "labels", rank), self.N, 8192)
        self.x_host = torch.from_numpy(x).pin_memory(); self.lab_host = torch.from_numpy(lab).pin_memory()
        self.net.x.copy_(self.x_host); self.net.labels.copy_(self.lab_host)
        self.units_per_step = self.N
        self.h2d = self.x_host.numel() * 4 + self.lab_host.numel() * 4
        self.d2h = 4

    def step(self):
        self.net.run_step()        # the captured CUDA graph when use_graph() was called, else launch by launch

    def step_eager(self):
        self.net.step()

    def use_graph(self):
        self.net.capture_step()
        return self.net.graph_launches

    def e2e_step(self):
        # the next minibatch (here: the same pinned buffers) is copied while this step computes
        return self.net.step_from_host(self.x_host, self.lab_host, self.x_host, self.lab_host)

    def describe(self):
        return dict(minibatch=self.N, fc_flop_per_step=3 * sum(self.net.fc_flops_fwd), params=self.net.store.n_real())


WORKLOADS = {"vgga": VggWorkload, "conv": ConvWorkload, "dnn": DnnWorkload}


# ---------------------------------------------------------------------------
# Oracle legs (CPU)
# ---------------------------------------------------------------------------
def oracle_sample(workload: str):
    """Returns (callable running one bounded sample through the oracle, units per call, description)."""
    import numpy as np
    import oracle
    import oracle.networks as ON
    from oracle import ConvShape
    from paper_1602_06709_b200 import inputs
    if workload == "vgga":
        n = 1
        x = inputs.uniform(inputs.tensor_id("cfg5", "x", 0), (n, 224, 224, 3), 0.0, 1.0)
        lab = inputs.labels(inputs.tensor_id("cfg5", "labels", 0), n, 1000)
        conv_params = [(inputs.he_normal_conv(inputs.tensor_id("cfg5", name, "w"), K, 3, 3, C), np.zeros(K, np.float32))
                       for name, C, K, _ in inputs.VGGA_CONV]
        fc_params = [(inputs.he_normal_fc(inputs.tensor_id("cfg5", f"fc{j + 1}", "w"), K, C), np.zeros(K, np.float32))
                     for j, (C, K) in enumerate(inputs.VGGA_FC)]
        spec = [(C, K, p) for _, C, K, p in inputs.VGGA_CONV]
        fn = lambda: ON.vgga_step(x, lab, conv_params, fc_params, spec, 0.01)
        return fn, n, f"full VGG-A training step (fwd+bwd+SGD) at minibatch {n} of 256, same recipe"
    if workload == "conv":
        n = 2
        s = ConvShape(N=n, C=256, K=256, H=56, W=56, R=3, S=3, pad_h=1, pad_w=1)
        x, w, dy = inputs.conv_inputs("cfg2", "conv0", n, 256, 56, 56, 256, 3, 3, 56, 56, "train")

        def fn():
            oracle.conv_fwd(s, x, w, np.zeros(256, np.float32), oracle.ACT_RELU)
            dw = oracle.conv_bwd_weights(s, x, dy)
            oracle.conv_bwd_data(s, dy, w, x)
            oracle.sgd_update(w, dw, 1e-6)
        return fn, 3 * s.flops() / 1e12, f"the three passes + update at minibatch {n} of 256, same layer"
    if workload == "dnn":
        n = 64
        dims = inputs.CFG4_DIMS
        x = inputs.normal(inputs.tensor_id("cfg4", "x", 0), (n, 440), 1.0)
        lab = inputs.labels(inputs.tensor_id("cfg4", "labels", 0), n, 8192)
        params = [(inputs.xavier_uniform_fc(inputs.tensor_id("cfg4", f"fc{j + 1}", "w"), K, C), np.zeros(K, np.float32))
                  for j, (C, K) in enumerate(zip(dims[:-1], dims[1:]))]
        fn = lambda: ON.dnn_step(x, lab, params, 0.01)
        return fn, n, f"full DNN training step at minibatch {n} of 1024, same recipe"
    raise ValueError(workload)


def time_oracle(workload: str, steps: int, warmup: int, min_seconds: float = 0.0):
    """steps > 0: exactly that many timed calls of the bounded sample.  min_seconds > 0 (the cpu_baseline leg): the
    sample is repeated until about that much CPU time has been measured (at most 16 calls)."""
    import oracle
    fn, units, sample = oracle_sample(workload)
    for _ in range(warmup):
        fn()
    t0 = time.perf_counter()
    done = 0
    while done < steps or (min_seconds > 0 and done < 16 and time.perf_counter() - t0 < min_seconds):
        fn()
        done += 1
    dt = time.perf_counter() - t0
    if done > 1 and min_seconds > 0:
        sample += f", {done} calls"
    return dict(value=units * done / dt, seconds_per_step=dt / done, cores=oracle.threads(), sample=sample,
                seconds=dt)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = WORKLOADS[args.workload]
    r = time_oracle(args.workload, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": wl.unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["seconds_per_step"] * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "sample": r["sample"]},
        "cpu_baseline": {"value": r["value"], "unit": wl.unit, "cores": r["cores"], "kind": "oracle",
                         "sample": r["sample"]},
        "e2e": {"value": r["value"], "unit": wl.unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
        "note": "the oracle (fp64 direct loops, OpenMP) timed on the host cores; no published reference code exists",
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import replicas

    world, rank, local_rank = replicas.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    replicas.init("nccl", torch.device("cuda", local_rank))
    if args.minibatch and not args.kernels_only:
        raise SystemExit("--minibatch changes the workload: only allowed with --kernels-only")
    B.lib()      # fail loudly here if the extension is missing

    def barrier():
        replicas.barrier(cuda=True)

    def max_over_ranks(v: float) -> float:
        return replicas.max_over_ranks(v, device="cuda")

    if args.layer and not (args.kernels_only and args.workload == "conv"):
        raise SystemExit("--layer changes the workload: only allowed with --workload conv --kernels-only")
    if args.layer:
        wl = ConvWorkload(rank, args.minibatch, tuple(int(v) for v in args.layer.split(",")))
    else:
        wl = WORKLOADS[args.workload](rank, args.minibatch)
    peaks = load_peaks()
    # The DNN step is ~45 short kernels and bound by the host's launch rate when issued one by one: by default it is
    # replayed from a CUDA graph of exactly those launches.  The VGG-A step keeps the GPU busy either way.
    use_graph = hasattr(wl, "use_graph") and (args.graph == "1" or (args.graph == "auto" and args.workload == "dnn"))
    graph_launches = wl.use_graph() if use_graph else 0

    def timed(fn, steps, warmup, sample_clocks=False):
        for _ in range(warmup):
            fn()
        barrier()
        sampler = ClockSampler(local_rank) if sample_clocks else None
        if sampler:
            sampler.start()
            time.sleep(0.25)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = B.launch_count()
        barrier()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        ms = max_over_ranks(e0.elapsed_time(e1))
        launches = B.launch_count() - n0 + (graph_launches * steps if fn == wl.step else 0)
        clocks = sampler.stop() if sampler else None
        return ms, launches, clocks

    ms, launches, clocks = timed(wl.step, args.steps, max(args.warmup, 3), sample_clocks=not args.kernels_only)
    status = B.last_device_status()
    if status != B.OK:
        raise SystemExit(f"device status {status}: {B.status_string(status)}")
    value = replicas.whole_job_throughput(wl.units_per_step, args.steps, world, ms)

    if args.kernels_only:      # for profiler captures: just the steps, one short line
        if rank == 0:
            print(json.dumps({"workload": wl.name, "minibatch": wl.N, "ms_per_step": ms / args.steps,
                              "gpu_launches": launches}), flush=True)
        return

    # end to end through the user-level call: pinned host minibatch in, result out, every step
    e2e_steps = max(3, min(args.steps, 10))
    ms_e2e, _, _ = timed(wl.e2e_step, e2e_steps, 1)
    e2e_value = replicas.whole_job_throughput(wl.units_per_step, e2e_steps, world, ms_e2e)

    # instrumented repeat of the same steps: CUDA events around every kernel launch on the launching stream
    prof_steps = max(1, min(args.steps, 5))
    barrier()
    B.profile_begin()
    for _ in range(prof_steps):
        wl.step_eager()       # (a graph replay does not pass through the library's per-launch events)
    stats = B.profile_end()
    barrier()
    total_ms = sum(s["total_ms"] for s in stats.values())
    kernels = {k: dict(launches=s["launches"] // prof_steps, ms_per_step=s["total_ms"] / prof_steps,
                       share=s["total_ms"] / total_ms if total_ms else 0.0,
                       work_per_step=s["work"] / prof_steps) for k, s in stats.items()}
    dom = max(stats.items(), key=lambda kv: kv[1]["total_ms"])[0]
    ds = stats[dom]
    contraction = dom in ("tc_fprop_kernel", "tc_wgrad_kernel", "generic_fwd", "generic_bwd_data", "generic_bwd_weights")
    if contraction:
        achieved = ds["work"] / (ds["total_ms"] / 1e3) / 1e12
        # the sustained figure for a kernel timed inside a long, power-capped step; the burst figure when the timed
        # region never met the power cap (short steps: the clock sampler saw no sw_power_cap)
        capped = bool(clocks and "sw_power_cap" in (clocks.get("reasons") or []))
        which = "sustained" if capped or not clocks else "burst"
        peak = peaks["bf16_" + which] * TF32_OVER_BF16_NOMINAL
        roofline = dict(bound="tensor", kernel=dom, achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                        traffic=None,
                        peak_source=f"{peaks['source']} bf16 {which} {peaks['bf16_' + which]:.1f} TFLOP/s x nominal "
                                    f"TF32/bf16 ratio {TF32_OVER_BF16_NOMINAL:.4f}",
                        launches_per_step=ds["launches"] // prof_steps,
                        flop_per_launch_avg=ds["work"] / ds["launches"], ms_per_launch_avg=ds["total_ms"] / ds["launches"],
                        timed_in="instrumented repeat of the timed steps (events on the launching stream)")
    else:
        achieved = ds["work"] / (ds["total_ms"] / 1e3) / 1e9
        roofline = dict(bound="hbm", kernel=dom, achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=achieved / peaks["hbm_gbs"], traffic=None, peak_source=f"{peaks['source']} copy bandwidth",
                        launches_per_step=ds["launches"] // prof_steps)
    roofline["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get(args.workload, {}).get(dom)

    extra = {}
    tc = [stats[k] for k in ("tc_fprop_kernel", "tc_wgrad_kernel") if k in stats]
    if tc:
        tflops = sum(s["work"] for s in tc) / (sum(s["total_ms"] for s in tc) / 1e3) / 1e12
        peak_s = peaks["bf16_sustained"] * TF32_OVER_BF16_NOMINAL
        extra["tensor_core_kernels"] = dict(tflops=tflops, frac_of_measured_sustained_tf32=tflops / peak_s,
                                            frac_of_nominal_1100=tflops / 1100.0)
    allc = [s for k, s in stats.items() if k in ("tc_fprop_kernel", "tc_wgrad_kernel", "generic_fwd",
                                                 "generic_bwd_data", "generic_bwd_weights")]
    if allc:
        extra["all_contractions_tflops"] = sum(s["work"] for s in allc) / (sum(s["total_ms"] for s in allc) / 1e3) / 1e12
    if "sgd_kernel" in stats:
        s = stats["sgd_kernel"]
        extra["sgd_update_gbs"] = s["work"] / (s["total_ms"] / 1e3) / 1e9

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r = time_oracle(args.workload, 1, 0, min_seconds=12.0)
        cpu = dict(value=r["value"], unit=wl.unit, cores=r["cores"], kind="oracle", sample=r["sample"],
                   seconds=r["seconds"])

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": wl.unit, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "tf32", "data": "synthetic",
            "config": {"workload": wl.name, "l2": "inputs larger than L2 (activations are GBs per step)"
                       if args.workload != "dnn" else "weights+activations 0.3 GB per step, larger than L2",
                       "parallelism": "replicas only" if world > 1 else "single GPU", "cuda_graph": bool(use_graph),
                       **wl.describe()},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": wl.unit, "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h,
                    "ms_per_step": ms_e2e / e2e_steps, "steps": e2e_steps},
            "gpu_launches": launches,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "kernels": kernels,
            **extra,
        }
        print(json.dumps(line), flush=True)
    replicas.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgga", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--graph", default="auto", choices=["auto", "0", "1"],
                    help="replay the step from a CUDA graph of its launches (auto: the DNN step only)")
    ap.add_argument("--minibatch", type=int, default=0, help="override the workload's minibatch (profiling only)")
    ap.add_argument("--layer", default="", help="C,K,H of another 3x3 pad-1 layer for --workload conv (profiling only)")
    ap.add_argument("--kernels-only", action="store_true",
                    help="run warm-up + timed steps only and print a short line (for profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
