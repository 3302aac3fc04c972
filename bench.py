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

    def __init__(self, rank: int, minibatch: int = 0, fused_update: bool = True):
        import torch
        from paper_1602_06709_b200 import inputs, networks
        self.torch = torch
        self.N = minibatch or 256
        # (fused_update: each layer's SGD update is applied by its own weight-gradient call; the data-parallel step,
        # which exchanges the gradients, keeps them and updates the owned strips)
        self.net = networks.VggA(self.N, fused_update=fused_update)
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

    def __init__(self, rank: int, minibatch: int = 0, layer=None, pooled=False):
        import torch
        from paper_1602_06709_b200 import binding as B
        from paper_1602_06709_b200 import inputs
        self.torch, self.B = torch, B
        self.pooled = pooled
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
        if pooled:      # the layer as a pooled first layer of a step: conv + ReLU + 2x2 pool in one call (y not stored),
            # weight gradient straight from the pooled gradient and the position codes
            assert B.conv_fwd_pool_is_fused(self.d) and B.conv_bwd_weights_pooled_is_fused(self.d)
            ws = max(ws, B.conv_bwd_weights_pooled_workspace_bytes(self.d))
            self.yp = torch.empty(c["N"], c["H"] // 2, c["W"] // 2, c["K"], device="cuda")
            self.codes = torch.empty(c["N"], c["H"] // 2, c["W"] // 2, c["K"], dtype=torch.uint8, device="cuda")
            self.dyp = self.dy[:, ::2, ::2, :].contiguous()
            self.db = torch.empty(c["K"], device="cuda")
        self.ws = torch.empty(max(ws, 256), dtype=torch.uint8, device="cuda")
        self.flops_pass = 2 * c["N"] * c["K"] * c["H"] * c["W"] * c["C"] * 9
        self.units_per_step = 3 * self.flops_pass / 1e12      # TFLOP per step
        self.h2d = (self.x_host.numel() + self.dy_host.numel()) * 4
        self.d2h = self.dw.numel() * 4
        self.dw_host = torch.empty_like(self.dw, device="cpu").pin_memory()

    def step(self):
        B = self.B
        if self.pooled:
            B.conv_fwd_pool(self.d, self.x, self.w, self.bias, None, self.yp, B.ACT_RELU, self.ws, pool_codes=self.codes)
            B.conv_bwd_weights_pooled(self.d, self.x, self.dyp, self.codes, True, self.dw, self.db, self.ws)
            return
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

    def __init__(self, rank: int, minibatch: int = 0, fused_update: bool = True):
        import torch
        from paper_1602_06709_b200 import inputs, networks
        self.torch = torch
        self.N = minibatch or inputs.CFG4_N
        self.net = networks.Dnn(self.N, fused_update=fused_update)
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

    for kv in args.tune:
        if not args.kernels_only:
            raise SystemExit("--tune changes which kernels run: only allowed with --kernels-only")
        name, _, val = kv.partition("=")
        B.set_tuning(name, val if name == "TILING" and not val.lstrip("-").isdigit() else int(val))
    if args.layer and not (args.kernels_only and args.workload == "conv"):
        raise SystemExit("--layer changes the workload: only allowed with --workload conv --kernels-only")
    if args.layer:
        wl = ConvWorkload(rank, args.minibatch, tuple(int(v) for v in args.layer.split(",")), pooled=args.pooled)
    else:
        wl = (WORKLOADS[args.workload](rank, args.minibatch, fused_update=False)
              if args.data_parallel and args.workload in ("vgga", "dnn") else WORKLOADS[args.workload](rank, args.minibatch))
    if args.data_parallel:
        # Sec. 3.1 / 3.4: the ranks share one model; every rank's step() exchanges the weight gradients layer by layer
        if not hasattr(wl, "net"):
            raise SystemExit("--data-parallel needs a network workload (vgga or dnn)")
        from paper_1602_06709_b200 import data_parallel
        dp = data_parallel.DataParallelStep(wl.net)
        wl.step = dp.step
        wl.step_eager = dp.step
        wl.e2e_step = None
    peaks = load_peaks()
    # The DNN step is ~33 short kernels and bound by the host's launch rate when issued one by one: by default it is
    # replayed from a CUDA graph of exactly those launches.  The VGG-A step (79 launches) keeps the GPU busy either way,
    # but the replay still closes the gaps between its launches (17.13 against 17.32 ms measured), so it is the default too.
    use_graph = hasattr(wl, "use_graph") and not args.data_parallel and \
        (args.graph == "1" or (args.graph == "auto" and (args.workload == "dnn" or (args.workload == "vgga" and not args.kernels_only))))
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
    unit, h2d, d2h = wl.unit, wl.h2d, wl.d2h

    if args.kernels_only:      # for profiler captures: just the steps, one short line
        if rank == 0:
            print(json.dumps({"workload": wl.name, "minibatch": wl.N, "ms_per_step": ms / args.steps,
                              "gpu_launches": launches}), flush=True)
        return

    # end to end through the user-level call: pinned host minibatch in, result out, every step
    e2e_steps = max(3, min(args.steps, 10))
    if wl.e2e_step is not None:
        ms_e2e, _, _ = timed(wl.e2e_step, e2e_steps, 1)
        e2e_value = replicas.whole_job_throughput(wl.units_per_step, e2e_steps, world, ms_e2e)
    else:       # (the data-parallel job is timed with resident inputs only)
        ms_e2e, e2e_value = float("nan"), None

    # instrumented repeat of the same steps: CUDA events around every kernel launch on the launching stream,
    # tagged with the pass (ABI call) the launch belongs to
    prof_steps = max(1, min(args.steps, 5))
    barrier()
    B.profile_begin()
    for _ in range(prof_steps):
        wl.step_eager()       # (a graph replay does not pass through the library's per-launch events)
    stats = B.profile_end()
    barrier()
    report = summarise_profile(stats, prof_steps, peaks, clocks, ms / args.steps, args.workload)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r = time_oracle(args.workload, 1, 0, min_seconds=12.0)
        cpu = dict(value=r["value"], unit=wl.unit, cores=r["cores"], kind="oracle", sample=r["sample"],
                   seconds=r["seconds"])

    config = {"workload": wl.name, "l2": "inputs larger than L2 (activations are GBs per step)"
              if args.workload != "dnn" else "weights+activations 0.3 GB per step, larger than L2",
              "parallelism": ("data-parallel: per-layer reduce-scatter / owned-strip SGD / all-gather" if args.data_parallel
                              else "replicas only" if world > 1 else "single GPU"), "cuda_graph": bool(use_graph),
              **wl.describe()}
    legs = None
    if world == 1 and args.workload == "vgga" and not args.no_legs:
        # the other configurations, a few repetitions each, so that one record carries them; and the TF32 stick
        del wl
        torch.cuda.empty_cache()
        legs = run_legs(torch, B)
        stick = measure_tf32_stick(torch, local_rank)
        report["roofline"].update(stick)
        if stick.get("peak_measured_tf32_burst"):
            report["roofline"]["frac_of_measured_tf32_burst"] = report["roofline"]["achieved"] / stick["peak_measured_tf32_burst"]
            report["roofline"]["frac_of_measured_tf32_sustained"] = report["roofline"]["achieved"] / stick["peak_measured_tf32_sustained"]

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "tf32", "data": "synthetic",
            "config": config,
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / e2e_steps, "steps": e2e_steps},
            "gpu_launches": launches,
            "cpu_baseline": cpu,
            **report,
        }
        if legs is not None:
            line["legs"] = legs
        print(json.dumps(line), flush=True)
    replicas.shutdown()


CONTRACTIONS = ("tc_fprop_kernel", "tc_wgrad_kernel", "generic_fwd", "generic_bwd_data", "generic_bwd_weights")
NOMINAL_TF32_TFLOPS = 1100.0


def summarise_profile(stats, prof_steps, peaks, clocks, ms_per_step, workload):
    """stats: {"<pass>/<kernel>": dict(launches, total_ms, work)} over prof_steps steps."""
    by_kernel, by_pass = {}, {}
    for name, s in stats.items():
        ps, k = name.split("/", 1)
        a = by_kernel.setdefault(k, dict(launches=0, total_ms=0.0, work=0.0))
        for f in ("launches", "total_ms", "work"):
            a[f] += s[f]
        b = by_pass.setdefault(ps, dict(ms=0.0, contraction_ms=0.0, flop=0.0, launches=0))
        b["ms"] += s["total_ms"]
        b["launches"] += s["launches"]
        if k in CONTRACTIONS:
            b["contraction_ms"] += s["total_ms"]
            b["flop"] += s["work"]
    total_ms = sum(s["total_ms"] for s in by_kernel.values())
    kernels = {k: dict(launches=s["launches"] // prof_steps, ms_per_step=s["total_ms"] / prof_steps,
                       share=s["total_ms"] / total_ms if total_ms else 0.0, work_per_step=s["work"] / prof_steps)
               for k, s in by_kernel.items()}

    def rate(flop, ms_):
        return flop / (ms_ / 1e3) / 1e12 if ms_ > 0 else None

    # burst figure: the timed region is a fraction of a second (the sustained figure belongs to seconds-long loops
    # at the power cap; MEASURED_PEAKS took it at a median 1305 MHz, this step runs at 1.7-1.96 GHz)
    peak_burst = peaks["bf16_burst"] * TF32_OVER_BF16_NOMINAL
    peak_sust = peaks["bf16_sustained"] * TF32_OVER_BF16_NOMINAL
    out = {"kernels": kernels}
    passes = {}
    for ps, key in (("conv_fwd", "fwd"), ("conv_bwd_data", "bwd_data"), ("conv_bwd_weights", "bwd_weights")):
        if ps in by_pass and by_pass[ps]["flop"] > 0:
            b = by_pass[ps]
            passes[key] = dict(tflops=rate(b["flop"], b["ms"]), ms=b["ms"] / prof_steps,
                               contraction_kernel_tflops=rate(b["flop"], b["contraction_ms"]),
                               contraction_kernel_ms=b["contraction_ms"] / prof_steps,
                               flop=b["flop"] / prof_steps, launches=b["launches"] // prof_steps)
    if passes:
        out["conv_passes"] = passes
        flop = sum(by_pass[ps]["flop"] for ps in ("conv_fwd", "conv_bwd_data", "conv_bwd_weights") if ps in by_pass)
        ms_all = sum(by_pass[ps]["ms"] for ps in ("conv_fwd", "conv_bwd_data", "conv_bwd_weights") if ps in by_pass)
        t = rate(flop, ms_all)
        out["conv_layers"] = dict(tflops=t, ms=ms_all / prof_steps, flop=flop / prof_steps,
                                  frac_of_nominal_1100=t / NOMINAL_TF32_TFLOPS, frac_of_measured=t / peak_burst,
                                  note="every launch of the three conv passes (staging, split reductions and "
                                       "transposes included) over the layers' own 2*N*K*P*Q*C*R*S")
    fcs = [by_pass[ps] for ps in ("fc_fwd", "fc_bwd") if ps in by_pass and by_pass[ps]["flop"] > 0]
    if fcs:
        flop = sum(b["flop"] for b in fcs); ms_all = sum(b["ms"] for b in fcs)
        out["fc_layers"] = dict(tflops=rate(flop, ms_all), ms=ms_all / prof_steps, flop=flop / prof_steps)
    tc = [s for k, s in by_kernel.items() if k in CONTRACTIONS]
    if tc:
        t = rate(sum(s["work"] for s in tc), sum(s["total_ms"] for s in tc))
        out["all_contractions"] = dict(tflops=t, frac_of_measured=t / peak_burst, frac_of_nominal_1100=t / NOMINAL_TF32_TFLOPS,
                                       flop_over_step_time_tflops=rate(sum(s["work"] for s in tc) / prof_steps, ms_per_step))
    if "sgd_kernel" in by_kernel:
        s = by_kernel["sgd_kernel"]
        out["sgd_update_gbs"] = s["work"] / (s["total_ms"] / 1e3) / 1e9

    dom = max(by_kernel.items(), key=lambda kv: kv[1]["total_ms"])[0]
    ds = by_kernel[dom]
    if dom in CONTRACTIONS:
        achieved = ds["work"] / (ds["total_ms"] / 1e3) / 1e12
        roofline = dict(bound="tensor", kernel=dom, achieved=achieved, peak=peak_burst, unit="TFLOP/s",
                        frac=achieved / peak_burst, traffic=None,
                        peak_source=f"{peaks['source']} bf16 burst {peaks['bf16_burst']:.1f} TFLOP/s x nominal TF32/bf16 "
                                    f"ratio {TF32_OVER_BF16_NOMINAL:.4f} (of {peaks['source']})",
                        frac_of_sustained_derived=achieved / peak_sust, peak_sustained_derived=peak_sust,
                        frac_of_nominal_1100=achieved / NOMINAL_TF32_TFLOPS,
                        launches_per_step=ds["launches"] // prof_steps,
                        flop_per_launch_avg=ds["work"] / ds["launches"], ms_per_launch_avg=ds["total_ms"] / ds["launches"],
                        timed_in="instrumented repeat of the timed steps (events on the launching stream)")
    else:
        achieved = ds["work"] / (ds["total_ms"] / 1e3) / 1e9
        roofline = dict(bound="hbm", kernel=dom, achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=achieved / peaks["hbm_gbs"], traffic=None, peak_source=f"{peaks['source']} copy bandwidth",
                        launches_per_step=ds["launches"] // prof_steps)
    roofline["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get(workload, {}).get(dom)
    roofline["traffic_source"] = "ncu capture summarised under profiles/ (a constant of this script, not measured by this run)"
    out["roofline"] = roofline
    return out


def measure_tf32_stick(torch, gpu_index):
    """A TF32 measuring stick outside the product path and outside every timed region: torch.matmul 8192^3 with
    allow_tf32 (cuBLAS), best of 10 (burst) and back to back for ~3 s (sustained), clocks sampled meanwhile."""
    try:
        old = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = True
        n = 8192
        a = torch.randn(n, n, device="cuda"); b = torch.randn(n, n, device="cuda"); c = torch.empty(n, n, device="cuda")
        flop = 2.0 * n ** 3
        for _ in range(3):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize()
        best = 1e30
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch.matmul(a, b, out=c); e1.record(); e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        sampler = ClockSampler(gpu_index); sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(10, int(3000.0 / best))
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record(); e1.synchronize()
        clk = sampler.stop()
        torch.backends.cuda.matmul.allow_tf32 = old
        return dict(peak_measured_tf32_burst=flop / (best / 1e3) / 1e12,
                    peak_measured_tf32_sustained=flop * reps / (e0.elapsed_time(e1) / 1e3) / 1e12,
                    peak_measured_tf32_how="torch.matmul fp32 8192^3 with allow_tf32 (a library GEMM, measuring stick only): "
                                           "best of 10, and back to back for ~3 s",
                    peak_measured_tf32_clocks=clk)
    except Exception as e:          # the stick is context; the bench line must not depend on it
        return dict(peak_measured_tf32_burst=None, peak_measured_tf32_sustained=None, peak_measured_tf32_how=f"failed: {e}")


def run_legs(torch, B):
    """Short legs for the other configurations: the three passes of the mid VGG-A layer (configs[1]) and of each
    OverFeat-FAST-shaped layer (configs[2]), and the DNN step (configs[3]).  Device-side seeded inputs with the
    recipe's distributions; L2 is flushed before every timed repetition (a 256 MB buffer is overwritten)."""
    gen = torch.Generator(device="cuda"); gen.manual_seed(160206709)
    flush = torch.empty(64 * 1024 * 1024, device="cuda")

    def time_call(fn, reps=5, warm=3):
        for _ in range(warm):
            fn()
        best, tot = 1e30, 0.0
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); e1.synchronize()
            t = e0.elapsed_time(e1); best = min(best, t); tot += t
        return tot / reps, best

    def conv_leg(N, C, K, H, R, stride, pad):
        d = B.conv_desc(N, C, K, H, H, R, R, stride, pad)
        P = (H + 2 * pad - R) // stride + 1
        x = torch.rand(N, H, H, C, device="cuda", generator=gen)
        w = torch.randn(K, R, R, C, device="cuda", generator=gen) * (2.0 / (R * R * C)) ** 0.5
        dy = torch.randn(N, P, P, K, device="cuda", generator=gen) * 1e-3
        bias = torch.zeros(K, device="cuda")
        y = torch.empty_like(dy); dx = torch.empty_like(x); dw = torch.empty_like(w)
        ws = torch.empty(max(256, max(B.conv_workspace_bytes(d, i) for i in range(3))), dtype=torch.uint8, device="cuda")
        flop = 2.0 * N * K * P * P * C * R * R
        out = {"shape": f"N={N} C={C} K={K} H=W={H} {R}x{R} stride {stride} pad {pad}", "flop_per_pass": flop}
        for key, fn in (("fwd", lambda: B.conv_fwd(d, x, w, bias, y, B.ACT_RELU, ws)),
                        ("bwd_data", lambda: B.conv_bwd_data(d, dy, w, None, dx, ws)),
                        ("bwd_weights", lambda: B.conv_bwd_weights(d, x, dy, dw, None, True, ws))):
            mean, best = time_call(fn)
            out[key] = dict(ms=mean, best_ms=best, tflops=flop / (mean / 1e3) / 1e12,
                            frac_of_nominal_1100=flop / (mean / 1e3) / 1e12 / NOMINAL_TF32_TFLOPS)
        return out

    legs = {"timing": "CUDA events per call, mean of 5 after 3 warm-ups, L2 flushed before each; whole ABI call "
                      "(staging, transposes and split reductions included)"}
    legs["cfg2_vgg_mid_layer"] = conv_leg(256, 256, 256, 56, 3, 1, 1)
    cfg3 = {}
    for name, (C, H, K, R, st, pad) in (("C1", (3, 231, 96, 11, 4, 0)), ("C2", (96, 24, 256, 5, 1, 0)),
                                        ("C3", (256, 12, 512, 3, 1, 1)), ("C4", (512, 12, 1024, 3, 1, 1)),
                                        ("C5", (1024, 12, 1024, 3, 1, 1))):
        cfg3[name] = conv_leg(256, C, K, H, R, st, pad)
        torch.cuda.empty_cache()
    legs["cfg3_overfeat_fast"] = cfg3
    dnn = DnnWorkload(0)
    dnn.use_graph()
    for _ in range(3):
        dnn.step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        dnn.step()
    e1.record(); e1.synchronize()
    ms_dnn = e0.elapsed_time(e1) / 20
    fl = 3 * sum(dnn.net.fc_flops_fwd) - dnn.net.fc_flops_fwd[0]       # the first layer has no backpropagation
    legs["cfg4_dnn_step"] = dict(ms_per_step=ms_dnn, frames_per_s=dnn.N / (ms_dnn / 1e3), tflops=fl / (ms_dnn / 1e3) / 1e12,
                                 flop_per_step=fl, cuda_graph=True, steps=20)
    status = B.last_device_status()
    if status != B.OK:
        raise SystemExit(f"device status {status} after the legs: {B.status_string(status)}")
    return legs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgga", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the short legs for the other configurations")
    ap.add_argument("--graph", default="auto", choices=["auto", "0", "1"],
                    help="replay the step from a CUDA graph of its launches (auto: the DNN step only)")
    ap.add_argument("--minibatch", type=int, default=0, help="override the workload's minibatch (profiling only)")
    ap.add_argument("--tune", action="append", default=[], metavar="KNOB=VALUE",
                    help="pin a launcher choice through pcl_set_tuning for this run (profiling only), e.g. XHALO_WGRAD=0")
    ap.add_argument("--layer", default="", help="C,K,H of another 3x3 pad-1 layer for --workload conv (profiling only)")
    ap.add_argument("--data-parallel", action="store_true",
                    help="vgga / dnn with --gpus N > 1: one data-parallel job (per-layer reduce-scatter of the weight "
                         "gradients, SGD on the owned strip, all-gather of the weights, overlapped with the backward "
                         "pass) instead of N independent replicas; every rank keeps the workload's minibatch "
                         "(the global minibatch grows with N: weak scaling)")
    ap.add_argument("--pooled", action="store_true",
                    help="with --layer: run the layer as a pooled first layer (conv+pool in one call, weight gradient "
                         "from the pooled gradient); profiling only")
    ap.add_argument("--kernels-only", action="store_true",
                    help="run warm-up + timed steps only and print a short line (for profiler captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
