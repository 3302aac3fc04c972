"""Blocking search for the forward-type tensor-core kernel (Sec. 2.2-2.3 re-posed for B200).

The paper picks the cache and register blocks of every layer with a brute-force
search that minimises bytes moved per flop under the cache capacity.  Here the
blocks are the kernel's tilings -- plain or haloed (three layouts), tile width
BN, single CTAs or CTA pairs (both tilings) -- and the search does both things the paper's does:

* the library's cost model (tensor pipe, shared-memory fill rate, issuing
  thread, epilogue warps; ``pcl_conv_plan_describe``) predicts every candidate;
* this script also MEASURES every candidate on the GPU (CUDA events around the
  ABI call, knobs pinned through ``pcl_set_tuning``), so that the model's choice,
  the launcher's own rule and the measured optimum can be compared layer by layer.

    python -m paper_1602_06709_b200.blocking_search [--minibatch 256] [--reps 5] [--layers vgga|overfeat] [--out table.md]
"""
from __future__ import annotations

import argparse
import re
import sys

import torch

from . import binding as B

VGGA = [("conv1", 3, 64, 224, 3, 1), ("conv2", 64, 128, 112, 3, 1), ("conv3", 128, 256, 56, 3, 1), ("conv4", 256, 256, 56, 3, 1),
        ("conv5", 256, 512, 28, 3, 1), ("conv6", 512, 512, 28, 3, 1), ("conv7", 512, 512, 14, 3, 1)]
OVERFEAT = [("C2", 96, 256, 24, 5, 0), ("C3", 256, 512, 12, 3, 1), ("C4", 512, 1024, 12, 3, 1), ("C5", 1024, 1024, 12, 3, 1)]


def _time(fn, reps, flush):
    for _ in range(2):
        fn()
    ts = []
    for _ in range(reps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record(); e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    return sorted(ts)[len(ts) // 2]


def _cfg_of(desc: str) -> str:
    m = re.match(r"tiling=(\S+) BN=(\d+) pair=(\d)", desc)
    return f"{m.group(1)}/BN{m.group(2)}/{'pair' if m.group(3) == '1' else 'single'}"


def _pred_clk(desc: str) -> float:
    return float(re.search(r"predicted_clk=(\d+)", desc).group(1))


def search_layer(name, N, C, K, H, R, pad, reps, flush, gen):
    d = B.conv_desc(N, C, K, H, H, R, R, 1, pad)
    P = H + 2 * pad - R + 1
    x = torch.rand(N, H, H, C, device="cuda", generator=gen)
    w = torch.randn(K, R, R, C, device="cuda", generator=gen) * (2.0 / (R * R * C)) ** 0.5
    dy = torch.randn(N, P, P, K, device="cuda", generator=gen) * 1e-3
    bias = torch.zeros(K, device="cuda")
    y = torch.empty_like(dy); dx = torch.empty_like(x)
    ws = torch.empty(max(256, max(B.conv_workspace_bytes(d, i) for i in range(3))), dtype=torch.uint8, device="cuda")
    passes = [("fwd", B.PASS_FWD, lambda: B.conv_fwd(d, x, w, bias, y, B.ACT_RELU, ws))]
    if C >= 4:
        passes.append(("bwd_data", B.PASS_BWD_DATA, lambda: B.conv_bwd_data(d, dy, w, None, dx, ws)))
    rows = []
    for pname, pid, fn in passes:
        B.reset_tuning()
        B.set_tuning("SELECT", 0)                      # the launcher's measured rules
        default_desc = B.conv_plan_describe(d, pid)
        results = {}
        results[_cfg_of(default_desc)] = (_time(fn, reps, flush), _pred_clk(default_desc))
        B.set_tuning("SELECT", 1)                      # the cost model's choice (the default for convolutions)
        model_desc = B.conv_plan_describe(d, pid)
        if _cfg_of(model_desc) not in results:
            results[_cfg_of(model_desc)] = (_time(fn, reps, flush), _pred_clk(model_desc))
        for tiling in ("plain", "halo0", "halo1", "halo2"):
            for bn in (64, 128, 256):
                if bn > max(64, (K + 31) // 32 * 32 if pid == B.PASS_FWD else (C + 31) // 32 * 32):
                    continue
                for pair in (0, 1):
                    B.reset_tuning()
                    B.set_tuning("TILING", tiling); B.set_tuning("BN", bn)
                    B.set_tuning("PAIR" if tiling == "plain" else "PAIR_HALO", pair)
                    desc = B.conv_plan_describe(d, pid)
                    cfg = _cfg_of(desc)
                    if cfg in results:
                        continue            # (an impossible candidate falls back to one already measured)
                    results[cfg] = (_time(fn, reps, flush), _pred_clk(desc))
        B.reset_tuning()
        st = B.last_device_status()
        if st != B.OK:
            raise SystemExit(f"device status {st} in {name} {pname}")
        rows.append((name, pname, _cfg_of(default_desc), _cfg_of(model_desc), results))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--minibatch", type=int, default=256)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--layers", default="vgga", choices=["vgga", "overfeat"])
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the search measures on a GPU")
    gen = torch.Generator(device="cuda"); gen.manual_seed(160206709)
    flush = torch.empty(64 << 20, device="cuda")
    layers = VGGA if args.layers == "vgga" else OVERFEAT
    lines = [f"| layer | pass | hand rule | ms | model's choice | ms | measured best | ms | candidates (ms measured / ms predicted at 1.75 GHz) |",
             "|---|---|---|---|---|---|---|---|---|"]
    worst_rule, worst_model = 1.0, 1.0
    for name, C, K, H, R, pad in layers:
        for lname, pname, dcfg, mcfg, res in search_layer(name, args.minibatch, C, K, H, R, pad, args.reps, flush, gen):
            best = min(res, key=lambda k: res[k][0])
            cand = "; ".join(f"{k} {v[0]:.3f}/{v[1] / 1.75e6:.3f}" for k, v in sorted(res.items(), key=lambda kv: kv[1][0]))
            lines.append(f"| {lname} | {pname} | {dcfg} | {res[dcfg][0]:.3f} | {mcfg} | {res[mcfg][0]:.3f} | {best} | {res[best][0]:.3f} | {cand} |")
            worst_rule = max(worst_rule, res[dcfg][0] / res[best][0]); worst_model = max(worst_model, res[mcfg][0] / res[best][0])
            print(lines[-1], flush=True)
        torch.cuda.empty_cache()
    lines.append("")
    lines.append(f"worst ratio to the measured best: hand rule {worst_rule:.3f}, model's choice {worst_model:.3f}")
    text = "\n".join(lines)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text + "\n")
    print(lines[-1])


if __name__ == "__main__":
    main()
