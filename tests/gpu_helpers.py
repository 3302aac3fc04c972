"""Helpers for the GPU parity tests: run one pass through the C ABI on seeded
inputs and compare with the fp64 oracle under the stated tolerance."""
import numpy as np
import torch

import oracle
from oracle import ConvShape
from paper_1602_06709_b200 import binding as B
from paper_1602_06709_b200 import inputs

# Tolerance of the parity bar: relative L2 <= 2e-3 and max-abs <= 1e-2 * RMS(reference), per tensor.
REL_L2_TOL = 2e-3
MAX_OVER_RMS_TOL = 1e-2


def dev(a, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda", dtype=dtype)


def assert_parity(got, ref, what):
    rel, mx = oracle.parity_errors(got, ref)
    assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"{what}: rel_l2={rel:.3e} max/rms={mx:.3e}"
    return rel, mx


def workspace(nbytes):
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda") if nbytes else None


def shape_to_desc(s: ConvShape):
    return B.ConvDesc(s.N, s.C, s.K, s.H, s.W, s.R, s.S, s.stride_h, s.stride_w, s.pad_h, s.pad_w)


def make_inputs(s: ConvShape, tag, kind="unit"):
    x, w, dy = inputs.conv_inputs("test", tag, s.N, s.C, s.H, s.W, s.K, s.R, s.S, s.P, s.Q, kind)
    bias = inputs.uniform(inputs.tensor_id("test", tag, "bias"), (s.K,), -0.5, 0.5)
    return x, w, dy, bias


def run_conv_fwd(s, x, w, bias, act):
    d = shape_to_desc(s)
    y = torch.full((s.N, s.P, s.Q, s.K), float("nan"), device="cuda")
    B.conv_fwd(d, dev(x), dev(w), None if bias is None else dev(bias), y, act,
               workspace(B.conv_workspace_bytes(d, B.PASS_FWD)))
    B.check_device_status()
    return y.cpu().numpy()


def run_conv_bwd_data(s, dy, w, mask):
    d = shape_to_desc(s)
    dx = torch.full((s.N, s.H, s.W, s.C), float("nan"), device="cuda")
    B.conv_bwd_data(d, dev(dy), dev(w), None if mask is None else dev(mask), dx,
                    workspace(B.conv_workspace_bytes(d, B.PASS_BWD_DATA)))
    B.check_device_status()
    return dx.cpu().numpy()


def run_conv_bwd_weights(s, x, dy, want_db, deterministic=True):
    d = shape_to_desc(s)
    dw = torch.full((s.K, s.R, s.S, s.C), float("nan"), device="cuda")
    db = torch.full((s.K,), float("nan"), device="cuda") if want_db else None
    B.conv_bwd_weights(d, dev(x), dev(dy), dw, db, deterministic,
                       workspace(B.conv_workspace_bytes(d, B.PASS_BWD_WEIGHTS)))
    B.check_device_status()
    return dw.cpu().numpy(), (db.cpu().numpy() if want_db else None)
