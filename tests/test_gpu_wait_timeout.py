"""The give-up path of the bounded device-side waits, taken once, safely.

Every wait in the tensor-core kernels polls for a limited time; a wait that runs
out records which role gave up, raises the CTA's abort flag, and the kernel
tears down (TMEM freed) and returns.  Here a host-selected test mode makes the
producer of one tiny single-CTA launch arm its first pipeline slot for 16 bytes
more than it copies, with the wait limit shortened to 2 ms: nothing faults or
spins without limit, the kernel returns by itself, the status call reports the
timeout once, and the next ordinary launch is correct."""
import time

import numpy as np
import pytest
import torch

import oracle
from oracle import ConvShape

pytestmark = pytest.mark.gpu

WAIT_MMA_FULL, WAIT_EPI_TMEM_FULL = 0x102, 0x104


def _timed_out_launch(run, what):
    from paper_1602_06709_b200 import binding as B
    assert B.last_device_status() == B.OK
    t0 = time.perf_counter()
    run()
    status = B.last_device_status()                 # synchronises: the kernel has returned by itself
    elapsed = time.perf_counter() - t0
    assert status == B.ERR_DEVICE_TIMEOUT, f"{what}: status {status}"
    assert B.last_wait_code() in (WAIT_MMA_FULL, WAIT_EPI_TMEM_FULL), hex(B.last_wait_code())
    assert elapsed < 1.0, f"{what}: gave up only after {elapsed:.2f} s with a 2 ms limit"
    assert B.last_device_status() == B.OK           # reported once, then cleared
    assert B.status_string(status) == "device-side wait timed out"


def test_forward_kernel_gives_up_and_the_context_stays_usable():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(B.PATH_TENSOR)
    s = ConvShape(N=1, C=64, K=32, H=8, W=8, R=1, S=1)          # one tile, one CTA, one pipeline slot
    x, w, dy, bias = G.make_inputs(s, "timeout_fwd")
    try:
        B.set_tuning("WAIT_LIMIT_US", 2000)
        B.set_tuning("FAULT_INJECT", 1)
        d = G.shape_to_desc(s)
        y = torch.zeros(s.N, s.P, s.Q, s.K, device="cuda")
        xt, wt, bt = G.dev(x), G.dev(w), G.dev(bias)
        _timed_out_launch(lambda: B.conv_fwd(d, xt, wt, bt, y, B.ACT_RELU, None), "forward")
    finally:
        B.reset_tuning()
        B.set_path(B.PATH_AUTO)
    # the same launch without the injection: correct, and no status left behind
    B.set_path(B.PATH_TENSOR)
    try:
        G.assert_parity(G.run_conv_fwd(s, x, w, bias, B.ACT_RELU), oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), "fwd after timeout")
    finally:
        B.set_path(B.PATH_AUTO)
    assert B.last_device_status() == B.OK


def test_weight_gradient_kernel_gives_up_and_the_context_stays_usable():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(B.PATH_TENSOR)
    s = ConvShape(N=1, C=32, K=32, H=8, W=8, R=3, S=3, pad_h=1, pad_w=1)      # one k-step per work item
    x, w, dy, _ = G.make_inputs(s, "timeout_wgrad")
    try:
        B.set_tuning("WAIT_LIMIT_US", 2000)
        B.set_tuning("FAULT_INJECT", 2)
        d = G.shape_to_desc(s)
        dw = torch.zeros(s.K, s.R, s.S, s.C, device="cuda")
        ws = G.workspace(B.conv_workspace_bytes(d, B.PASS_BWD_WEIGHTS))
        xt, dyt = G.dev(x), G.dev(dy)
        _timed_out_launch(lambda: B.conv_bwd_weights(d, xt, dyt, dw, None, True, ws), "weight gradient")
    finally:
        B.reset_tuning()
        B.set_path(B.PATH_AUTO)
    B.set_path(B.PATH_TENSOR)
    try:
        dw2, _ = G.run_conv_bwd_weights(s, x, dy, False)
        G.assert_parity(dw2, oracle.conv_bwd_weights(s, x, dy), "bwd_weights after timeout")
    finally:
        B.set_path(B.PATH_AUTO)
    assert B.last_device_status() == B.OK
