"""Pins for the convolution oracle: each test checks it against something other
than itself (literal transcription in the paper's own index order, invariants,
finite differences, special cases, a library routine)."""
import itertools
import os

import numpy as np
import pytest

import oracle
from oracle import ConvShape

RNG = np.random.default_rng(1234)

TINY = [
    ConvShape(N=2, C=3, K=4, H=5, W=6, R=3, S=3, stride_h=1, stride_w=1, pad_h=1, pad_w=1),
    ConvShape(N=1, C=2, K=3, H=7, W=5, R=3, S=2, stride_h=2, stride_w=2, pad_h=0, pad_w=1),
    ConvShape(N=2, C=1, K=1, H=9, W=9, R=5, S=5, stride_h=4, stride_w=4, pad_h=2, pad_w=2),
    ConvShape(N=1, C=2, K=2, H=2, W=3, R=3, S=3, stride_h=1, stride_w=1, pad_h=2, pad_w=1),  # R > H
    ConvShape(N=2, C=3, K=2, H=6, W=4, R=1, S=1),
    ConvShape(N=1, C=2, K=3, H=8, W=7, R=2, S=3, stride_h=3, stride_w=2, pad_h=1, pad_w=0),
]


def rand_case(d, dtype=np.float64):
    x = RNG.uniform(-1, 1, (d.N, d.H, d.W, d.C)).astype(dtype)
    w = RNG.uniform(-1, 1, (d.K, d.R, d.S, d.C)).astype(dtype)
    dy = RNG.uniform(-1, 1, (d.N, d.P, d.Q, d.K)).astype(dtype)
    b = RNG.uniform(-1, 1, d.K).astype(dtype)
    return x, w, dy, b


# ---------------------------------------------------------------------------
# 1. literal transcription of the 7-nested loop in the paper's index order:
#    tensors N,C,H,W; weights IFM,OFM,KH,KW; scatter form for backprop.
# ---------------------------------------------------------------------------
def paper_loops(d, x_nchw, w_iokk, dy_nkpq):
    out = np.zeros((d.N, d.K, d.P, d.Q))
    gin = np.zeros((d.N, d.C, d.H, d.W))
    gw = np.zeros((d.C, d.K, d.R, d.S))
    for i0, i1, i2, i3, i4, i5, i6 in itertools.product(
            range(d.N), range(d.C), range(d.K), range(d.P), range(d.Q), range(d.R), range(d.S)):
        h = i3 * d.stride_h + i5 - d.pad_h
        ww = i4 * d.stride_w + i6 - d.pad_w
        if not (0 <= h < d.H and 0 <= ww < d.W):
            continue
        out[i0, i2, i3, i4] += x_nchw[i0, i1, h, ww] * w_iokk[i1, i2, i5, i6]
        gin[i0, i1, h, ww] += dy_nkpq[i0, i2, i3, i4] * w_iokk[i1, i2, i5, i6]
        gw[i1, i2, i5, i6] += x_nchw[i0, i1, h, ww] * dy_nkpq[i0, i2, i3, i4]
    return out, gin, gw


@pytest.mark.parametrize("d", TINY)
def test_brute_force_paper_index_order(d):
    x, w, dy, _ = rand_case(d)
    out, gin, gw = paper_loops(d, x.transpose(0, 3, 1, 2), w.transpose(3, 0, 1, 2), dy.transpose(0, 3, 1, 2))
    y = oracle.conv_fwd(d, x, w)
    dx = oracle.conv_bwd_data(d, dy, w)
    dw = oracle.conv_bwd_weights(d, x, dy)
    np.testing.assert_allclose(y, out.transpose(0, 2, 3, 1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dx, gin.transpose(0, 2, 3, 1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dw, gw.transpose(1, 2, 3, 0), rtol=0, atol=1e-12)


@pytest.mark.parametrize("d", TINY[:3])
def test_f32_instantiation_matches_f64_on_f32_values(d):
    x, w, dy, b = rand_case(d, np.float32)
    for a32, a64 in [
        (oracle.conv_fwd(d, x, w, b, oracle.ACT_RELU),
         oracle.conv_fwd(d, x.astype(np.float64), w.astype(np.float64), b.astype(np.float64), oracle.ACT_RELU)),
        (oracle.conv_bwd_data(d, dy, w), oracle.conv_bwd_data(d, dy.astype(np.float64), w.astype(np.float64))),
        (oracle.conv_bwd_weights(d, x, dy), oracle.conv_bwd_weights(d, x.astype(np.float64), dy.astype(np.float64))),
    ]:
        np.testing.assert_array_equal(a32, a64)


# ---------------------------------------------------------------------------
# 2. adjoint identities <dy, conv(x,w)> = <bwd_data(dy,w), x> = <bwd_weights(x,dy), w>
# ---------------------------------------------------------------------------
ADJ_SHAPES = TINY + [
    ConvShape(N=4, C=16, K=32, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1),             # config 1
    ConvShape(N=1, C=256, K=256, H=56, W=56, R=3, S=3, pad_h=1, pad_w=1),           # config 2, N reduced
    ConvShape(N=1, C=3, K=96, H=231, W=231, R=11, S=11, stride_h=4, stride_w=4),    # OverFeat C1, N reduced
    ConvShape(N=2, C=96, K=256, H=24, W=24, R=5, S=5),
    ConvShape(N=2, C=256, K=512, H=12, W=12, R=3, S=3, pad_h=1, pad_w=1),
    ConvShape(N=1, C=3, K=64, H=224, W=224, R=3, S=3, pad_h=1, pad_w=1),            # VGG-A conv1
    ConvShape(N=8, C=440, K=2048, H=1, W=1, R=1, S=1),                              # DNN layer 1
]


@pytest.mark.parametrize("d", ADJ_SHAPES)
def test_adjoint_identities(d):
    x, w, dy, _ = rand_case(d)
    a = np.vdot(dy, oracle.conv_fwd(d, x, w))
    b = np.vdot(oracle.conv_bwd_data(d, dy, w), x)
    c = np.vdot(oracle.conv_bwd_weights(d, x, dy), w)
    scale = max(abs(a), 1e-30)
    assert abs(a - b) / scale < 1e-11
    assert abs(a - c) / scale < 1e-11


# ---------------------------------------------------------------------------
# 3. finite differences of L = <dy, act(conv(x,w)+b)>
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("d", TINY[:4])
@pytest.mark.parametrize("act", [oracle.ACT_NONE, oracle.ACT_SIGMOID])
def test_finite_differences(d, act):
    x, w, dy, b = rand_case(d)

    def loss(x_, w_, b_):
        return float(np.vdot(dy, oracle.conv_fwd(d, x_, w_, b_, act)))

    y = oracle.conv_fwd(d, x, w, b, act)
    dz = oracle.act_grad(y, dy, act)
    dx = oracle.conv_bwd_data(d, dz, w)
    dw, db = oracle.conv_bwd_weights(d, x, dz, want_db=True)
    h = 1e-6
    for arr, grad, which in [(x, dx, 0), (w, dw, 1), (b, db, 2)]:
        flat = arr.reshape(-1)
        for i in RNG.choice(flat.size, size=min(6, flat.size), replace=False):
            old = flat[i]
            flat[i] = old + h; lp = loss(x, w, b)
            flat[i] = old - h; lm = loss(x, w, b)
            flat[i] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - grad.reshape(-1)[i]) < 1e-7 * max(1.0, abs(fd)), (which, i)


def test_relu_mask_on_bwd_data():
    d = TINY[0]
    x, w, dy, _ = rand_case(d)
    plain = oracle.conv_bwd_data(d, dy, w)
    masked = oracle.conv_bwd_data(d, dy, w, relu_mask_src=x)
    np.testing.assert_array_equal(masked, np.where(x > 0, plain, 0.0))
    assert (x <= 0).any() and (x > 0).any()


# ---------------------------------------------------------------------------
# 4. special cases that reduce to library / textbook routines
# ---------------------------------------------------------------------------
def test_1x1_conv_is_a_matrix_product():
    d = ConvShape(N=3, C=7, K=5, H=4, W=6, R=1, S=1)
    x, w, dy, b = rand_case(d)
    y = oracle.conv_fwd(d, x, w, b)
    np.testing.assert_allclose(y.reshape(-1, d.K), x.reshape(-1, d.C) @ w.reshape(d.K, d.C).T + b, atol=1e-13)
    dx = oracle.conv_bwd_data(d, dy, w)
    np.testing.assert_allclose(dx.reshape(-1, d.C), dy.reshape(-1, d.K) @ w.reshape(d.K, d.C), atol=1e-13)
    dw = oracle.conv_bwd_weights(d, x, dy)
    np.testing.assert_allclose(dw.reshape(d.K, d.C), dy.reshape(-1, d.K).T @ x.reshape(-1, d.C), atol=1e-13)


def test_fc_is_the_1x1_special_case():
    N, C, K = 9, 13, 6
    x = RNG.normal(size=(N, C)); w = RNG.normal(size=(K, C)); b = RNG.normal(size=K); dy = RNG.normal(size=(N, K))
    y = oracle.fc_fwd(x, w, b, oracle.ACT_SIGMOID)
    z = x @ w.T + b
    np.testing.assert_allclose(y, 1 / (1 + np.exp(-z)), atol=1e-14)
    dz, dx, dw, db = oracle.fc_bwd(x, w, y, dy, oracle.ACT_SIGMOID, dz_dtype=np.float64)
    dz_ref = dy * y * (1 - y)
    np.testing.assert_allclose(dz, dz_ref, atol=1e-15)
    np.testing.assert_allclose(dx, dz_ref @ w, atol=1e-13)
    np.testing.assert_allclose(dw, dz_ref.T @ x, atol=1e-13)
    np.testing.assert_allclose(db, dz_ref.sum(0), atol=1e-13)


def test_delta_kernel_is_a_shift():
    d = ConvShape(N=1, C=2, K=2, H=6, W=7, R=3, S=3, pad_h=1, pad_w=1)
    x = RNG.normal(size=(1, 6, 7, 2))
    w = np.zeros((2, 3, 3, 2))
    w[0, 0, 2, 0] = 1.0     # y[..,0](p,q) = x[..,0](p-1, q+1)
    w[1, 2, 1, 1] = 1.0     # y[..,1](p,q) = x[..,1](p+1, q)
    y = oracle.conv_fwd(d, x, w)
    ref = np.zeros_like(y)
    ref[0, 1:, :-1, 0] = x[0, :-1, 1:, 0]
    ref[0, :-1, :, 1] = x[0, 1:, :, 1]
    np.testing.assert_array_equal(y, ref)


def test_all_ones_counts_valid_taps():
    d = ConvShape(N=1, C=5, K=2, H=6, W=5, R=3, S=3, pad_h=1, pad_w=1)
    y = oracle.conv_fwd(d, np.ones((1, 6, 5, 5)), np.ones((2, 3, 3, 5)))
    rows = np.array([2, 3, 3, 3, 3, 2]); cols = np.array([2, 3, 3, 3, 2])
    ref = d.C * rows[:, None] * cols[None, :]
    np.testing.assert_array_equal(y[0, :, :, 0], ref)
    np.testing.assert_array_equal(y[0, :, :, 1], ref)


@pytest.mark.parametrize("d", TINY + [ConvShape(N=2, C=8, K=6, H=12, W=12, R=5, S=5, pad_h=2, pad_w=2)])
def test_against_torch_float64_conv2d_and_autograd(d):
    torch = pytest.importorskip("torch")
    import torch.nn.functional as F
    x, w, dy, b = rand_case(d)
    xt = torch.tensor(x.transpose(0, 3, 1, 2).copy(), requires_grad=True)
    wt = torch.tensor(w.transpose(0, 3, 1, 2).copy(), requires_grad=True)
    bt = torch.tensor(b, requires_grad=True)
    yt = F.conv2d(xt, wt, bt, stride=(d.stride_h, d.stride_w), padding=(d.pad_h, d.pad_w))
    yt.backward(torch.tensor(dy.transpose(0, 3, 1, 2).copy()))
    np.testing.assert_allclose(oracle.conv_fwd(d, x, w, b), yt.detach().numpy().transpose(0, 2, 3, 1), atol=1e-12)
    np.testing.assert_allclose(oracle.conv_bwd_data(d, dy, w), xt.grad.numpy().transpose(0, 2, 3, 1), atol=1e-12)
    dw, db = oracle.conv_bwd_weights(d, x, dy, want_db=True)
    np.testing.assert_allclose(dw, wt.grad.numpy().transpose(0, 2, 3, 1), atol=1e-12)
    np.testing.assert_allclose(db, bt.grad.numpy(), atol=1e-12)


@pytest.mark.parametrize("d", TINY[:3])
def test_sampled_entry_points_agree_with_full(d):
    x, w, dy, b = rand_case(d, np.float32)
    for full, fn in [
        (oracle.conv_fwd(d, x, w, b, oracle.ACT_RELU), lambda at: oracle.conv_fwd(d, x, w, b, oracle.ACT_RELU, at=at)),
        (oracle.conv_bwd_data(d, dy, w, x), lambda at: oracle.conv_bwd_data(d, dy, w, x, at=at)),
        (oracle.conv_bwd_weights(d, x, dy), lambda at: oracle.conv_bwd_weights(d, x, dy, at=at)),
    ]:
        at = RNG.choice(full.size, size=min(17, full.size), replace=False)
        np.testing.assert_array_equal(fn(at), full.reshape(-1)[at])


# ---------------------------------------------------------------------------
# 5. bookkeeping closed forms printed in the paper
# ---------------------------------------------------------------------------
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_bytes_per_flop_worked_example():
    for out_h, out_w, k_h, k_w, s, size, printed, digits in _rows("bf_ratio_sec2_2.txt"):
        out_h, out_w, k_h, k_w, s, size = map(int, (out_h, out_w, k_h, k_w, s, size))
        in_h, in_w = out_h * s + k_h - 1, out_w * s + k_w - 1
        d = ConvShape(N=1, C=1, K=1, H=in_h, W=in_w, R=k_h, S=k_w, stride_h=s, stride_w=s)
        assert (d.P, d.Q) == (out_h, out_w)
        bf = size * (d.P * d.Q + d.H * d.W + d.R * d.S) / d.flops()
        assert round(bf, int(digits)) == float(printed)


def test_output_dims_and_flop_count():
    for H, R, st, pad, P in _rows("flops_sec3_1.txt"):
        H, R, st, pad, P = map(int, (H, R, st, pad, P))
        d = ConvShape(N=2, C=3, K=5, H=H, W=H, R=R, S=R, stride_h=st, stride_w=st, pad_h=pad, pad_w=pad)
        assert d.P == P and d.Q == P
        assert 3 * d.flops() == 3 * 2 * d.N * d.C * d.K * R * R * P * P
    # flops() counts exactly the multiply-adds the literal loop executes when nothing is clipped
    d = ConvShape(N=1, C=2, K=3, H=6, W=6, R=3, S=3)
    n_macs = sum(1 for _ in itertools.product(range(d.N), range(d.C), range(d.K), range(d.P), range(d.Q),
                                              range(d.R), range(d.S)))
    assert d.flops() == 2 * n_macs
