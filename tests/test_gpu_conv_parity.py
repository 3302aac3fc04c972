"""GPU parity: the three convolution passes through the C ABI against the fp64
oracle, element by element, on seeded inputs.  Shapes span several tiles and
ragged tails in every tiled dimension; both kernel families are exercised."""
import numpy as np
import pytest
import torch

import gpu_helpers as G
import oracle
from oracle import ConvShape

pytestmark = pytest.mark.gpu

TENSOR_SHAPES = {
    "cfg1": ConvShape(N=4, C=16, K=32, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1),
    "ragged": ConvShape(N=3, C=40, K=72, H=19, W=23, R=3, S=3, pad_h=1, pad_w=1),
    "k5_nopad": ConvShape(N=2, C=32, K=64, H=24, W=24, R=5, S=5),
    "one_by_one": ConvShape(N=5, C=64, K=128, H=9, W=9, R=1, S=1),
    "wide_k": ConvShape(N=4, C=64, K=320, H=12, W=12, R=3, S=3, pad_h=1, pad_w=1),
    "deep_c": ConvShape(N=2, C=288, K=48, H=14, W=14, R=3, S=3, pad_h=1, pad_w=1),
    "rect_kernel": ConvShape(N=2, C=24, K=40, H=10, W=17, R=2, S=3, pad_h=1, pad_w=0),
    "many_pixels": ConvShape(N=6, C=32, K=32, H=56, W=56, R=3, S=3, pad_h=1, pad_w=1),
}
FEW_CHANNEL_SHAPES = {   # C < 4, stride 1: staged 4-channel copy + overlapping TMA windows
    "rgb": ConvShape(N=2, C=3, K=16, H=20, W=20, R=3, S=3, pad_h=1, pad_w=1),
    "rgb_big": ConvShape(N=3, C=3, K=64, H=40, W=36, R=3, S=3, pad_h=1, pad_w=1),
    "gray_5x5": ConvShape(N=2, C=1, K=24, H=17, W=19, R=5, S=5, pad_h=2, pad_w=2),
    "two_ch_nopad": ConvShape(N=2, C=2, K=36, H=12, W=15, R=3, S=2),
    "rgb_7x7_pad": ConvShape(N=1, C=3, K=8, H=14, W=14, R=7, S=7, pad_h=3, pad_w=1),
}
# Strided layers on the tensor cores: forward and weight gradient fetch every stride-th pixel by TMA, backward-data
# runs one stride-1 sub-convolution per phase of the input grid; few-channel layers with kernel rows wider than one
# 32-float window (S > 8) take taps 8 pixels apart.
STRIDED_SHAPES = {
    "rgb_stride4": ConvShape(N=2, C=3, K=24, H=47, W=47, R=11, S=11, stride_h=4, stride_w=4),
    "stride2": ConvShape(N=3, C=20, K=36, H=15, W=18, R=3, S=3, stride_h=2, stride_w=2, pad_h=1, pad_w=1),
    "mixed_stride": ConvShape(N=2, C=8, K=12, H=16, W=16, R=3, S=5, stride_h=1, stride_w=2, pad_h=0, pad_w=2),
    "stride2_wide": ConvShape(N=4, C=64, K=96, H=30, W=34, R=3, S=3, stride_h=2, stride_w=2, pad_h=1, pad_w=1),
    "stride3_k2": ConvShape(N=2, C=16, K=32, H=20, W=23, R=2, S=2, stride_h=3, stride_w=3),   # pixels no tap reaches
    "stride4_k5_pad2": ConvShape(N=2, C=32, K=64, H=33, W=29, R=5, S=5, stride_h=4, stride_w=4, pad_h=2, pad_w=2),
    "stride2x3_k3x4": ConvShape(N=2, C=24, K=40, H=26, W=31, R=3, S=4, stride_h=2, stride_w=3, pad_h=1, pad_w=2),
    "rgb_11x11_s1": ConvShape(N=1, C=3, K=16, H=24, W=26, R=11, S=11),
    "gray_s2": ConvShape(N=2, C=1, K=20, H=21, W=22, R=3, S=3, stride_h=2, stride_w=2, pad_h=1, pad_w=1),
    "rgb_9x17_s2": ConvShape(N=2, C=3, K=12, H=40, W=45, R=9, S=17, stride_h=2, stride_w=2, pad_h=4, pad_w=8),
}
GENERIC_SHAPES = {
    "odd_channels": ConvShape(N=2, C=7, K=9, H=11, W=13, R=3, S=3, pad_h=1, pad_w=1),
}


def _cases():
    from paper_1602_06709_b200 import binding as B
    out = []
    for tag, s in TENSOR_SHAPES.items():
        out.append(pytest.param(tag, s, B.PATH_TENSOR, id=f"tensor-{tag}"))
        out.append(pytest.param(tag, s, B.PATH_GENERIC, id=f"generic-{tag}"))
    for tag, s in FEW_CHANNEL_SHAPES.items():
        out.append(pytest.param(tag, s, B.PATH_AUTO, id=f"few-{tag}"))
        out.append(pytest.param(tag, s, B.PATH_GENERIC, id=f"generic-{tag}"))
    for tag, s in STRIDED_SHAPES.items():
        out.append(pytest.param(tag, s, B.PATH_TENSOR, id=f"tensor-{tag}"))     # (forced: a fallback would be refused)
        out.append(pytest.param(tag, s, B.PATH_GENERIC, id=f"generic-{tag}"))
    for tag, s in GENERIC_SHAPES.items():
        out.append(pytest.param(tag, s, B.PATH_AUTO, id=f"auto-{tag}"))
    return out


@pytest.fixture
def path_guard():
    from paper_1602_06709_b200 import binding as B
    yield
    B.set_path(B.PATH_AUTO)


@pytest.mark.parametrize("tag,s,path", _cases())
def test_conv_three_passes(tag, s, path, path_guard):
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(path)
    x, w, dy, bias = G.make_inputs(s, tag)
    # forward, fused bias + ReLU
    y = G.run_conv_fwd(s, x, w, bias, B.ACT_RELU)
    G.assert_parity(y, oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), "fwd relu")
    y = G.run_conv_fwd(s, x, w, None, B.ACT_NONE)
    G.assert_parity(y, oracle.conv_fwd(s, x, w), "fwd plain")
    # backward data, with and without the fused ReLU mask
    dx = G.run_conv_bwd_data(s, dy, w, None)
    G.assert_parity(dx, oracle.conv_bwd_data(s, dy, w), "bwd_data")
    dx = G.run_conv_bwd_data(s, dy, w, x)
    ref = oracle.conv_bwd_data(s, dy, w, x)
    G.assert_parity(dx, ref, "bwd_data masked")
    assert np.array_equal(dx == 0, ref == 0) or np.count_nonzero((dx == 0) != (ref == 0)) < 1e-4 * dx.size
    # weight gradient: deterministic two-pass and atomic variants, with bias gradient
    dw_ref, db_ref = oracle.conv_bwd_weights(s, x, dy, want_db=True)
    dw, db = G.run_conv_bwd_weights(s, x, dy, True, deterministic=True)
    G.assert_parity(dw, dw_ref, "bwd_weights")
    G.assert_parity(db, db_ref, "dbias")
    dw2, _ = G.run_conv_bwd_weights(s, x, dy, True, deterministic=True)
    assert np.array_equal(dw, dw2), "two-pass weight gradient must be bitwise reproducible"
    dw3, _ = G.run_conv_bwd_weights(s, x, dy, False, deterministic=False)
    G.assert_parity(dw3, dw_ref, "bwd_weights atomics")


def test_cfg1_with_sgd_update():
    """Config 1 end to end: fwd, bwd_data, bwd_weights, then w <- w - 0.01*dw."""
    import torch
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    c = inputs.CFG1
    s = ConvShape(N=c["N"], C=c["C"], K=c["K"], H=c["H"], W=c["W"], R=c["R"], S=c["S"], pad_h=c["pad"], pad_w=c["pad"])
    x, w, dy = inputs.conv_inputs("cfg1", "conv", s.N, s.C, s.H, s.W, s.K, s.R, s.S, s.P, s.Q, "unit")
    bias = np.zeros(s.K, dtype=np.float32)
    y = G.run_conv_fwd(s, x, w, bias, B.ACT_NONE)
    G.assert_parity(y, oracle.conv_fwd(s, x, w, bias), "fwd")
    dx = G.run_conv_bwd_data(s, dy, w, None)
    G.assert_parity(dx, oracle.conv_bwd_data(s, dy, w), "bwd_data")
    dw, _ = G.run_conv_bwd_weights(s, x, dy, False)
    dw_ref = oracle.conv_bwd_weights(s, x, dy)
    G.assert_parity(dw, dw_ref, "bwd_weights")
    wt = G.dev(w)
    B.sgd_update(wt, G.dev(dw), 0.01)
    # the update itself is exact fp32 arithmetic on the GPU's own dw
    ref = oracle.sgd_update(w, dw, 0.01)
    np.testing.assert_allclose(wt.cpu().numpy(), ref, rtol=0, atol=1e-7)
    G.assert_parity(wt.cpu().numpy(), oracle.sgd_update(w, dw_ref, 0.01), "updated weights")


HALO_SHAPES = {
    "fits_16x16": ConvShape(N=3, C=64, K=64, H=32, W=48, R=3, S=3, pad_h=1, pad_w=1),       # two boxes side by side
    "fits_8x32": ConvShape(N=2, C=32, K=128, H=64, W=24, R=3, S=3, pad_h=1, pad_w=1),
    "ragged": ConvShape(N=2, C=96, K=40, H=21, W=19, R=3, S=3, pad_h=1, pad_w=1),
    "k5": ConvShape(N=2, C=32, K=32, H=20, W=20, R=5, S=5, pad_h=2, pad_w=2),
    "wide": ConvShape(N=2, C=64, K=256, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1),              # BN = 256: one box only
}


@pytest.mark.parametrize("tiling", ["plain", "halo0", "halo1", "halo2", "halo1_pair", "halo2_pair"])
@pytest.mark.parametrize("tag", sorted(HALO_SHAPES))
def test_forward_type_kernel_every_tiling(tag, tiling, path_guard, monkeypatch):
    """The forward-type kernel has a plain tiling and three haloed ones (taps as row-shifted views of one
    input patch), the haloed ones also as CTA pairs over two images; the TILING and PAIR_HALO knobs pin one.  All must
    agree with the oracle for forward and backward-data (shapes whose tile width or weight layout does not allow a
    pair run as single CTAs)."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    if tiling.endswith("_pair"):
        tiling = tiling[:-5]
        B.set_tuning("PAIR_HALO", 1)
    B.set_tuning("TILING", tiling)
    B.set_path(B.PATH_TENSOR)
    s = HALO_SHAPES[tag]
    x, w, dy, bias = G.make_inputs(s, "halo_" + tag)
    y = G.run_conv_fwd(s, x, w, bias, B.ACT_RELU)
    G.assert_parity(y, oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), f"fwd {tiling}")
    dx = G.run_conv_bwd_data(s, dy, w, x)
    G.assert_parity(dx, oracle.conv_bwd_data(s, dy, w, x), f"bwd_data {tiling}")


PIPELINE_SHAPES = {
    # several image groups per tile row, so that CTA pairs form; an odd group count leaves one pair half empty
    "odd_groups": ConvShape(N=6, C=64, K=96, H=28, W=28, R=3, S=3, pad_h=1, pad_w=1),
    "even_groups_wide": ConvShape(N=8, C=128, K=256, H=14, W=14, R=3, S=3, pad_h=1, pad_w=1),
    "fc_like": ConvShape(N=384, C=192, K=320, H=1, W=1, R=1, S=1),
    "ragged_c": ConvShape(N=5, C=72, K=48, H=20, W=20, R=3, S=3, pad_h=1, pad_w=1),     # C % 32 != 0: no grouped copies
}


@pytest.mark.parametrize("variant", ["pair0", "pair1_ks1", "pair1_ks2_nogroup", "pair1_ks2_group", "pair0_ks2_group"])
@pytest.mark.parametrize("tag", sorted(PIPELINE_SHAPES))
def test_forward_type_kernel_pipeline_variants(tag, variant, path_guard, monkeypatch):
    """The plain tiling runs as single CTAs or CTA pairs (one M = 256 MMA over two tiles), with one or
    two k-steps per pipeline slot fetched by one copy per k-step or one per slot.  Every combination
    must agree with the oracle (forward with the fused epilogue, backward-data with mask and fused
    bias gradient path left to the network tests)."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    env = {"pair0": dict(PAIR="0", KS="1"), "pair1_ks1": dict(PAIR="1", KS="1"),
           "pair1_ks2_nogroup": dict(PAIR="1", KS="2", GRP="0"),
           "pair1_ks2_group": dict(PAIR="1", KS="2", GRP="1"),
           "pair0_ks2_group": dict(PAIR="0", KS="2", GRP="1")}[variant]
    for k, v in env.items():
        B.set_tuning(k, v)
    B.set_tuning("TILING", "plain")
    B.set_path(B.PATH_TENSOR)
    s = PIPELINE_SHAPES[tag]
    x, w, dy, bias = G.make_inputs(s, "pipe_" + tag)
    y = G.run_conv_fwd(s, x, w, bias, B.ACT_RELU)
    G.assert_parity(y, oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), f"fwd {variant}")
    dx = G.run_conv_bwd_data(s, dy, w, x)
    G.assert_parity(dx, oracle.conv_bwd_data(s, dy, w, x), f"bwd_data {variant}")
    assert B.last_device_status() == 0


@pytest.mark.parametrize("tiling", ["plain", "halo0", "halo1", "halo2", "auto"])
@pytest.mark.parametrize("tag", sorted(PIPELINE_SHAPES))
def test_forward_with_sixteen_epilogue_warps(tag, tiling, path_guard, monkeypatch):
    """Launches with a very short reduction run sixteen epilogue warps instead of eight (four per TMEM lane
    quarter share a tile's 32-column chunks).  the EPI_WARPS knob = 32 forces that variant wherever it can run: the
    result must equal the eight-warp variant's bit for bit (same accumulators, same epilogue arithmetic)."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_tuning("TILING", tiling)
    B.set_tuning("PAIR", "0")
    B.set_tuning("SPLIT_ACC", "0")
    B.set_path(B.PATH_TENSOR)
    s = PIPELINE_SHAPES[tag]
    x, w, dy, bias = G.make_inputs(s, "epi16_" + tag)
    res = {}
    for warps in ("8", "32"):
        B.set_tuning("EPI_WARPS", warps)
        res[warps] = G.run_conv_fwd(s, x, w, bias, B.ACT_RELU)
    G.assert_parity(res["32"], oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), f"fwd {tiling}")
    assert np.array_equal(res["8"], res["32"])
    assert B.last_device_status() == 0


XHALO_SHAPES = {
    # single-CTA weight-gradient items (odd number of 128-map tiles), few input maps, S > 1
    "c64_k128": ConvShape(N=3, C=64, K=128, H=28, W=28, R=3, S=3, pad_h=1, pad_w=1),
    "ragged_q": ConvShape(N=2, C=64, K=96, H=13, W=21, R=3, S=3, pad_h=1, pad_w=1),
    "c32_5x5_nopad": ConvShape(N=2, C=32, K=64, H=20, W=24, R=5, S=5),
    "rect_pad2": ConvShape(N=5, C=32, K=40, H=9, W=16, R=2, S=3, pad_h=0, pad_w=2),
    "three_k_tiles": ConvShape(N=2, C=64, K=320, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1),
    "row_kernel": ConvShape(N=4, C=64, K=128, H=10, W=40, R=1, S=3, pad_h=0, pad_w=1),
    "wide_box": ConvShape(N=2, C=64, K=64, H=6, W=64, R=3, S=3, pad_h=1, pad_w=1),
}


@pytest.mark.parametrize("pix", ["64", "32"])
@pytest.mark.parametrize("tag", sorted(XHALO_SHAPES))
def test_weight_gradient_with_haloed_input_boxes(tag, pix, path_guard, monkeypatch):
    """Layers with few input maps fetch one haloed input box per k-step and take the S taps of a kernel row as
    row-shifted views of it (one MMA over 32*S columns); the XHALO_WGRAD knob = 0 keeps one box per tap.  Both must agree
    with the oracle; the two-pass result must repeat bit for bit."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(B.PATH_TENSOR)
    B.set_tuning("PIX_WGRAD", pix)
    s = XHALO_SHAPES[tag]
    x, w, dy, _ = G.make_inputs(s, "xhalo_" + tag)
    dw_ref, db_ref = oracle.conv_bwd_weights(s, x, dy, want_db=True)
    for mode in ("1", "0"):
        B.set_tuning("XHALO_WGRAD", mode)
        dw, db = G.run_conv_bwd_weights(s, x, dy, True, deterministic=True)
        G.assert_parity(dw, dw_ref, f"bwd_weights xhalo={mode}")
        G.assert_parity(db, db_ref, "dbias")
        dw2, _ = G.run_conv_bwd_weights(s, x, dy, False, deterministic=True)
        assert np.array_equal(dw, dw2)
        dw3, _ = G.run_conv_bwd_weights(s, x, dy, False, deterministic=False)
        G.assert_parity(dw3, dw_ref, f"bwd_weights atomics xhalo={mode}")
    assert B.last_device_status() == 0


@pytest.mark.parametrize("tiling", ["plain", "halo1", "auto"])
@pytest.mark.parametrize("tag", ["odd_groups", "even_groups_wide", "fc_like"])
def test_backward_data_reads_weights_in_place(tag, tiling, path_guard, monkeypatch):
    """Backward-data takes the KRSC weights as an MN-major operand (taps flipped by index) when the layer's
    input-map count is a multiple of 32; the WEIGHTS_IN_PLACE knob = 0 forces the flipped, transposed copy.  Same
    products, same order of additions: the two must agree bit for bit, and with the oracle."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_tuning("TILING", tiling)
    B.set_path(B.PATH_TENSOR)
    s = PIPELINE_SHAPES[tag]
    x, w, dy, _ = G.make_inputs(s, "inplace_" + tag)
    B.set_tuning("WEIGHTS_IN_PLACE", "1")
    dx1 = G.run_conv_bwd_data(s, dy, w, x)
    B.set_tuning("WEIGHTS_IN_PLACE", "0")
    dx0 = G.run_conv_bwd_data(s, dy, w, x)
    G.assert_parity(dx1, oracle.conv_bwd_data(s, dy, w, x), "bwd_data in place")
    assert np.array_equal(dx0, dx1)
    assert B.last_device_status() == 0


@pytest.mark.parametrize("mode", ["solo", "ordered", "split"])
@pytest.mark.parametrize("tag", ["fits_16x16", "fits_8x32", "k5"])
def test_two_issuers_keep_results_reproducible(tag, mode, path_guard, monkeypatch):
    """Narrow single-CTA tiles may run two MMA-issuing threads: either ordered by a sequence number (the
    additions then happen in the order of one issuer: bit-identical to it) or with an accumulator each that
    the epilogue adds (a different, but fixed, order).  Every mode must match the oracle and repeat itself
    bit for bit; the ordered mode must equal the single issuer exactly."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    env = {"solo": dict(ISSUERS="1"), "ordered": dict(ISSUERS="2", SPLIT_ACC="0"),
           "split": dict(ISSUERS="2", SPLIT_ACC="1")}
    B.set_path(B.PATH_TENSOR)
    s = HALO_SHAPES[tag]
    x, w, dy, bias = G.make_inputs(s, "issuers_" + tag)

    def run(m):
        for k in ("ISSUERS", "SPLIT_ACC"):
            B.set_tuning(k, None)
        for k, v in env[m].items():
            B.set_tuning(k, v)
        return G.run_conv_fwd(s, x, w, bias, B.ACT_RELU), G.run_conv_bwd_data(s, dy, w, x)

    y, dx = run(mode)
    G.assert_parity(y, oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), f"fwd {mode}")
    G.assert_parity(dx, oracle.conv_bwd_data(s, dy, w, x), f"bwd_data {mode}")
    y2, dx2 = run(mode)
    assert np.array_equal(y, y2) and np.array_equal(dx, dx2)
    if mode == "ordered":
        y1, dx1 = run("solo")
        assert np.array_equal(y, y1) and np.array_equal(dx, dx1)
    assert B.last_device_status() == 0


def test_two_issuer_backward_data_repeats_bit_for_bit(path_guard):
    """Regression: a 96-map backward-data launch (plain tiling, three pipeline stages, two issuers with an
    accumulator each) once lost slot releases and summed wrongly when one issuer could overtake the other.
    Twenty repetitions must finish without a device-side timeout and agree bit for bit."""
    import torch
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    B.set_path(B.PATH_TENSOR)
    s = ConvShape(N=64, C=96, K=256, H=24, W=24, R=5, S=5)
    x, w, dy, _ = G.make_inputs(s, "two_issuer_regression")
    d = G.shape_to_desc(s)
    dyt, wt, xt = G.dev(dy), G.dev(w), G.dev(x)
    ws = G.workspace(B.conv_workspace_bytes(d, B.PASS_BWD_DATA))
    first = None
    for _ in range(20):
        dx = torch.empty(s.N, s.H, s.W, s.C, device="cuda")
        B.conv_bwd_data(d, dyt, wt, xt, dx, ws)
        B.check_device_status()
        if first is None:
            first = dx
            G.assert_parity(dx.cpu().numpy(), oracle.conv_bwd_data(s, dy, w, x), "bwd_data")
        else:
            assert torch.equal(first, dx)


POOLED_WGRAD_SHAPES = {
    # few-channel first layers with even outputs: ragged boxes in q and p, several images per box, R != S, K > 128
    "rgb": ConvShape(N=2, C=3, K=16, H=20, W=36, R=3, S=3, pad_h=1, pad_w=1),
    "rgb_k64": ConvShape(N=3, C=3, K=64, H=40, W=36, R=3, S=3, pad_h=1, pad_w=1),
    "gray_5x5": ConvShape(N=2, C=1, K=24, H=18, W=20, R=5, S=5, pad_h=2, pad_w=2),
    "two_ch_nopad": ConvShape(N=5, C=2, K=36, H=12, W=15, R=3, S=2),
    "rgb_k160": ConvShape(N=2, C=3, K=160, H=8, W=8, R=3, S=3, pad_h=1, pad_w=1),
    "tiny_maps": ConvShape(N=9, C=3, K=8, H=4, W=6, R=3, S=3, pad_h=1, pad_w=1),
}


@pytest.mark.parametrize("relu", [True, False])
@pytest.mark.parametrize("tag", sorted(POOLED_WGRAD_SHAPES))
def test_weight_gradient_from_pooled_gradient(tag, relu, path_guard):
    """pcl_conv_bwd_weights_pooled: the weight gradient of a pooled first layer straight from the pooled gradient and
    the windows' position codes (the kernel builds its dy tiles on chip).  Reference: the oracle's code-routed
    pooling backward pass followed by the oracle's weight gradient."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    s = POOLED_WGRAD_SHAPES[tag]
    d = G.shape_to_desc(s)
    assert B.conv_bwd_weights_pooled_is_fused(d)
    x, _, _, _ = G.make_inputs(s, "pooled_" + tag)
    P2, Q2 = s.P // 2, s.Q // 2
    dyp = inputs.normal(inputs.tensor_id("pooled_wgrad", tag, "dyp"), (s.N, P2, Q2, s.K), 1.0)
    codes = (inputs.uniform(inputs.tensor_id("pooled_wgrad", tag, "codes"), (s.N, P2, Q2, s.K), 0.0, 8.0)
             .astype(np.int64).clip(0, 7).astype(np.uint8))
    dy = oracle.maxpool2x2_bwd_codes(codes, dyp, relu).astype(np.float32)
    dw_ref, db_ref = oracle.conv_bwd_weights(s, x, dy, want_db=True)
    ws = G.workspace(B.conv_bwd_weights_pooled_workspace_bytes(d))
    outs = []
    for _ in range(2):
        dw = G.guarded((s.K, s.R, s.S, s.C))
        db = G.guarded((s.K,))
        B.conv_bwd_weights_pooled(d, G.dev(x), G.dev(dyp), torch.from_numpy(codes).cuda(), relu, dw, db, ws)
        B.check_device_status()
        outs.append((dw.cpu().numpy(), db.cpu().numpy()))
    G.assert_parity(outs[0][0], dw_ref, "dw from pooled dy")
    G.assert_parity(outs[0][1], db_ref, "db from pooled dy")
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    # without the bias gradient
    dw2 = G.guarded((s.K, s.R, s.S, s.C))
    B.conv_bwd_weights_pooled(d, G.dev(x), G.dev(dyp), torch.from_numpy(codes).cuda(), relu, dw2, None, ws)
    B.check_device_status()
    assert np.array_equal(dw2.cpu().numpy(), outs[0][0])
    # from the staged input that the layer's forward call leaves at the start of its workspace: bit for bit the same
    n_staged = B.conv_staged_input_bytes(d)
    assert n_staged > 0
    ws_f = G.workspace(B.conv_workspace_bytes(d, B.PASS_FWD))
    assert ws_f.numel() >= n_staged
    w = inputs.normal(inputs.tensor_id("pooled_wgrad", tag, "w"), (s.K, s.R, s.S, s.C), 0.3)
    B.conv_fwd(d, G.dev(x), G.dev(w), None, G.guarded((s.N, s.P, s.Q, s.K)), B.ACT_RELU, ws_f)
    dw3 = G.guarded((s.K, s.R, s.S, s.C)); db3 = G.guarded((s.K,))
    B.conv_bwd_weights_pooled_staged(d, ws_f, G.dev(dyp), torch.from_numpy(codes).cuda(), relu, dw3, db3, ws)
    B.check_device_status()
    assert np.array_equal(dw3.cpu().numpy(), outs[0][0]) and np.array_equal(db3.cpu().numpy(), outs[0][1])


def test_weight_gradient_from_pooled_gradient_only_where_fused():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    s = ConvShape(N=2, C=32, K=32, H=8, W=8, R=3, S=3, pad_h=1, pad_w=1)       # not a few-channel layer
    d = G.shape_to_desc(s)
    assert not B.conv_bwd_weights_pooled_is_fused(d)
    z = lambda *shape: torch.zeros(*shape, device="cuda")
    with pytest.raises(B.PclError) as e:
        B.conv_bwd_weights_pooled(d, z(2, 8, 8, 32), z(2, 4, 4, 32), torch.zeros(2, 4, 4, 32, dtype=torch.uint8, device="cuda"),
                                  True, z(32, 3, 3, 32), None, G.workspace(1 << 20))
    assert e.value.code == B.ERR_UNSUPPORTED_SHAPE


@pytest.mark.parametrize("form", ["packed", "phases"])
@pytest.mark.parametrize("tag", sorted(STRIDED_SHAPES))
def test_strided_backward_data_both_forms(tag, form, path_guard):
    """Backward-data of a strided layer runs either as one stride-1 convolution whose output maps are (phase, input
    map) pairs followed by a scatter (layers with stride_h * stride_w * C <= 256), or as one launch per phase
    (the PACKED_BWD knob = 0 forces that form): both against the oracle, with and without the ReLU mask."""
    from paper_1602_06709_b200 import binding as B
    s = STRIDED_SHAPES[tag]
    if s.stride_h == 1 and s.stride_w == 1:
        pytest.skip("stride-1 layer")
    B.set_path(B.PATH_TENSOR)
    B.set_tuning("PACKED_BWD", 1 if form == "packed" else 0)
    x, w, dy, _ = G.make_inputs(s, "strided_bwd_" + tag)
    G.assert_parity(G.run_conv_bwd_data(s, dy, w, None), oracle.conv_bwd_data(s, dy, w), f"bwd_data {form}")
    G.assert_parity(G.run_conv_bwd_data(s, dy, w, x), oracle.conv_bwd_data(s, dy, w, x), f"bwd_data {form} masked")
