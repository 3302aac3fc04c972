"""GPU parity for the fully-connected passes, the SGD update and the glue
kernels (max-pool, softmax cross-entropy), through the C ABI, against the oracle."""
import numpy as np
import pytest
import torch

import gpu_helpers as G
import oracle
from oracle import ConvShape

pytestmark = pytest.mark.gpu

FC_CASES = [
    # N, C, K, act            (ragged in every dimension; K > 256 spans several column tiles)
    (96, 960, 264, "relu"),      # 30 channel blocks: reduction splits of 3 and 5 divide the slots
    (256, 1920, 128, "sigmoid"),
    (130, 440, 200, "sigmoid"),
    (64, 96, 520, "relu"),
    (257, 36, 1000, "none"),
    (8, 2052, 64, "sigmoid"),
    (300, 32, 32, "none"),
    (132, 64, 264, "relu"),     # minibatch not a multiple of 32: ragged reduction of the forward-form weight gradient
]


@pytest.fixture
def path_guard():
    from paper_1602_06709_b200 import binding as B
    yield
    B.set_path(B.PATH_AUTO)


@pytest.mark.parametrize("N,C,K,act", FC_CASES)
@pytest.mark.parametrize("path", ["tensor", "tensor_dw_forward_form", "tensor_dw_wgrad_form", "generic"])
def test_fc_fwd_bwd(N, C, K, act, path, path_guard, monkeypatch):
    """The FC weight gradient has two forms on the tensor path: the weight-gradient kernel, or (short reductions,
    C % 32 == 0) the forward-type kernel over dz^T with x read in place as an MN-major operand;
    the FC_DW_FORWARD knob pins one."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    if path.startswith("tensor_dw"):
        B.set_tuning("FC_DW_FORWARD", "1" if "forward" in path else "0")
    B.set_path(B.PATH_GENERIC if path == "generic" else B.PATH_TENSOR)
    code = {"none": B.ACT_NONE, "relu": B.ACT_RELU, "sigmoid": B.ACT_SIGMOID}[act]
    tid = lambda r: inputs.tensor_id("fc", N, C, K, r)
    x = inputs.normal(tid("x"), (N, C), 1.0)
    w = inputs.xavier_uniform_fc(tid("w"), K, C)
    b = inputs.uniform(tid("b"), (K,), -0.5, 0.5)
    dy = inputs.normal(tid("dy"), (N, K), 1.0)
    xt, wt, bt = G.dev(x), G.dev(w), G.dev(b)
    yt = G.guarded((N, K))
    B.fc_fwd(N, C, K, xt, wt, bt, yt, code)
    B.check_device_status()
    y = yt.cpu().numpy()
    G.assert_parity(y, oracle.fc_fwd(x, w, b, code), "fc fwd")
    # with scratch the launcher may split the reduction over more CTAs (few tiles, long reduction); the KSPLIT knob pins
    # the number of splits where it divides the reduction's pipeline slots
    for ks in ("0", "2", "3", "5"):
        B.set_tuning("KSPLIT", ks)
        ws_f = G.workspace(B.fc_workspace_bytes(N, C, K, B.PASS_FWD))
        yt2 = G.guarded((N, K))
        B.fc_fwd(N, C, K, xt, wt, bt, yt2, code, ws_f)
        B.check_device_status()
        G.assert_parity(yt2.cpu().numpy(), oracle.fc_fwd(x, w, b, code), f"fc fwd, KSPLIT={ks}")
    B.set_tuning("KSPLIT", None)
    # backward is checked on the GPU's own forward output (per-call parity)
    dyt = G.dev(dy)
    dxt = G.guarded((N, C))
    dwt = G.guarded((K, C))
    dbt = G.guarded((K,))
    ws = G.workspace(B.fc_workspace_bytes(N, C, K, B.PASS_BWD_DATA))
    B.fc_bwd(N, C, K, xt, wt, yt, code, dyt, dxt, dwt, dbt, ws)
    B.check_device_status()
    dz_ref, dx_ref, dw_ref, db_ref = oracle.fc_bwd(x, w, y, dy, code, dz_dtype=np.float32)
    np.testing.assert_allclose(dyt.cpu().numpy(), dz_ref, rtol=1e-5, atol=1e-7)     # dz written back into dy
    dz_gpu = dyt.cpu().numpy()
    # contractions are checked against the oracle fed the GPU's own dz
    sh = oracle.ConvShape(N=N, C=C, K=K, H=1, W=1, R=1, S=1)
    G.assert_parity(dxt.cpu().numpy(), oracle.conv_bwd_data(sh, dz_gpu, w), "fc dx")
    dw_o, db_o = oracle.conv_bwd_weights(sh, x, dz_gpu, want_db=True)
    G.assert_parity(dwt.cpu().numpy(), dw_o, "fc dw")
    G.assert_parity(dbt.cpu().numpy(), db_o, "fc db")
    # first-layer form: dx skipped
    dyt2 = G.dev(dy)
    dwt2 = torch.empty_like(dwt)
    B.fc_bwd(N, C, K, xt, wt, yt, code, dyt2, None, dwt2, None, ws)
    B.check_device_status()
    assert torch.equal(dwt2, dwt)


@pytest.mark.parametrize("n", [0, 1, 3, 4, 1000, 4097, 1 << 20, (1 << 20) + 3])
def test_sgd_update(n):
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    w = inputs.normal(inputs.tensor_id("sgd", n, "w"), (n,), 1.0)
    dw = inputs.normal(inputs.tensor_id("sgd", n, "dw"), (n,), 1.0)
    wt = torch.from_numpy(w).cuda(); dwt = torch.from_numpy(dw).cuda()
    if n == 0:
        B.sgd_update(wt, dwt, 0.01)
        return
    B.sgd_update(wt, dwt, 0.01)
    ref = oracle.sgd_update(w, dw, 0.01)
    # one fused multiply-add in fp32: within half an ulp of the exact value
    got = wt.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= np.spacing(np.abs(ref).astype(np.float32)).astype(np.float64) * 0.5 + 1e-30)


def test_sgd_update_unaligned_views():
    from paper_1602_06709_b200 import binding as B
    base_w = torch.randn(1001, device="cuda"); base_g = torch.randn(1001, device="cuda")
    w = base_w[1:]; g = base_g[1:]                       # 4-byte aligned only
    ref = oracle.sgd_update(w.cpu().numpy(), g.cpu().numpy(), 0.5)
    B.sgd_update(w, g, 0.5)
    np.testing.assert_allclose(w.cpu().numpy(), ref, rtol=1e-6, atol=1e-7)


@pytest.mark.parametrize("N,H,W,C", [(2, 8, 6, 8), (3, 14, 14, 5), (1, 2, 2, 1), (2, 28, 28, 64)])
def test_maxpool(N, H, W, C):
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    x = np.maximum(inputs.normal(inputs.tensor_id("pool", N, H, W, C, "x"), (N, H, W, C), 1.0), 0.0)  # post-ReLU: has ties at 0
    dy = inputs.normal(inputs.tensor_id("pool", N, H, W, C, "dy"), (N, H // 2, W // 2, C), 1.0)
    xt, dyt = G.dev(x), G.dev(dy)
    yt = G.guarded((N, H // 2, W // 2, C))
    B.maxpool2x2_fwd(N, H, W, C, xt, yt)
    assert np.array_equal(yt.cpu().numpy(), oracle.maxpool2x2_fwd(x).astype(np.float32))
    dxt = G.guarded((N, H, W, C))
    B.maxpool2x2_bwd(N, H, W, C, xt, dyt, None, dxt)
    assert np.array_equal(dxt.cpu().numpy(), oracle.maxpool2x2_bwd(x, dy).astype(np.float32))
    B.maxpool2x2_bwd(N, H, W, C, xt, dyt, xt, dxt)
    assert np.array_equal(dxt.cpu().numpy(), oracle.maxpool2x2_bwd(x, dy, x).astype(np.float32))


@pytest.mark.parametrize("N,K", [(4, 10), (37, 1000), (256, 1000), (64, 8192), (1, 3), (5, 2048), (5, 2049), (3, 9000)])
def test_softmax_xent(N, K):
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    z = inputs.normal(inputs.tensor_id("xent", N, K, "z"), (N, K), 3.0)
    lab = inputs.labels(inputs.tensor_id("xent", N, K, "lab"), N, K)
    zt = G.dev(z); lt = torch.from_numpy(lab).cuda()
    loss = G.guarded((1,))
    dz = G.guarded((N, K))
    B.softmax_xent(N, K, zt, lt, loss, dz)
    loss_ref, dz_ref = oracle.softmax_xent(z, lab)
    assert abs(loss.item() - loss_ref) <= 1e-5 * max(1.0, abs(loss_ref))
    G.assert_parity(dz.cpu().numpy(), dz_ref, "dlogits")
    np.testing.assert_allclose(dz.cpu().numpy(), dz_ref, rtol=1e-4, atol=1e-8)


@pytest.mark.parametrize("x_act", ["none", "relu", "sigmoid"])
@pytest.mark.parametrize("N,C,K", [(96, 960, 264), (130, 440, 200), (64, 96, 520), (256, 2048, 2048), (33, 36, 40), (8, 30, 12)])
def test_fc_bwd_fused_epilogue(N, C, K, x_act, path_guard):
    """pcl_fc_bwd_fused: backpropagation with the gradient of the activation that produced x and the column sums of dx
    (the layer below's dz and bias gradient) formed in the kernel's epilogue, against the oracle's chain rule."""
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    code = {"none": B.ACT_NONE, "relu": B.ACT_RELU, "sigmoid": B.ACT_SIGMOID}[x_act]
    pre = inputs.normal(inputs.tensor_id("fcf", N, C, K, "pre"), (N, C), 1.0).astype(np.float64)
    x = {"none": pre, "relu": np.maximum(pre, 0.0), "sigmoid": 1.0 / (1.0 + np.exp(-pre))}[x_act].astype(np.float32)
    w = inputs.normal(inputs.tensor_id("fcf", N, C, K, "w"), (K, C), (1.0 / C) ** 0.5)
    dz = inputs.normal(inputs.tensor_id("fcf", N, C, K, "dz"), (N, K), 1.0)
    xt, wt = G.dev(x), G.dev(w)
    for want_cs in (True, False):
        dzt = G.dev(dz)
        dx = G.guarded((N, C)); dw = G.guarded((K, C)); db = G.guarded((K,))
        cs = G.guarded((C,)) if want_cs else None
        ws = G.workspace(B.fc_workspace_bytes(N, C, K, B.PASS_BWD_DATA))
        B.fc_bwd_fused(N, C, K, xt, wt, None, B.ACT_NONE, dzt, dx, code, cs, dw, db, ws)
        B.check_device_status()
        G.check_guards()
        _, dx_ref, dw_ref, db_ref = oracle.fc_bwd(x, w, None, dz, oracle.ACT_NONE, dz_dtype=np.float32)
        xd = x.astype(np.float64)
        g = {"none": 1.0, "relu": (xd > 0).astype(np.float64), "sigmoid": xd * (1.0 - xd)}[x_act]
        G.assert_parity(dx.cpu().numpy(), dx_ref * g, f"dx times {x_act}'")
        G.assert_parity(dw.cpu().numpy(), dw_ref, "dw")
        G.assert_parity(db.cpu().numpy(), db_ref, "db")
        if want_cs:
            # the sums are of the values the kernel wrote (per-call parity of the reduction itself)
            G.assert_parity(cs.cpu().numpy(), dx.cpu().numpy().astype(np.float64).sum(axis=0), "column sums of dx")
            cs2 = G.guarded((C,)); dx2 = G.guarded((N, C))
            B.fc_bwd_fused(N, C, K, xt, wt, None, B.ACT_NONE, G.dev(dz), dx2, code, cs2, dw, db, ws)
            assert torch.equal(cs, cs2) and torch.equal(dx, dx2), "fused sums must be bitwise reproducible"


def test_softmax_xent_label_outside_the_classes_is_reported_and_never_used_as_an_index():
    """A label outside [0, K) must not become an address: the row gets no target and no loss term, and the status
    call reports it once."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    N, K = 6, 40
    z = inputs.normal(inputs.tensor_id("xent_bad", N, K, "z"), (N, K), 2.0)
    lab = np.array([3, -1, K, 17, K + 1000, 0], dtype=np.int32)
    good = (lab >= 0) & (lab < K)
    zt = G.dev(z); lt = torch.from_numpy(lab).cuda()
    loss = G.guarded((1,))
    dz = G.guarded((N, K))
    assert B.last_device_status() == B.OK
    B.softmax_xent(N, K, zt, lt, loss, dz)
    assert B.last_device_status() == B.ERR_BAD_LABEL
    assert B.last_device_status() == B.OK                      # reported once, then cleared
    loss_ref, dz_ref = oracle.softmax_xent(z, np.where(good, lab, 0))
    zs = z.astype(np.float64) - z.max(axis=1, keepdims=True)
    sm = np.exp(zs) / np.exp(zs).sum(axis=1, keepdims=True)
    dz_ref[~good] = sm[~good] / N                              # no one-hot on the rows without a target
    terms = -(zs[np.arange(N), np.where(good, lab, 0)] - np.log(np.exp(zs).sum(axis=1)))
    np.testing.assert_allclose(dz.cpu().numpy(), dz_ref, rtol=1e-4, atol=1e-8)
    assert abs(loss.item() - terms[good].sum() / N) <= 1e-5


@pytest.mark.parametrize("N,H,W,C", [(2, 8, 6, 8), (3, 14, 14, 20), (2, 28, 28, 64), (1, 4, 4, 1024)])
def test_maxpool_bwd_with_fused_column_sums(N, H, W, C):
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    x = np.maximum(inputs.normal(inputs.tensor_id("poolcs", N, H, W, C, "x"), (N, H, W, C), 1.0), 0.0)
    dy = inputs.normal(inputs.tensor_id("poolcs", N, H, W, C, "dy"), (N, H // 2, W // 2, C), 1.0)
    xt, dyt = G.dev(x), G.dev(dy)
    dxt = G.guarded((N, H, W, C))
    cs = G.guarded((C,))
    ws = G.workspace(B.maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C))
    B.maxpool2x2_bwd_colsum(N, H, W, C, xt, dyt, xt, dxt, cs, ws)
    ref = oracle.maxpool2x2_bwd(x, dy, x)
    assert np.array_equal(dxt.cpu().numpy(), ref.astype(np.float32))
    G.assert_parity(cs.cpu().numpy(), ref.reshape(-1, C).sum(axis=0), "pool dx column sums")
    cs2 = torch.empty_like(cs)
    B.maxpool2x2_bwd_colsum(N, H, W, C, xt, dyt, xt, dxt, cs2, ws)
    assert torch.equal(cs, cs2)


@pytest.mark.parametrize("tiling", ["auto", "plain", "halo1"])
@pytest.mark.parametrize("shape", [(3, 40, 72, 19, 23), (2, 64, 64, 32, 32), (2, 128, 320, 12, 12), (2, 7, 9, 11, 13),
                                   # more tiles than SMs (a CTA keeps its column sums over several tiles); dx wider than one
                                   # tile (tiles differ in their columns: one row of sums per tile)
                                   (16, 32, 48, 40, 40), (2, 320, 64, 12, 12)])
def test_conv_bwd_data_with_fused_column_sums(shape, tiling, monkeypatch):
    import gpu_helpers as G
    from oracle import ConvShape
    from paper_1602_06709_b200 import binding as B
    if tiling != "auto":
        B.set_tuning("TILING", tiling)
    N, C, K, H, W = shape
    s = ConvShape(N=N, C=C, K=K, H=H, W=W, R=3, S=3, pad_h=1, pad_w=1)
    x, w, dy, _ = G.make_inputs(s, f"dgradcs{C}")
    d = G.shape_to_desc(s)
    dx = G.guarded((N, H, W, C))
    cs = G.guarded((C,))
    ws = G.workspace(B.conv_bwd_data_colsum_workspace_bytes(d))
    B.conv_bwd_data_colsum(d, G.dev(dy), G.dev(w), G.dev(x), dx, cs, ws)
    B.check_device_status()
    ref = oracle.conv_bwd_data(s, dy, w, x)
    G.assert_parity(dx.cpu().numpy(), ref, "dx")
    # the sums are of the GPU's own dx (per-call parity), formed in fp32 in a fixed order
    G.assert_parity(cs.cpu().numpy(), dx.cpu().numpy().astype(np.float64).reshape(-1, C).sum(axis=0), "dx column sums")
    cs2 = torch.empty_like(cs)
    B.conv_bwd_data_colsum(d, G.dev(dy), G.dev(w), G.dev(x), dx, cs2, ws)
    assert torch.equal(cs, cs2)


def inputs_normal(tag, shape):
    from paper_1602_06709_b200 import inputs
    return inputs.normal(inputs.tensor_id(*tag), shape, 1.0)


POOL_FUSED_SHAPES = [
    # N, C, K, H, W: even outputs; several image groups; ragged in q/p; C < 4 (few-channel path); halo-eligible 16x16 fits
    (3, 32, 64, 12, 20), (4, 64, 96, 28, 28), (2, 3, 16, 20, 36), (2, 64, 128, 32, 48), (5, 24, 40, 6, 10), (2, 7, 9, 10, 12),
]


@pytest.mark.parametrize("store", ["tma", "direct", "tma_16_epilogue_warps"])
@pytest.mark.parametrize("tiling", ["auto", "plain", "halo0", "halo1", "halo2"])
@pytest.mark.parametrize("shape", POOL_FUSED_SHAPES)
def test_conv_fwd_with_fused_maxpool(shape, tiling, store, monkeypatch):
    """conv -> ReLU -> 2x2 max pool in one call: y must match the oracle's convolution, and the pooled
    tensor must be bit-for-bit the 2x2 maxima of the y the same call wrote (the epilogue takes the
    maximum of the raw accumulators, which commutes exactly with the bias add and the ReLU)."""
    import gpu_helpers as G
    from oracle import ConvShape
    from paper_1602_06709_b200 import binding as B
    if tiling != "auto":
        B.set_tuning("TILING", tiling)
    # the epilogue writes y either with TMA stores from its staging tiles or with per-lane coalesced stores
    B.set_tuning("TMA_STORE", "0" if store == "direct" else "1")
    # the kernel variant with sixteen epilogue warps (chosen by itself only for very short reductions), single CTAs
    B.set_tuning("EPI_WARPS", "32" if store == "tma_16_epilogue_warps" else "8")
    if store == "tma_16_epilogue_warps":
        B.set_tuning("PAIR", "0")
    N, C, K, H, W = shape
    s = ConvShape(N=N, C=C, K=K, H=H, W=W, R=3, S=3, pad_h=1, pad_w=1)
    x, w, _, bias = G.make_inputs(s, f"fwdpool{C}_{K}")
    d = G.shape_to_desc(s)
    for act, oact in ((B.ACT_RELU, oracle.ACT_RELU), (B.ACT_NONE, oracle.ACT_NONE)):
        y = G.guarded((N, H, W, K))
        yp = G.guarded((N, H // 2, W // 2, K))
        ws = G.workspace(B.conv_workspace_bytes(d, B.PASS_FWD))
        codes = G.guarded((N, H // 2, W // 2, K), torch.uint8, fill=255)
        B.conv_fwd_pool(d, G.dev(x), G.dev(w), G.dev(bias), y, yp, act, ws, pool_codes=codes)
        B.check_device_status()
        G.assert_parity(y.cpu().numpy(), oracle.conv_fwd(s, x, w, bias, oact), "y")
        yh = y.cpu().numpy()
        assert np.array_equal(yp.cpu().numpy(), oracle.maxpool2x2_fwd(yh.astype(np.float64)).astype(np.float32))
        # the position codes route a gradient exactly as the pooling backward pass does from the y this call wrote
        g = inputs_normal(("fwdpool_g", N, H, W, K), (N, H // 2, W // 2, K))
        for relu in (False, True):
            dx = G.guarded((N, H, W, K))
            B.maxpool2x2_bwd_codes(N, H, W, K, codes, G.dev(g), relu, dx)
            ref = oracle.maxpool2x2_bwd(yh, g, yh if relu else None)
            assert np.array_equal(dx.cpu().numpy(), ref.astype(np.float32))
        assert np.array_equal(codes.cpu().numpy(), oracle.maxpool2x2_codes(yh))
        # without y (where the call runs as one kernel): the same pooled tensor and codes, bit for bit
        if B.conv_fwd_pool_is_fused(d):
            yp2 = torch.full_like(yp, float("nan")); codes2 = torch.full_like(codes, 255)
            B.conv_fwd_pool(d, G.dev(x), G.dev(w), G.dev(bias), None, yp2, act, ws, pool_codes=codes2)
            B.check_device_status()
            assert torch.equal(yp2, yp) and torch.equal(codes2, codes)
            yp3 = torch.full_like(yp, float("nan"))
            B.conv_fwd_pool(d, G.dev(x), G.dev(w), G.dev(bias), None, yp3, act, ws)     # no codes either
            B.check_device_status()
            assert torch.equal(yp3, yp)


@pytest.mark.parametrize("shape", [
    ConvShape(N=3, C=16, K=32, H=24, W=40, R=3, S=3, stride_h=2, stride_w=2, pad_h=1, pad_w=1),
    ConvShape(N=2, C=3, K=24, H=47, W=55, R=11, S=11, stride_h=4, stride_w=4),      # few-channel, two windows per row
])
def test_strided_conv_fwd_with_fused_maxpool(shape):
    """A strided layer followed by the 2x2 pool, as one call: y against the oracle, the pooled tensor and the codes
    bit for bit the maxima / positions of that y, with and without storing y."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    s = shape
    assert s.P % 2 == 0 and s.Q % 2 == 0
    x, w, _, bias = G.make_inputs(s, f"fwdpool_strided{s.C}")
    d = G.shape_to_desc(s)
    assert B.conv_fwd_pool_is_fused(d)
    ws = G.workspace(B.conv_workspace_bytes(d, B.PASS_FWD))
    y = G.guarded((s.N, s.P, s.Q, s.K))
    yp = G.guarded((s.N, s.P // 2, s.Q // 2, s.K))
    codes = G.guarded((s.N, s.P // 2, s.Q // 2, s.K), torch.uint8, fill=255)
    B.conv_fwd_pool(d, G.dev(x), G.dev(w), G.dev(bias), y, yp, B.ACT_RELU, ws, pool_codes=codes)
    B.check_device_status()
    G.assert_parity(y.cpu().numpy(), oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU), "y")
    yh = y.cpu().numpy()
    assert np.array_equal(yp.cpu().numpy(), oracle.maxpool2x2_fwd(yh.astype(np.float64)).astype(np.float32))
    assert np.array_equal(codes.cpu().numpy(), oracle.maxpool2x2_codes(yh))
    yp2 = torch.full_like(yp, float("nan")); codes2 = torch.full_like(codes, 255)
    B.conv_fwd_pool(d, G.dev(x), G.dev(w), G.dev(bias), None, yp2, B.ACT_RELU, ws, pool_codes=codes2)
    B.check_device_status()
    assert torch.equal(yp2, yp) and torch.equal(codes2, codes)


def test_conv_fwd_pool_rejects_odd_output():
    import gpu_helpers as G
    from oracle import ConvShape
    from paper_1602_06709_b200 import binding as B
    s = ConvShape(N=1, C=8, K=8, H=7, W=8, R=3, S=3, pad_h=1, pad_w=1)
    d = G.shape_to_desc(s)
    x = torch.zeros(1, 7, 8, 8, device="cuda"); w = torch.zeros(8, 3, 3, 8, device="cuda")
    y = torch.zeros(1, 7, 8, 8, device="cuda"); yp = torch.zeros(1, 3, 4, 8, device="cuda")
    with pytest.raises(B.PclError):
        B.conv_fwd_pool(d, x, w, None, y, yp, B.ACT_RELU, None)


def test_conv_fwd_pool_without_y_only_where_fused():
    """A layer whose channel count is not a multiple of 4 runs the generic convolution and a separate pooling kernel,
    which reads y: y is required.  (Strided layers are on the tensor-core path and fuse the pooling.)"""
    import gpu_helpers as G
    from oracle import ConvShape
    from paper_1602_06709_b200 import binding as B
    s = ConvShape(N=1, C=7, K=8, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1)
    d = G.shape_to_desc(s)
    assert not B.conv_fwd_pool_is_fused(d)
    x = torch.zeros(1, 16, 16, 7, device="cuda"); w = torch.zeros(8, 3, 3, 7, device="cuda")
    yp = torch.zeros(1, 8, 8, 8, device="cuda")
    s2 = ConvShape(N=1, C=8, K=8, H=16, W=16, R=3, S=3, stride_h=2, stride_w=2, pad_h=1, pad_w=1)
    assert B.conv_fwd_pool_is_fused(G.shape_to_desc(s2))
    with pytest.raises(B.PclError) as e:
        B.conv_fwd_pool(d, x, w, None, None, yp, B.ACT_RELU, None)
    assert e.value.code == B.ERR_UNSUPPORTED_SHAPE
    s1 = ConvShape(N=1, C=8, K=8, H=16, W=16, R=3, S=3, pad_h=1, pad_w=1)
    assert B.conv_fwd_pool_is_fused(G.shape_to_desc(s1))


@pytest.mark.parametrize("N,H,W,C", [(2, 8, 6, 8), (3, 14, 14, 5), (2, 28, 28, 64), (1, 4, 4, 1024)])
def test_maxpool_with_position_codes(N, H, W, C):
    """Forward pooling that records each window's position code, and the backward pass that takes the codes
    instead of x: bit-exact against the oracle's pooling passes, with and without the ReLU mask and with the
    fused column sums (equal to the x-based kernel's)."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    x = np.maximum(inputs.normal(inputs.tensor_id("poolcodes", N, H, W, C, "x"), (N, H, W, C), 1.0), 0.0)  # ties at 0
    dy = inputs.normal(inputs.tensor_id("poolcodes", N, H, W, C, "dy"), (N, H // 2, W // 2, C), 1.0)
    xt, dyt = G.dev(x), G.dev(dy)
    yt = G.guarded((N, H // 2, W // 2, C))
    codes = G.guarded((N, H // 2, W // 2, C), torch.uint8, fill=255)
    B.maxpool2x2_fwd_codes(N, H, W, C, xt, yt, codes)
    assert np.array_equal(yt.cpu().numpy(), oracle.maxpool2x2_fwd(x).astype(np.float32))
    assert int(codes.max()) <= 7
    for relu in (False, True):
        dxt = G.guarded((N, H, W, C))
        B.maxpool2x2_bwd_codes(N, H, W, C, codes, dyt, relu, dxt)
        ref = oracle.maxpool2x2_bwd(x, dy, x if relu else None)
        assert np.array_equal(dxt.cpu().numpy(), ref.astype(np.float32))
    cs = G.guarded((C,))
    ws = G.workspace(B.maxpool2x2_bwd_colsum_workspace_bytes(N, H, W, C))
    dxt = G.guarded((N, H, W, C))
    B.maxpool2x2_bwd_codes(N, H, W, C, codes, dyt, True, dxt, cs, ws)
    ref = oracle.maxpool2x2_bwd(x, dy, x)
    assert np.array_equal(dxt.cpu().numpy(), ref.astype(np.float32))
    G.assert_parity(cs.cpu().numpy(), ref.reshape(-1, C).sum(axis=0), "pool dx column sums")
    cs_x = torch.empty_like(cs)
    B.maxpool2x2_bwd_colsum(N, H, W, C, xt, dyt, xt, dxt, cs_x, ws)
    assert torch.equal(cs, cs_x)


# ---- the SGD step applied by the weight gradient's own second pass / epilogue (Sec. 3.1) -----------------------------
SGD_CONV_SHAPES = [
    # N, C, K, H, W, R: a split pixel reduction (the update rides on its second pass); a reduction too short to split
    # (dw goes through the scratch); the few-channel staged path; a strided layer
    (8, 64, 96, 28, 28, 3), (2, 32, 32, 6, 6, 3), (4, 3, 16, 20, 20, 3), (4, 16, 24, 19, 19, 5),
]


@pytest.mark.parametrize("N,C,K,H,W,R", SGD_CONV_SHAPES)
def test_conv_bwd_weights_sgd_equals_gradient_then_update(N, C, K, H, W, R):
    """pcl_conv_bwd_weights_sgd: w - lr * dw with dw never stored must equal, bit for bit, the deterministic weight
    gradient followed by pcl_sgd_update, and agree with the oracle's gradient and update."""
    import gpu_helpers as G
    from oracle import ConvShape
    from paper_1602_06709_b200 import binding as B
    stride = 2 if R == 5 else 1
    s = ConvShape(N=N, C=C, K=K, H=H, W=W, R=R, S=R, pad_h=R // 2, pad_w=R // 2, stride_h=stride, stride_w=stride)
    x, w, dy, _ = G.make_inputs(s, f"wsgd{C}_{K}")
    d = G.shape_to_desc(s)
    lr = 0.0625
    xt, dyt = G.dev(x), G.dev(dy)
    w_two = G.dev(w).clone(); dw = G.guarded(w.shape); db = G.guarded((K,))
    ws = G.workspace(B.conv_workspace_bytes(d, B.PASS_BWD_WEIGHTS))
    B.conv_bwd_weights(d, xt, dyt, dw, db, True, ws)
    B.sgd_update(w_two, dw, lr)
    w_one = G.guarded(w.shape); w_one.copy_(G.dev(w)); db2 = G.guarded((K,))
    ws2 = G.workspace(B.conv_bwd_weights_sgd_workspace_bytes(d))
    B.conv_bwd_weights_sgd(d, xt, dyt, w_one, lr, db2, ws2)
    B.check_device_status()
    G.check_guards()
    assert torch.equal(w_one, w_two), "fused update differs from gradient + update"
    assert torch.equal(db, db2)
    dw_ref = oracle.conv_bwd_weights(s, x, dy)
    G.assert_parity((G.dev(w) - w_one).cpu().numpy() / lr, dw_ref, "(w_old - w_new) / lr against the oracle's dw")


@pytest.mark.parametrize("N,C,K", [(64, 4096, 2048), (256, 512, 384), (96, 440, 2048), (1024, 256, 256)])
@pytest.mark.parametrize("x_act", ["none", "sigmoid"])
def test_fc_bwd_fused_sgd_equals_backward_then_update(N, C, K, x_act):
    """pcl_fc_bwd_fused_sgd (both forms of the FC weight gradient: the forward-type GEMM whose epilogue applies the
    update, and the weight-gradient kernel with the update in its second pass or after its scratch): dx, column sums and
    bias gradient as pcl_fc_bwd_fused on the OLD weights, the new weights bit-equal to the two-call form."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    code = {"none": B.ACT_NONE, "sigmoid": B.ACT_SIGMOID}[x_act]
    pre = inputs.normal(inputs.tensor_id("fcsgd", N, C, K, "pre"), (N, C), 1.0).astype(np.float64)
    x = {"none": pre, "sigmoid": 1.0 / (1.0 + np.exp(-pre))}[x_act].astype(np.float32)
    w = inputs.normal(inputs.tensor_id("fcsgd", N, C, K, "w"), (K, C), (1.0 / C) ** 0.5)
    dz = inputs.normal(inputs.tensor_id("fcsgd", N, C, K, "dz"), (N, K), 1.0)
    lr = 0.03125
    xt = G.dev(x)
    # two calls
    w_two = G.dev(w).clone()
    dx = G.guarded((N, C)); dw = G.guarded((K, C)); db = G.guarded((K,)); cs = G.guarded((C,))
    ws = G.workspace(B.fc_workspace_bytes(N, C, K, B.PASS_BWD_DATA))
    B.fc_bwd_fused(N, C, K, xt, w_two, None, B.ACT_NONE, G.dev(dz), dx, code, cs, dw, db, ws)
    B.sgd_update(w_two, dw, lr)
    # one call
    w_one = G.guarded((K, C)); w_one.copy_(G.dev(w))
    dx1 = G.guarded((N, C)); db1 = G.guarded((K,)); cs1 = G.guarded((C,))
    ws1 = G.workspace(B.fc_bwd_fused_sgd_workspace_bytes(N, C, K))
    B.fc_bwd_fused_sgd(N, C, K, xt, w_one, None, B.ACT_NONE, G.dev(dz), dx1, code, cs1, lr, db1, ws1)
    B.check_device_status()
    G.check_guards()
    assert torch.equal(dx, dx1) and torch.equal(cs, cs1) and torch.equal(db, db1)
    assert torch.equal(w_one, w_two), "fused update differs from backward + update"
    _, _, dw_ref, _ = oracle.fc_bwd(x, w, None, dz, oracle.ACT_NONE, dz_dtype=np.float32)
    G.assert_parity((G.dev(w) - w_one).cpu().numpy() / lr, dw_ref, "(w_old - w_new) / lr against the oracle's dw")
