"""GPU parity at the full workload sizes, in the launch configuration the
benchmark times.  The oracle cannot produce whole tensors at these sizes in
seconds, so each output tensor is checked on sampled elements the oracle
computes one by one (uniformly random ones plus, for every dimension, elements
from its first and last entries: boundary tiles, the last image, the last
output maps), plus properties that hold at any size (bitwise
reproducibility of the two-pass weight gradient)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import ConvShape

pytestmark = pytest.mark.gpu

SAMPLES = 192


def _sampled_three_passes(s, cfg, layer, samples=SAMPLES, skip_bwd_data=False):
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs
    rng = np.random.default_rng(7)
    x, w, dy = inputs.conv_inputs(cfg, layer, s.N, s.C, s.H, s.W, s.K, s.R, s.S, s.P, s.Q, "train")
    bias = inputs.uniform(inputs.tensor_id(cfg, layer, "bias"), (s.K,), -0.1, 0.1)
    d = G.shape_to_desc(s)
    xt, wt, dyt, bt = G.dev(x), G.dev(w), G.dev(dy), G.dev(bias)
    ws = G.workspace(max(B.conv_workspace_bytes(d, i) for i in range(3)))

    def check(t, ref_fn, what):
        flat = t.reshape(-1)
        idx = G.sample_indices(t.shape, samples, rng)       # random + first / last entries of every dimension
        got = flat[torch.from_numpy(idx).cuda()].cpu().numpy()
        G.assert_parity(got, ref_fn(idx), f"{layer} {what}")

    y = torch.empty(s.N, s.P, s.Q, s.K, device="cuda")
    B.conv_fwd(d, xt, wt, bt, y, B.ACT_RELU, ws)
    B.check_device_status()
    check(y, lambda at: oracle.conv_fwd(s, x, w, bias, oracle.ACT_RELU, at=at), "fwd")
    # ReLU zeroes about half of the outputs: make sure the sample saw both kinds
    del y
    dw = torch.empty(s.K, s.R, s.S, s.C, device="cuda")
    db = torch.empty(s.K, device="cuda")
    B.conv_bwd_weights(d, xt, dyt, dw, db, True, ws)
    B.check_device_status()
    check(dw, lambda at: oracle.conv_bwd_weights(s, x, dy, at=at), "bwd_weights")
    G.assert_parity(db.cpu().numpy(), dy.reshape(-1, s.K).astype(np.float64).sum(axis=0), f"{layer} dbias")
    dw2 = torch.empty_like(dw)
    B.conv_bwd_weights(d, xt, dyt, dw2, None, True, ws)
    assert torch.equal(dw, dw2), "two-pass weight gradient must be bitwise reproducible"
    del dw, dw2
    if not skip_bwd_data:
        dx = torch.empty(s.N, s.H, s.W, s.C, device="cuda")
        B.conv_bwd_data(d, dyt, wt, xt, dx, ws)
        B.check_device_status()
        check(dx, lambda at: oracle.conv_bwd_data(s, dy, w, x, at=at), "bwd_data")


def test_config2_vgg_mid_layer_full_size():
    from paper_1602_06709_b200 import inputs
    c = inputs.CFG2
    s = ConvShape(N=c["N"], C=c["C"], K=c["K"], H=c["H"], W=c["W"], R=3, S=3, pad_h=1, pad_w=1)
    _sampled_three_passes(s, "cfg2", "conv")


@pytest.mark.parametrize("layer", range(5))
def test_config3_overfeat_layers_full_size(layer):
    from paper_1602_06709_b200 import inputs
    name, C, H, W, K, R, S, st, pad = inputs.CFG3_LAYERS[layer]
    s = ConvShape(N=256, C=C, K=K, H=H, W=W, R=R, S=S, stride_h=st, stride_w=st, pad_h=pad, pad_w=pad)
    _sampled_three_passes(s, "cfg3", name, samples=96 if layer == 0 else SAMPLES)


def test_config4_dnn_step_full_size():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs, networks
    net = networks.Dnn(inputs.CFG4_N)
    x = inputs.normal(inputs.tensor_id("cfg4", "x", 0), (net.N, 440), 1.0)
    lab = inputs.labels(inputs.tensor_id("cfg4", "labels", 0), net.N, 8192)
    net.x.copy_(torch.from_numpy(x)); net.labels.copy_(torch.from_numpy(lab))
    before = net.store.params.cpu().numpy().copy()
    net.step()
    B.check_device_status()
    report = G.verify_dnn_step(net, before, samples=2048)
    assert len(report) == 6 + 6 + 5


def test_config5_vgga_step_full_size():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs, networks
    net = networks.VggA(256)
    x = inputs.uniform(inputs.tensor_id("cfg5", "x", 0), (256, 224, 224, 3), 0.0, 1.0)
    lab = inputs.labels(inputs.tensor_id("cfg5", "labels", 0), 256, 1000)
    net.x.copy_(torch.from_numpy(x)); net.labels.copy_(torch.from_numpy(lab))
    del x
    before = net.store.params.cpu().numpy().copy()
    net.step()
    B.check_device_status()
    report = G.verify_vgg_step(net, before, samples=96)
    assert len(report) >= 8 + 3 + 3 + 3 + 8 + 7
    assert np.isfinite(net.loss.item())
