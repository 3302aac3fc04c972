"""GPU parity of whole training steps (VGG-A-shaped CNN, sigmoid DNN): every
library call inside the step is checked against the oracle on the inputs that
call received.  Small versions are checked element by element; the full-size
workloads are checked on sampled outputs."""
import numpy as np
import pytest
import torch

import oracle
import oracle.networks as ON

pytestmark = pytest.mark.gpu

SMALL_CONV = [("conv1", 3, 8, True), ("conv2", 8, 16, True), ("conv3", 16, 32, False), ("conv4", 32, 32, True),
              ("conv5", 32, 64, False), ("conv6", 64, 64, True), ("conv7", 64, 64, False), ("conv8", 64, 64, True)]


def _randomise_biases(net, scale=0.1):
    from paper_1602_06709_b200 import inputs
    for i, shp in enumerate(net.store.shapes):
        if len(shp) == 1:
            b = inputs.uniform(inputs.tensor_id("bias", i), shp, -scale, scale)
            net.store.p(i).copy_(torch.from_numpy(b))


def _small_vgg(N=4, hw=32, keep_unpooled=False):
    from paper_1602_06709_b200 import inputs, networks
    net = networks.VggA(N, hw=hw, conv=SMALL_CONV, fc=[(64, 128), (128, 128), (128, 10)], classes=10, cfg="small",
                        keep_unpooled=keep_unpooled)
    _randomise_biases(net)
    x = inputs.uniform(inputs.tensor_id("small", "x"), (N, hw, hw, 3), 0.0, 1.0)
    lab = inputs.labels(inputs.tensor_id("small", "labels"), N, 10)
    net.x.copy_(torch.from_numpy(x)); net.labels.copy_(torch.from_numpy(lab))
    return net, x, lab


@pytest.mark.parametrize("keep_unpooled", [False, True])
def test_small_vgg_step_per_call(keep_unpooled):
    """keep_unpooled=False is the step as benched: pooled layers store only the pooled tensor and the position
    codes; True also stores their full-resolution outputs, which lets the pooling be checked exactly."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    net, x, lab = _small_vgg(keep_unpooled=keep_unpooled)
    assert all((net.y[i] is None) == (L.pool and not keep_unpooled) for i, L in enumerate(net.convs))
    before = net.store.params.cpu().numpy().copy()
    net.step()
    B.check_device_status()
    report = G.verify_vgg_step(net, before, samples=0)
    assert len(report) >= 8 + 3 + 3 + 3 + 8 + 7


def test_unstored_pooled_layer_outputs_change_nothing():
    """One step with and without the pooled layers' full-resolution outputs stored: identical pooled tensors, codes
    and parameters.  Only the first layer's own parameters may differ in their last bits: without the stored tensors
    its weight gradient comes straight from the pooled gradient, which sums in another order."""
    from paper_1602_06709_b200 import binding as B
    res = []
    for keep in (False, True):
        net, x, lab = _small_vgg(N=8, keep_unpooled=keep)
        assert net.first_from_pooled == (not keep)
        net.step()
        B.check_device_status()
        first = net.store.offsets[2]          # conv1's weights and bias come first in the flat buffer
        res.append((net.store.params.cpu().numpy().copy(), [c.cpu().numpy().copy() for c in net.pool_codes if c is not None],
                    [t.cpu().numpy().copy() for t in net.pooled if t is not None], first))
    first = res[0][3]
    assert np.array_equal(res[0][0][first:], res[1][0][first:])
    np.testing.assert_allclose(res[0][0][:first], res[1][0][:first], rtol=0, atol=1e-6)
    for a, b in zip(res[0][1] + res[0][2], res[1][1] + res[1][2]):
        assert np.array_equal(a, b)


def test_small_vgg_step_end_to_end_against_chained_oracle():
    """Information-level check of the whole chain (TF32 truncation compounds over
    11 layers, so the bound is looser than the per-call bar)."""
    from paper_1602_06709_b200 import binding as B
    net, x, lab = _small_vgg()
    st = net.store
    conv_params = [(net.conv_w(i).cpu().numpy(), net.conv_b(i).cpu().numpy()) for i in range(8)]
    fc_params = [(net.fc_w(j).cpu().numpy(), net.fc_b(j).cpu().numpy()) for j in range(3)]
    net.step()
    B.check_device_status()
    ref = ON.vgga_step(x, lab, conv_params, fc_params, [(c, k, p) for _, c, k, p in SMALL_CONV], net.lr)
    assert abs(net.loss.item() - ref["loss"]) <= 2e-2 * abs(ref["loss"])
    rel, _ = oracle.parity_errors(net.fc_out[-1].cpu().numpy(), ref["logits"])
    assert rel < 3e-2
    rel, _ = oracle.parity_errors(net.conv_dw(0).cpu().numpy(), ref["conv_grads"][0][0])
    assert rel < 1e-1
    rel, _ = oracle.parity_errors(net.conv_w(7).cpu().numpy(), ref["conv_params"][7][0])
    assert rel < 1e-3


def test_small_dnn_step_per_call():
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs, networks
    N, dims = 96, [44, 160, 160, 72]
    net = networks.Dnn(N, dims=dims, cfg="small_dnn")
    _randomise_biases(net)
    x = inputs.normal(inputs.tensor_id("small_dnn", "x"), (N, dims[0]), 1.0)
    lab = inputs.labels(inputs.tensor_id("small_dnn", "labels"), N, dims[-1])
    net.x.copy_(torch.from_numpy(x)); net.labels.copy_(torch.from_numpy(lab))
    params = [(net.w(j).cpu().numpy(), net.b(j).cpu().numpy()) for j in range(3)]
    before = net.store.params.cpu().numpy().copy()
    net.step()
    B.check_device_status()
    G.verify_dnn_step(net, before, samples=0)
    ref = ON.dnn_step(x, lab, params, net.lr)
    assert abs(net.loss.item() - ref["loss"]) <= 1e-2 * abs(ref["loss"])


def test_host_feed_with_overlapped_copy_matches_plain_copies():
    """step_from_host() with the next minibatch handed over in advance (its copy runs on a second stream
    while the step computes) must give exactly the losses and parameters of plain per-step copies."""
    from paper_1602_06709_b200 import inputs, networks
    N, dims = 64, [40, 96, 64]
    batches = []
    for i in range(4):
        x = inputs.normal(inputs.tensor_id("feed", "x", i), (N, dims[0]), 1.0)
        lab = inputs.labels(inputs.tensor_id("feed", "labels", i), N, dims[-1])
        batches.append((torch.from_numpy(x).pin_memory(), torch.from_numpy(lab).pin_memory()))

    def run(overlap):
        net = networks.Dnn(N, dims=dims, cfg="feed_dnn")
        losses = []
        for i, (x, lab) in enumerate(batches):
            nxt = batches[i + 1] if overlap and i + 1 < len(batches) else (None, None)
            losses.append(net.step_from_host(x, lab, nxt[0], nxt[1]))
        return losses, net.store.params.cpu().numpy().copy()

    l0, p0 = run(False)
    l1, p1 = run(True)
    # (the scalar loss is summed with atomics, so its last bits vary from run to run; the parameters do not)
    assert np.allclose(l0, l1, rtol=1e-5, atol=0)
    assert np.array_equal(p0, p1)
    assert len(set(l0)) > 1      # the minibatches differ, so a stale buffer would show


@pytest.mark.parametrize("kind", ["dnn", "vgg"])
def test_captured_step_graph_equals_eager_steps(kind):
    """capture_step() records the step's launches into a CUDA graph (one per input buffer of the host feed);
    replaying it must leave exactly the parameters that eager steps leave, also with the overlapped host feed
    that alternates between the two input buffers."""
    from paper_1602_06709_b200 import inputs, networks
    if kind == "dnn":
        N, dims = 64, [40, 96, 64]
        make = lambda: networks.Dnn(N, dims=dims, cfg="graph_dnn")
        xshape, classes, normal = (N, dims[0]), dims[-1], True
    else:
        N, hw = 4, 32
        make = lambda: networks.VggA(N, hw=hw, conv=SMALL_CONV, fc=[(64, 128), (128, 128), (128, 10)], classes=10,
                                     cfg="graph_vgg")
        xshape, classes, normal = (N, hw, hw, 3), 10, False
    batches = []
    for i in range(4):
        tid = inputs.tensor_id("graph", kind, "x", i)
        x = inputs.normal(tid, xshape, 1.0) if normal else inputs.uniform(tid, xshape, 0.0, 1.0)
        lab = inputs.labels(inputs.tensor_id("graph", kind, "labels", i), N, classes)
        batches.append((torch.from_numpy(x).pin_memory(), torch.from_numpy(lab).pin_memory()))

    def run(graph, overlap):
        net = make()
        before = net.store.params.cpu().numpy().copy()
        if graph:
            net.capture_step()
            assert np.array_equal(net.store.params.cpu().numpy(), before)       # capturing changes nothing
        losses = []
        for i, (x, lab) in enumerate(batches):
            nxt = batches[i + 1] if overlap and i + 1 < len(batches) else (None, None)
            losses.append(net.step_from_host(x, lab, nxt[0], nxt[1]))
        return losses, net.store.params.cpu().numpy().copy()

    l0, p0 = run(False, False)
    for overlap in (False, True):
        l1, p1 = run(True, overlap)
        assert np.allclose(l0, l1, rtol=1e-5, atol=0)       # (the scalar loss is summed with atomics)
        assert np.array_equal(p0, p1)
    assert len(set(l0)) > 1


@pytest.mark.parametrize("kind", ["vgg", "dnn"])
def test_data_parallel_step_on_one_rank_equals_the_plain_step(kind):
    """The data-parallel step (per-layer hooks, exchange stream, update of each layer as soon as its backpropagation
    has been issued) with a single rank must leave bit-identical parameters to the plain step: same kernels, the
    update only moves from one launch over the whole store to one per layer on the second stream."""
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import data_parallel, inputs, networks

    def make():
        if kind == "vgg":
            return _small_vgg()[0]
        net = networks.Dnn(64, dims=[40, 96, 96, 32], cfg="small_dnn")
        _randomise_biases(net)
        net.x.copy_(torch.from_numpy(inputs.normal(inputs.tensor_id("small_dnn", "x"), (64, 40), 1.0)))
        net.labels.copy_(torch.from_numpy(inputs.labels(inputs.tensor_id("small_dnn", "labels"), 64, 32)))
        return net
    plain, dp_net = make(), make()
    assert torch.equal(plain.store.params, dp_net.store.params)
    dp = data_parallel.DataParallelStep(dp_net)
    for _ in range(3):
        plain.step()
        dp.step()
    dp.finish()
    torch.cuda.synchronize()
    B.check_device_status()
    assert torch.equal(plain.store.params, dp_net.store.params)
    assert torch.allclose(plain.loss, dp_net.loss, rtol=1e-5)        # (the loss scalar is summed with atomics)
    buckets = dp_net.param_buckets()
    assert len(buckets) == len(dp_net.store.shapes) // 2
    assert sum(length for _, length in buckets) == dp_net.store.total and all(length % 64 == 0 for _, length in buckets)


def test_hybrid_fc_layer_with_library_kernels_single_rank():
    """hybrid.HybridFc with the library's FC kernels as its contractions (one rank: one group of one): forward,
    backward and update against the oracle's fully-connected passes."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import hybrid, inputs
    N, C, K, lr = 96, 256, 128, 0.05
    x = inputs.normal(inputs.tensor_id("hyb", "x"), (N, C), 1.0)
    w = inputs.normal(inputs.tensor_id("hyb", "w"), (K, C), (1.0 / C) ** 0.5)
    b = inputs.uniform(inputs.tensor_id("hyb", "b"), (K,), -0.5, 0.5)
    dy = inputs.normal(inputs.tensor_id("hyb", "dy"), (N, K), 1.0)
    L = hybrid.HybridFc(C, K, 1, "relu", lr, ops=hybrid.LibraryOps(), w_full=torch.from_numpy(w), b_full=torch.from_numpy(b),
                        device="cuda")
    y = L.forward(G.dev(x))
    y_ref = oracle.fc_fwd(x, w, b, oracle.ACT_RELU)
    G.assert_parity(y.cpu().numpy(), y_ref, "hybrid fc forward")
    dx = L.backward(G.dev(dy))
    _, dx_ref, dw_ref, db_ref = oracle.fc_bwd(x, w, y.cpu().numpy(), dy, oracle.ACT_RELU, dz_dtype=np.float32)
    G.assert_parity(dx.cpu().numpy(), dx_ref, "hybrid fc dx")
    G.assert_parity(L.dw.cpu().numpy(), dw_ref, "hybrid fc dw")
    G.assert_parity(L.db.cpu().numpy(), db_ref, "hybrid fc db")
    dw_gpu = L.dw.cpu().numpy().copy()
    L.update()
    np.testing.assert_allclose(L.w.cpu().numpy(), oracle.sgd_update(w, dw_gpu, lr), rtol=0, atol=1e-6)


@pytest.mark.parametrize("which", ["vgg", "dnn"])
def test_fused_update_step_equals_plain_step(which):
    """fused_update: every weight tensor but the first layer's is updated by its own weight-gradient call (second pass
    of the split reduction, GEMM epilogue, or scratch + update), the backpropagation of the layer reading the old weights
    first.  Two steps must leave every parameter tensor bit-identical to the plain step's (gradients stored, one SGD
    launch), and the losses equal."""
    from paper_1602_06709_b200 import binding as B
    from paper_1602_06709_b200 import inputs, networks
    nets = []
    for fused in (False, True):
        if which == "vgg":
            N, hw = 4, 32
            net = networks.VggA(N, hw=hw, conv=SMALL_CONV, fc=[(64, 128), (128, 128), (128, 10)], classes=10, cfg="small",
                                fused_update=fused)
            x = inputs.uniform(inputs.tensor_id("small", "x"), (N, hw, hw, 3), 0.0, 1.0)
            lab = inputs.labels(inputs.tensor_id("small", "labels"), N, 10)
        else:
            N, dims = 96, [44, 160, 160, 72]
            net = networks.Dnn(N, dims=dims, cfg="small_dnn", fused_update=fused)
            x = inputs.normal(inputs.tensor_id("small_dnn", "x"), (N, dims[0]), 1.0)
            lab = inputs.labels(inputs.tensor_id("small_dnn", "labels"), N, dims[-1])
        _randomise_biases(net)
        net.x.copy_(torch.from_numpy(x)); net.labels.copy_(torch.from_numpy(lab))
        losses = []
        for _ in range(2):
            net.step()
            losses.append(net.loss.item())
        B.check_device_status()
        nets.append((net, losses))
    (plain, lp), (fused, lf) = nets
    assert fused.store.tail_offset < fused.store.total and not fused.store.in_order
    assert all(abs(a - b) <= 1e-5 * abs(a) for a, b in zip(lp, lf))       # (the loss is summed with atomics: last bits vary)
    for i in range(len(plain.store.shapes)):
        assert torch.equal(plain.store.p(i), fused.store.p(i)), f"parameter tensor {i} differs"


def test_launch_plans_are_cached_and_change_nothing():
    """The second call with the same descriptor and buffers is served from the launch-plan cache (no tiling selection,
    no tensor-map encoding); other buffers or a changed knob build a plan of their own; results are those of a build
    with the cache switched off, bit for bit."""
    import gpu_helpers as G
    from paper_1602_06709_b200 import binding as B
    N, C, K, H = 4, 64, 96, 24
    d = B.conv_desc(N, C, K, H, H, 3, 3, 1, 1)
    g = torch.Generator(device="cuda").manual_seed(42)
    x = torch.rand(N, H, H, C, device="cuda", generator=g)
    w = torch.randn(K, 3, 3, C, device="cuda", generator=g) * 0.05
    dy = torch.randn(N, H, H, K, device="cuda", generator=g) * 1e-2
    b = torch.zeros(K, device="cuda")
    ws = G.workspace(max(B.conv_workspace_bytes(d, i) for i in range(3)))

    def three_passes(xx):
        y = torch.empty(N, H, H, K, device="cuda"); dx = torch.empty_like(xx); dw = torch.empty_like(w)
        B.conv_fwd(d, xx, w, b, y, B.ACT_RELU, ws)
        B.conv_bwd_data(d, dy, w, xx, dx, ws)
        B.conv_bwd_weights(d, xx, dy, dw, None, True, ws)
        return y, dx, dw

    B.set_tuning("PLAN_CACHE", 0)
    ref = three_passes(x)
    h0, m0 = B.plan_cache_stats()
    B.set_tuning("PLAN_CACHE", 1)
    y1 = torch.empty(N, H, H, K, device="cuda")
    B.conv_fwd(d, x, w, b, y1, B.ACT_RELU, ws)
    h1, m1 = B.plan_cache_stats()
    assert (h1, m1) == (h0, m0 + 1)                      # a new plan
    B.conv_fwd(d, x, w, b, y1, B.ACT_RELU, ws)
    h2, m2 = B.plan_cache_stats()
    assert (h2, m2) == (h1 + 1, m1)                      # served from the cache
    x2 = x.clone()
    y2 = torch.empty(N, H, H, K, device="cuda")
    B.conv_fwd(d, x2, w, b, y2, B.ACT_RELU, ws)          # other buffers: another plan
    assert B.plan_cache_stats() == (h2, m2 + 1)
    B.set_tuning("BN", 32)                               # a knob changed: another plan, and the knob is honoured
    B.conv_fwd(d, x, w, b, y2, B.ACT_RELU, ws)
    assert B.plan_cache_stats() == (h2, m2 + 2)
    assert "BN=32" in B.conv_plan_describe(d, B.PASS_FWD)
    B.set_tuning("BN", None)
    for _ in range(2):                                   # cached plans of all three passes, twice: identical results
        got = three_passes(x)
        for a_, b_ in zip(ref, got):
            assert torch.equal(a_, b_)
    B.check_device_status()
