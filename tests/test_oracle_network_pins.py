"""Pins for the chained fp64 oracle steps (oracle/networks.py), independent of
the CUDA path: a small VGG-shaped net and a small sigmoid DNN are rebuilt with
torch float64 on the CPU (library conv2d / max_pool2d / linear / cross_entropy
and autograd), and the oracle's loss, every gradient, the skipped first-layer
backpropagation and the updated parameters must agree to ~1e-10; finite
differences of the loss pin a first-layer, a pooled-layer and an FC weight.

Order of the step: weight gradient before backpropagation, first layer without
backpropagation (Sec. 3.1); per-layer rules of Sec. 2.1 (Algorithm 1 and the
two update rules); topologies as in Sec. 5 (conv -> ReLU [-> 2x2 pool] blocks,
then FC layers; sigmoid hidden layers for the DNN)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import networks as ON

LR = 0.05


def _small_vgg(seed=7, N=4, HW=16):
    rng = np.random.default_rng(seed)
    spec = [(3, 8, True), (8, 16, True), (16, 16, False), (16, 24, True)]
    x = rng.uniform(0.0, 1.0, size=(N, HW, HW, 3))
    convs = []
    for C, K, _ in spec:
        w = rng.normal(0.0, np.sqrt(2.0 / (9 * C)), size=(K, 3, 3, C))
        b = rng.normal(0.0, 0.3, size=K)        # non-zero, some strongly negative: post-ReLU zeros and ties
        convs.append((w, b))
    hw = HW // 8
    dims = [hw * hw * 24, 32, 20, 10]
    fcs = []
    for C, K in zip(dims[:-1], dims[1:]):
        fcs.append((rng.normal(0.0, np.sqrt(2.0 / C), size=(K, C)), rng.normal(0.0, 0.2, size=K)))
    labels = rng.integers(0, 10, size=N)
    return x, labels, convs, fcs, spec


def _torch_vgg_loss(x, labels, convs, fcs, spec):
    """Same network through torch float64 library ops.  Oracle tensors are
    NHWC / KRSC; torch wants NCHW / KCRS, and the flatten order of the oracle
    is (h, w, c)."""
    a = torch.from_numpy(x).permute(0, 3, 1, 2)
    for (C, K, pool), (w, b) in zip(spec, convs):
        a = F.relu(F.conv2d(a, w.permute(0, 3, 1, 2), b, padding=1))
        if pool:
            a = F.max_pool2d(a, 2)
    h = a.permute(0, 2, 3, 1).reshape(a.shape[0], -1)
    for j, (w, b) in enumerate(fcs):
        h = F.linear(h, w, b)
        if j + 1 < len(fcs):
            h = F.relu(h)
    return F.cross_entropy(h, torch.from_numpy(labels), reduction="mean"), h


def test_vgga_step_matches_torch_float64_autograd():
    x, labels, convs, fcs, spec = _small_vgg()
    out = ON.vgga_step(x, labels, convs, fcs, spec, LR)
    # post-ReLU zeros must be present (ties inside pooling windows included) for the pin to cover them
    y0 = out["conv_out"][0]
    win = y0.reshape(y0.shape[0], y0.shape[1] // 2, 2, y0.shape[2] // 2, 2, y0.shape[3])
    assert (win.max(axis=(2, 4)) == 0).any() and (y0 == 0).mean() > 0.05

    tc = [(torch.from_numpy(w).requires_grad_(), torch.from_numpy(b).requires_grad_()) for w, b in convs]
    tf = [(torch.from_numpy(w).requires_grad_(), torch.from_numpy(b).requires_grad_()) for w, b in fcs]
    loss, logits = _torch_vgg_loss(x, labels, tc, tf, spec)
    loss.backward()
    assert abs(out["loss"] - loss.item()) <= 1e-12 * max(1.0, abs(loss.item()))
    np.testing.assert_allclose(out["logits"], logits.detach().numpy(), rtol=0, atol=1e-11)
    for i, ((dw, db), (tw, tb)) in enumerate(zip(out["conv_grads"], tc)):
        np.testing.assert_allclose(dw, tw.grad.numpy(), rtol=0, atol=1e-12, err_msg=f"conv{i} dw")
        np.testing.assert_allclose(db, tb.grad.numpy(), rtol=0, atol=1e-12, err_msg=f"conv{i} db")
        assert np.abs(tw.grad.numpy()).max() > 1e-6          # the pin is not vacuous
    for j, ((dw, db), (tw, tb)) in enumerate(zip(out["fc_grads"], tf)):
        np.testing.assert_allclose(dw, tw.grad.numpy(), rtol=0, atol=1e-12, err_msg=f"fc{j} dw")
        np.testing.assert_allclose(db, tb.grad.numpy(), rtol=0, atol=1e-12, err_msg=f"fc{j} db")
    # vanilla SGD (Sec. 1): w - lr * dw, with lr at fp32 precision
    lr = float(np.float32(LR))
    for (nw, nb), (tw, tb) in zip(out["conv_params"] + out["fc_params"], tc + tf):
        np.testing.assert_allclose(nw, (tw - lr * tw.grad).detach().numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(nb, (tb - lr * tb.grad).detach().numpy(), rtol=0, atol=1e-12)


def _fd(loss_of, arr, idx, h=1e-6):
    old = arr[idx]
    arr[idx] = old + h
    lp = loss_of()
    arr[idx] = old - h
    lm = loss_of()
    arr[idx] = old
    return (lp - lm) / (2 * h)


def test_vgga_step_gradients_match_finite_differences_of_its_own_loss():
    x, labels, convs, fcs, spec = _small_vgg(seed=11)
    out = ON.vgga_step(x, labels, convs, fcs, spec, LR)
    loss_of = lambda: ON.vgga_step(x, labels, convs, fcs, spec, LR)["loss"]
    rng = np.random.default_rng(3)
    # first layer (no backpropagation through it), a pooled inner layer, an unpooled layer, an FC layer
    targets = [("conv", 0), ("conv", 1), ("conv", 2), ("fc", 0), ("fc", 2)]
    for kind, i in targets:
        params = convs if kind == "conv" else fcs
        grads = out["conv_grads"] if kind == "conv" else out["fc_grads"]
        w, b = params[i]
        dw, db = grads[i]
        for _ in range(3):
            idx = tuple(int(rng.integers(0, s)) for s in w.shape)
            g = _fd(loss_of, w, idx)
            assert abs(g - dw[idx]) <= 1e-7 + 1e-5 * abs(g), (kind, i, idx, g, dw[idx])
        k = int(rng.integers(0, b.size))
        g = _fd(loss_of, b, (k,))
        assert abs(g - db[k]) <= 1e-7 + 1e-5 * abs(g), (kind, i, "bias", k, g, db[k])


def _small_dnn(seed=5, N=6):
    rng = np.random.default_rng(seed)
    dims = [12, 16, 16, 16, 9]
    x = rng.normal(0.0, 1.0, size=(N, dims[0]))
    params = []
    for C, K in zip(dims[:-1], dims[1:]):
        a = np.sqrt(6.0 / (C + K))
        params.append((rng.uniform(-a, a, size=(K, C)), rng.normal(0.0, 0.2, size=K)))
    labels = rng.integers(0, dims[-1], size=N)
    return x, labels, params


def test_dnn_step_matches_torch_float64_autograd():
    x, labels, params = _small_dnn()
    out = ON.dnn_step(x, labels, params, LR)
    tp = [(torch.from_numpy(w).requires_grad_(), torch.from_numpy(b).requires_grad_()) for w, b in params]
    h = torch.from_numpy(x)
    for j, (w, b) in enumerate(tp):
        h = F.linear(h, w, b)
        if j + 1 < len(tp):
            h = torch.sigmoid(h)
    loss = F.cross_entropy(h, torch.from_numpy(labels), reduction="mean")
    loss.backward()
    assert abs(out["loss"] - loss.item()) <= 1e-12
    np.testing.assert_allclose(out["logits"], h.detach().numpy(), rtol=0, atol=1e-12)
    lr = float(np.float32(LR))
    for j, ((dw, db), (tw, tb), (nw, nb)) in enumerate(zip(out["grads"], tp, out["params"])):
        np.testing.assert_allclose(dw, tw.grad.numpy(), rtol=0, atol=1e-13, err_msg=f"layer {j} dw")
        np.testing.assert_allclose(db, tb.grad.numpy(), rtol=0, atol=1e-13, err_msg=f"layer {j} db")
        np.testing.assert_allclose(nw, (tw - lr * tw.grad).detach().numpy(), rtol=0, atol=1e-13)
        np.testing.assert_allclose(nb, (tb - lr * tb.grad).detach().numpy(), rtol=0, atol=1e-13)


def test_dnn_step_gradients_match_finite_differences_of_its_own_loss():
    x, labels, params = _small_dnn(seed=9)
    out = ON.dnn_step(x, labels, params, LR)
    loss_of = lambda: ON.dnn_step(x, labels, params, LR)["loss"]
    rng = np.random.default_rng(1)
    for j in (0, 2, len(params) - 1):
        w, b = params[j]
        dw, db = out["grads"][j]
        for _ in range(3):
            idx = tuple(int(rng.integers(0, s)) for s in w.shape)
            g = _fd(loss_of, w, idx)
            assert abs(g - dw[idx]) <= 1e-8 + 1e-6 * abs(g), (j, idx, g, dw[idx])
        k = int(rng.integers(0, b.size))
        g = _fd(loss_of, b, (k,))
        assert abs(g - db[k]) <= 1e-8 + 1e-6 * abs(g)
