"""Pins for the non-contraction oracle pieces: SGD, max-pool, softmax
cross-entropy, activations, the parity metric."""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(99)


def test_sgd_closed_form_and_fixed_point():
    w = RNG.normal(size=1000).astype(np.float32)
    dw = RNG.normal(size=1000).astype(np.float32)
    out = oracle.sgd_update(w, dw, 0.01)
    lr = float(np.float32(0.01))
    for i in (0, 17, 999):
        assert out[i] == float(w[i]) - lr * float(dw[i])
    np.testing.assert_array_equal(oracle.sgd_update(w, np.zeros_like(w), 0.5), w.astype(np.float64))
    # a quadratic bowl L = 0.5*|w|^2 has dw = w: one step scales w by (1 - lr)
    np.testing.assert_allclose(oracle.sgd_update(w, w, 0.25), 0.75 * w.astype(np.float64), rtol=1e-15)


def test_maxpool_forward_brute_force():
    x = RNG.normal(size=(2, 6, 4, 3))
    y = oracle.maxpool2x2_fwd(x)
    for n in range(2):
        for p in range(3):
            for q in range(2):
                for c in range(3):
                    assert y[n, p, q, c] == max(x[n, 2 * p + i, 2 * q + j, c] for i in range(2) for j in range(2))


def test_maxpool_backward_first_max_and_fd():
    x = RNG.normal(size=(1, 4, 4, 2))
    dy = RNG.normal(size=(1, 2, 2, 2))
    dx = oracle.maxpool2x2_bwd(x, dy)
    # brute force with first-max tie-break
    ref = np.zeros_like(x)
    for p in range(2):
        for q in range(2):
            for c in range(2):
                best, arg = -np.inf, None
                for i in range(2):
                    for j in range(2):
                        v = x[0, 2 * p + i, 2 * q + j, c]
                        if v > best:
                            best, arg = v, (i, j)
                ref[0, 2 * p + arg[0], 2 * q + arg[1], c] = dy[0, p, q, c]
    np.testing.assert_array_equal(dx, ref)
    # finite difference of <dy, pool(x)> (no ties in a random draw)
    h = 1e-6
    for i in RNG.choice(x.size, 8, replace=False):
        xp = x.copy().reshape(-1); xm = x.copy().reshape(-1)
        xp[i] += h; xm[i] -= h
        fd = (np.vdot(dy, oracle.maxpool2x2_fwd(xp.reshape(x.shape))) -
              np.vdot(dy, oracle.maxpool2x2_fwd(xm.reshape(x.shape)))) / (2 * h)
        assert abs(fd - dx.reshape(-1)[i]) < 1e-8


def test_maxpool_backward_ties_go_to_first_and_mask():
    x = np.zeros((1, 2, 2, 1))
    dy = np.full((1, 1, 1, 1), 3.0)
    dx = oracle.maxpool2x2_bwd(x, dy)
    assert dx[0, 0, 0, 0] == 3.0 and dx.sum() == 3.0
    x[0, 1, 0, 0] = 0.0; x[0, 0, 1, 0] = 0.0
    # after the ReLU mask (x <= 0 everywhere) nothing survives: tie-independent
    assert oracle.maxpool2x2_bwd(x, dy, relu_mask_src=x).sum() == 0.0


def test_maxpool_position_codes_brute_force_and_routing():
    """Codes by a literal loop over each window (first maximum in row-major order, bit 2 for a maximum <= 0);
    routing by codes must equal the pooling backward pass from x, with and without the ReLU mask taken from x."""
    x = np.maximum(RNG.normal(size=(2, 6, 4, 3)), 0.0)        # post-ReLU values: ties among zeros
    x[0, 0:2, 0:2, 0] = 0.0                                   # an all-zero window
    x[1, 2:4, 2:4, 1] = 5.0                                   # a positive four-way tie
    codes = oracle.maxpool2x2_codes(x)
    assert codes.dtype == np.uint8 and codes.shape == (2, 3, 2, 3)
    for n in range(2):
        for p in range(3):
            for q in range(2):
                for c in range(3):
                    win = [x[n, 2 * p + i, 2 * q + j, c] for i in range(2) for j in range(2)]
                    e = min(k for k in range(4) if win[k] == max(win))
                    assert codes[n, p, q, c] == e + (4 if max(win) <= 0 else 0)
    assert codes[0, 0, 0, 0] == 4 and codes[1, 1, 1, 1] == 0
    dy = RNG.normal(size=(2, 3, 2, 3))
    np.testing.assert_array_equal(oracle.maxpool2x2_bwd_codes(codes, dy, False), oracle.maxpool2x2_bwd(x, dy))
    np.testing.assert_array_equal(oracle.maxpool2x2_bwd_codes(codes, dy, True),
                                  oracle.maxpool2x2_bwd(x, dy, relu_mask_src=x))
    # a hand-written case: code 3 sends the gradient to the window's last position, code 6 (masked) nowhere
    g = oracle.maxpool2x2_bwd_codes(np.array([[[[3, 6]]]], dtype=np.uint8), np.array([[[[2.0, 7.0]]]]), True)
    assert g.shape == (1, 2, 2, 2) and g[0, 1, 1, 0] == 2.0 and g.sum() == 2.0
    g = oracle.maxpool2x2_bwd_codes(np.array([[[[3, 6]]]], dtype=np.uint8), np.array([[[[2.0, 7.0]]]]), False)
    assert g[0, 1, 0, 1] == 7.0 and g.sum() == 9.0


def test_softmax_xent_closed_forms():
    N, K = 5, 7
    z = RNG.normal(size=(N, K)) * 3
    lab = RNG.integers(0, K, N)
    loss, dz = oracle.softmax_xent(z, lab)
    np.testing.assert_allclose(dz.sum(axis=1), 0.0, atol=1e-15)
    # uniform logits: loss = log K
    l0, d0 = oracle.softmax_xent(np.zeros((N, K)), lab)
    assert abs(l0 - np.log(K)) < 1e-14
    # shift invariance
    l1, d1 = oracle.softmax_xent(z + 100.0, lab)
    assert abs(l1 - loss) < 1e-12
    np.testing.assert_allclose(d1, dz, atol=1e-14)
    # direct definition
    p = np.exp(z) / np.exp(z).sum(1, keepdims=True)
    assert abs(loss + np.mean(np.log(p[np.arange(N), lab]))) < 1e-13
    # finite differences
    h = 1e-6
    for i in RNG.choice(z.size, 10, replace=False):
        zp = z.copy().reshape(-1); zm = z.copy().reshape(-1)
        zp[i] += h; zm[i] -= h
        fd = (oracle.softmax_xent(zp.reshape(N, K), lab)[0] - oracle.softmax_xent(zm.reshape(N, K), lab)[0]) / (2 * h)
        assert abs(fd - dz.reshape(-1)[i]) < 1e-8


def test_softmax_xent_matches_torch():
    torch = pytest.importorskip("torch")
    z = RNG.normal(size=(6, 11)); lab = RNG.integers(0, 11, 6)
    zt = torch.tensor(z, requires_grad=True)
    lt = torch.nn.functional.cross_entropy(zt, torch.tensor(lab))
    lt.backward()
    loss, dz = oracle.softmax_xent(z, lab)
    assert abs(loss - lt.item()) < 1e-13
    np.testing.assert_allclose(dz, zt.grad.numpy(), atol=1e-14)


def test_activation_gradients_fd():
    z = RNG.normal(size=50)
    dy = RNG.normal(size=50)
    h = 1e-6
    sig = lambda v: 1 / (1 + np.exp(-v))
    np.testing.assert_allclose(oracle.act_grad(sig(z), dy, oracle.ACT_SIGMOID),
                               dy * (sig(z + h) - sig(z - h)) / (2 * h), atol=1e-9)
    relu = lambda v: np.maximum(v, 0)
    np.testing.assert_allclose(oracle.act_grad(relu(z), dy, oracle.ACT_RELU),
                               dy * (relu(z + h) - relu(z - h)) / (2 * h), atol=1e-9)
    assert oracle.act_grad(np.zeros(3), np.ones(3), oracle.ACT_RELU).sum() == 0.0   # gradient at exactly 0 is 0


def test_parity_metric():
    ref = np.array([3.0, -4.0])
    got = np.array([3.0, -4.5])
    rel, mx = oracle.parity_errors(got, ref)
    assert abs(rel - 0.5 / 5.0) < 1e-15
    assert abs(mx - 0.5 / (5.0 / np.sqrt(2))) < 1e-15
    assert oracle.parity_errors(ref, ref) == (0.0, 0.0)
