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


# Guard bands: every output and workspace these helpers allocate sits between two 4 KB bands filled with a byte
# pattern; check_guards() (called by the helpers after each call and by an autouse fixture at the end of every
# test) asserts that no kernel wrote past either end of its buffer.
GUARD_BYTES = 4096
GUARD_BYTE = 0xA5
_guards = []


def guarded(shape, dtype=torch.float32, fill=float("nan")):
    """A tensor of `shape` in the middle of a pattern-filled allocation (256-byte aligned)."""
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    raw = torch.full((GUARD_BYTES + n + GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
    t = raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(*shape)
    if fill is not None:
        t.fill_(fill)
    _guards.append((raw, n))
    return t


def check_guards(clear=False):
    torch.cuda.synchronize()
    for raw, n in _guards:
        lo, hi = raw[:GUARD_BYTES], raw[GUARD_BYTES + n:]
        assert bool((lo == GUARD_BYTE).all()), "a kernel wrote in front of its buffer"
        assert bool((hi == GUARD_BYTE).all()), "a kernel wrote past the end of its buffer"
    if clear:
        _guards.clear()


def workspace(nbytes):
    return guarded((max(nbytes, 256),), torch.uint8, fill=None) if nbytes else None


def shape_to_desc(s: ConvShape):
    return B.ConvDesc(s.N, s.C, s.K, s.H, s.W, s.R, s.S, s.stride_h, s.stride_w, s.pad_h, s.pad_w)


def make_inputs(s: ConvShape, tag, kind="unit"):
    x, w, dy = inputs.conv_inputs("test", tag, s.N, s.C, s.H, s.W, s.K, s.R, s.S, s.P, s.Q, kind)
    bias = inputs.uniform(inputs.tensor_id("test", tag, "bias"), (s.K,), -0.5, 0.5)
    return x, w, dy, bias


def run_conv_fwd(s, x, w, bias, act):
    d = shape_to_desc(s)
    y = guarded((s.N, s.P, s.Q, s.K))
    B.conv_fwd(d, dev(x), dev(w), None if bias is None else dev(bias), y, act,
               workspace(B.conv_workspace_bytes(d, B.PASS_FWD)))
    B.check_device_status()
    check_guards()
    return y.cpu().numpy()


def run_conv_bwd_data(s, dy, w, mask):
    d = shape_to_desc(s)
    dx = guarded((s.N, s.H, s.W, s.C))
    B.conv_bwd_data(d, dev(dy), dev(w), None if mask is None else dev(mask), dx,
                    workspace(B.conv_workspace_bytes(d, B.PASS_BWD_DATA)))
    B.check_device_status()
    check_guards()
    return dx.cpu().numpy()


def run_conv_bwd_weights(s, x, dy, want_db, deterministic=True):
    d = shape_to_desc(s)
    dw = guarded((s.K, s.R, s.S, s.C))
    db = guarded((s.K,)) if want_db else None
    B.conv_bwd_weights(d, dev(x), dev(dy), dw, db, deterministic,
                       workspace(B.conv_workspace_bytes(d, B.PASS_BWD_WEIGHTS)))
    B.check_device_status()
    check_guards()
    return dw.cpu().numpy(), (db.cpu().numpy() if want_db else None)


# ---------------------------------------------------------------------------
# Per-call verification of a whole training step: every library call of the
# step is re-computed by the oracle from the inputs the GPU call actually
# received (copied back from the device) and compared with what the GPU call
# wrote.  `samples` > 0 checks that many randomly chosen output elements per
# tensor (for sizes where the full oracle would take too long); 0 checks all.
# ---------------------------------------------------------------------------
def sample_indices(shape, samples, rng, edge=6):
    """Flat indices of `samples` uniformly random elements plus stratified ones: for every dimension, `edge`
    elements whose coordinate in that dimension lies in its last min(32, d) entries (the last image, the last tile
    row / column, the last 32 output maps, the last k tile) and `edge` in its first min(8, d), the other
    coordinates random -- a defect confined to a boundary tile cannot hide from these at any tensor size."""
    shape = tuple(int(d) for d in shape)
    size = int(np.prod(shape))
    idx = [rng.choice(size, size=min(samples, size), replace=False).astype(np.int64)]
    for j, dj in enumerate(shape):
        for lo, hi in ((max(0, dj - 32), dj), (0, min(8, dj))):
            coords = [rng.integers(0, d, size=edge) for d in shape]
            coords[j] = rng.integers(lo, hi, size=edge)
            idx.append(np.ravel_multi_index(coords, shape).astype(np.int64))
    return np.unique(np.concatenate(idx))


def _cmp(got_t, ref_fn, size, samples, rng, what, report):
    got = got_t.detach().cpu().numpy().reshape(-1)
    if samples and size > samples:
        idx = sample_indices(got_t.shape, samples, rng) if got_t.numel() == size else \
            np.sort(rng.choice(size, size=samples, replace=False)).astype(np.int64)
        ref = ref_fn(idx)
        g = got[idx]
    else:
        ref = ref_fn(None).reshape(-1)
        g = got
    rel, mx = oracle.parity_errors(g, ref)
    report.append((what, rel, mx))
    assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"{what}: rel_l2={rel:.3e} max/rms={mx:.3e}"


def _check_pooled_only(net, i, s, xin, w, b, samples, rng, report):
    """A pooled layer whose full-resolution output was not stored: the pooled tensor against the oracle's
    pool(relu(conv)), and the position codes against the oracle's own window values -- a code must name a position
    whose value is the window's maximum up to the parity tolerance (TF32 rounding may reorder near-ties, never
    more), and bit 2 must say exactly whether the stored maximum is <= 0."""
    L = net.convs[i]
    N, P, Q, K = s.N, s.P, s.Q, s.K
    size = N * (P // 2) * (Q // 2) * K
    got_p = net.pooled[i].detach().cpu().numpy().reshape(-1)
    codes = net.pool_codes[i].detach().cpu().numpy().reshape(-1)
    idx = (sample_indices((N, P // 2, Q // 2, K), samples, rng) if samples and size > samples
           else np.arange(size, dtype=np.int64))
    k = idx % K; q2 = (idx // K) % (Q // 2); p2 = (idx // (K * (Q // 2))) % (P // 2); n = idx // (K * (Q // 2) * (P // 2))
    win = np.stack([((n * P + 2 * p2 + e // 2) * Q + 2 * q2 + e % 2) * K + k for e in range(4)], axis=1)   # [len][4]
    if samples and size > samples:
        yw = oracle.conv_fwd(s, xin, w, b, oracle.ACT_RELU, at=win.reshape(-1)).reshape(-1, 4)
    else:
        yw = oracle.conv_fwd(s, xin, w, b, oracle.ACT_RELU).reshape(-1)[win]
    ref = yw.max(axis=1)
    rel, mx = oracle.parity_errors(got_p[idx], ref)
    report.append((f"{L.name} fwd+pool", rel, mx))
    assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"{L.name} fwd+pool: rel_l2={rel:.3e} max/rms={mx:.3e}"
    c = codes[idx].astype(np.int64)
    assert c.max() <= 7, f"{L.name}: position code out of range"
    assert np.array_equal(c >= 4, got_p[idx] <= 0.0), f"{L.name}: bit 2 of the codes != (stored maximum <= 0)"
    tol = MAX_OVER_RMS_TOL * float(np.sqrt(np.mean(ref * ref)))
    chosen = yw[np.arange(len(idx)), c & 3]
    assert np.all(chosen >= ref - tol), f"{L.name}: a code names a position that is not the window's maximum"


def verify_vgg_step(net, params_before, samples=0, seed=0):
    """net: VggA after exactly one step(); params_before: flat params (numpy) before the step."""
    rng = np.random.default_rng(seed)
    report = []
    N = net.N
    st = net.store

    def pview(i):
        n = int(np.prod(st.shapes[i]))
        return params_before[st.offsets[i]:st.offsets[i] + n].reshape(st.shapes[i])

    host = lambda t: t.detach().cpu().numpy()
    nconv = len(net.convs)
    # forward convolutions and pools
    for i, L in enumerate(net.convs):
        s = ConvShape(N=N, C=L.C, K=L.K, H=L.H, W=L.W, R=3, S=3, pad_h=1, pad_w=1)
        xin = host(net.layer_input(i)); w = pview(2 * i); b = pview(2 * i + 1)
        if net.y[i] is None:
            _check_pooled_only(net, i, s, xin, w, b, samples, rng, report)
            continue
        _cmp(net.y[i], lambda at: oracle.conv_fwd(s, xin, w, b, oracle.ACT_RELU, at=at), net.y[i].numel(), samples,
             rng, f"{L.name} fwd", report)
        if L.pool:
            nchk = N if not samples else min(N, 2)       # sampled runs check the pooling on the first images only
            y = host(net.y[i][:nchk])
            assert np.array_equal(host(net.pooled[i][:nchk]), oracle.maxpool2x2_fwd(y).astype(np.float32)), f"{L.name} pool"
    # forward FC
    a = host(net.pooled[-1]).reshape(N, net.flat)
    for j, (C, K) in enumerate(net.fcs):
        act = oracle.ACT_RELU if j + 1 < len(net.fcs) else oracle.ACT_NONE
        w = pview(2 * (nconv + j)); b = pview(2 * (nconv + j) + 1)
        s = ConvShape(N=N, C=C, K=K, H=1, W=1, R=1, S=1)
        a_in = a
        _cmp(net.fc_out[j], lambda at: oracle.conv_fwd(s, a_in, w, b, act, at=at), N * K, samples, rng,
             f"fc{j + 1} fwd", report)
        a = host(net.fc_out[j])
    # loss
    loss_ref, dlog_ref = oracle.softmax_xent(a, host(net.labels))
    assert abs(net.loss.item() - loss_ref) <= 1e-5 * max(1.0, abs(loss_ref))
    # backward FC (fc_dout[j] now holds dz_j; the incoming dy is not kept, so check dz of the last layer only
    # against the loss gradient and the contractions against the GPU's own dz)
    rel, mx = oracle.parity_errors(host(net.fc_dout[-1]), dlog_ref)
    assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL
    for j in reversed(range(len(net.fcs))):
        C, K = net.fcs[j]
        s = ConvShape(N=N, C=C, K=K, H=1, W=1, R=1, S=1)
        dz = host(net.fc_dout[j])
        a_in = host(net.fc_out[j - 1]) if j > 0 else host(net.pooled[-1]).reshape(N, net.flat)
        w = pview(2 * (nconv + j))
        _cmp(net.fc_dw(j), lambda at: oracle.conv_bwd_weights(s, a_in, dz, at=at), K * C, samples, rng,
             f"fc{j + 1} dw", report)
        db_ref = dz.astype(np.float64).sum(axis=0)
        rel, mx = oracle.parity_errors(host(net.fc_db(j)), db_ref)
        assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"fc{j + 1} db"
        # dx of layer j is the dy of layer j-1 before its activation gradient was applied in place; for j == 0 it
        # is kept in dpooled[-1]
        if j == 0:
            _cmp(net.dpooled[-1], lambda at: oracle.conv_bwd_data(s, dz, w, at=at), N * C, samples, rng,
                 "fc1 dx", report)
        else:
            # fc_dout[j-1] = dx_j * act'(out_{j-1}): re-apply the activation gradient to the oracle's dx
            out_prev = host(net.fc_out[j - 1]).reshape(-1)

            def ref_fn(at, s=s, dz=dz, w=w, out_prev=out_prev):
                if at is None:
                    dx = oracle.conv_bwd_data(s, dz, w).reshape(-1)
                    return np.where(out_prev > 0, dx, 0.0)
                dx = oracle.conv_bwd_data(s, dz, w, at=at)
                return np.where(out_prev[at] > 0, dx, 0.0)
            _cmp(net.fc_dout[j - 1], ref_fn, N * C, samples, rng, f"fc{j + 1} dx (masked)", report)
    # backward convolutions
    for i in reversed(range(nconv)):
        L = net.convs[i]
        s = ConvShape(N=N, C=L.C, K=L.K, H=L.H, W=L.W, R=3, S=3, pad_h=1, pad_w=1)
        if net.dy[i] is None:
            # first layer, weight gradient taken straight from the pooled gradient: the reference dy is the oracle's
            # code-routed pooling backward pass (image by image, to bound the host memory of the full-size run)
            codes_h, dp_h = host(net.pool_codes[i]), host(net.dpooled[i])
            dz = np.empty((N, L.H, L.W, L.K), np.float32)
            for n in range(N):
                dz[n] = oracle.maxpool2x2_bwd_codes(codes_h[n:n + 1], dp_h[n:n + 1], True)[0]
            xin = host(net.layer_input(i))
            _cmp(net.conv_dw(i), lambda at: oracle.conv_bwd_weights(s, xin, dz, at=at), net.conv_dw(i).numel(), samples,
                 rng, f"{L.name} dw (from pooled dy)", report)
            db_ref = dz.reshape(-1, L.K).astype(np.float64).sum(axis=0)
            rel, mx = oracle.parity_errors(host(net.conv_db(i)), db_ref)
            assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"{L.name} db (from pooled dy)"
            continue
        if L.pool and net.y[i] is None:      # routed by the position codes the forward call recorded, bit for bit
            nchk = N if not samples else min(N, 2)
            ref = oracle.maxpool2x2_bwd_codes(host(net.pool_codes[i][:nchk]), host(net.dpooled[i][:nchk]), True)
            assert np.array_equal(host(net.dy[i][:nchk]), ref.astype(np.float32)), f"{L.name} pool bwd (codes)"
        elif L.pool:
            nchk = N if not samples else min(N, 2)
            y = host(net.y[i][:nchk]); dp = host(net.dpooled[i][:nchk])
            assert np.array_equal(host(net.dy[i][:nchk]), oracle.maxpool2x2_bwd(y, dp, y).astype(np.float32)), f"{L.name} pool bwd"
        dz = host(net.dy[i]); xin = host(net.layer_input(i)); w = pview(2 * i)
        _cmp(net.conv_dw(i), lambda at: oracle.conv_bwd_weights(s, xin, dz, at=at), net.conv_dw(i).numel(), samples,
             rng, f"{L.name} dw", report)
        db_ref = dz.reshape(-1, L.K).astype(np.float64).sum(axis=0)
        rel, mx = oracle.parity_errors(host(net.conv_db(i)), db_ref)
        assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"{L.name} db"
        if i > 0:
            prev = net.convs[i - 1]
            if prev.pool:
                _cmp(net.dpooled[i - 1], lambda at: oracle.conv_bwd_data(s, dz, w, None, at=at),
                     net.dpooled[i - 1].numel(), samples, rng, f"{L.name} dx", report)
            else:
                mask = host(net.y[i - 1])
                _cmp(net.dy[i - 1], lambda at: oracle.conv_bwd_data(s, dz, w, mask, at=at), net.dy[i - 1].numel(),
                     samples, rng, f"{L.name} dx (masked)", report)
    # SGD update of every parameter, against the GPU's own gradients
    grads = host(st.grads); after = host(st.params)
    ref = oracle.sgd_update(params_before, grads, net.lr)
    np.testing.assert_allclose(after, ref, rtol=0, atol=1e-6 * max(1.0, float(np.abs(ref).max())))
    return report


def verify_dnn_step(net, params_before, samples=0, seed=0):
    rng = np.random.default_rng(seed)
    report = []
    N = net.N
    st = net.store
    host = lambda t: t.detach().cpu().numpy()

    def pview(i):
        n = int(np.prod(st.shapes[i]))
        return params_before[st.offsets[i]:st.offsets[i] + n].reshape(st.shapes[i])

    n = len(net.layers)
    a = host(net.x)
    for j, (C, K) in enumerate(net.layers):
        act = oracle.ACT_SIGMOID if j + 1 < n else oracle.ACT_NONE
        s = ConvShape(N=N, C=C, K=K, H=1, W=1, R=1, S=1)
        w = pview(2 * j); b = pview(2 * j + 1); a_in = a
        _cmp(net.out[j], lambda at: oracle.conv_fwd(s, a_in, w, b, act, at=at), N * K, samples, rng, f"fc{j + 1} fwd",
             report)
        a = host(net.out[j])
    loss_ref, dlog_ref = oracle.softmax_xent(a, host(net.labels))
    assert abs(net.loss.item() - loss_ref) <= 1e-5 * max(1.0, abs(loss_ref))
    rel, mx = oracle.parity_errors(host(net.dout[-1]), dlog_ref)
    assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL
    for j in reversed(range(n)):
        C, K = net.layers[j]
        s = ConvShape(N=N, C=C, K=K, H=1, W=1, R=1, S=1)
        dz = host(net.dout[j]); a_in = host(net.out[j - 1]) if j > 0 else host(net.x); w = pview(2 * j)
        _cmp(net.dw(j), lambda at: oracle.conv_bwd_weights(s, a_in, dz, at=at), K * C, samples, rng, f"fc{j + 1} dw",
             report)
        rel, mx = oracle.parity_errors(host(net.db(j)), dz.astype(np.float64).sum(axis=0))
        assert rel <= REL_L2_TOL and mx <= MAX_OVER_RMS_TOL, f"fc{j + 1} db"
        if j > 0:
            out_prev = host(net.out[j - 1]).reshape(-1).astype(np.float64)

            def ref_fn(at, s=s, dz=dz, w=w, out_prev=out_prev):
                if at is None:
                    return oracle.conv_bwd_data(s, dz, w).reshape(-1) * out_prev * (1.0 - out_prev)
                return oracle.conv_bwd_data(s, dz, w, at=at) * out_prev[at] * (1.0 - out_prev[at])
            _cmp(net.dout[j - 1], ref_fn, N * C, samples, rng, f"fc{j + 1} dx (times sigmoid')", report)
    grads = host(st.grads); after = host(st.params)
    ref = oracle.sgd_update(params_before, grads, net.lr)
    np.testing.assert_allclose(after, ref, rtol=0, atol=1e-6 * max(1.0, float(np.abs(ref).max())))
    return report
