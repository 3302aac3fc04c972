"""TEST INFRASTRUCTURE: fp64 oracle of one full training step of the two
topologies (VGG-A CNN, fully-connected DNN), chaining the per-layer oracle
functions in float64 with no intermediate rounding.  Used by the chained parity
tests and by the benchmark's CPU-baseline leg only.  Pinned by
``tests/test_oracle_network_pins.py`` (torch float64 library networks with
autograd; finite differences of the loss)."""
from __future__ import annotations

import numpy as np

import oracle as O
from oracle import ConvShape


def vgga_step(x, labels, conv_params, fc_params, conv_spec, lr):
    """conv_spec: list of (C, K, pool).  conv_params / fc_params: lists of (w, b)
    (KRSC / [K,C]).  Per layer: weight gradient, then backpropagation; the first
    layer skips backpropagation (Sec. 3.1).  Returns a dict with the loss, every
    gradient and the updated parameters."""
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    x = f64(x)
    N = x.shape[0]
    acts_in, ys = [], []
    a = x
    for (C, K, pool), (w, b) in zip(conv_spec, conv_params):
        H, W = a.shape[1], a.shape[2]
        sh = ConvShape(N=N, C=C, K=K, H=H, W=W, R=3, S=3, pad_h=1, pad_w=1)
        acts_in.append(a)
        y = O.conv_fwd(sh, a, f64(w), f64(b), O.ACT_RELU)
        ys.append(y)
        a = O.maxpool2x2_fwd(y) if pool else y
    flat = a.reshape(N, -1)
    fc_in, fc_out = [], []
    h = flat
    for j, (w, b) in enumerate(fc_params):
        act = O.ACT_RELU if j + 1 < len(fc_params) else O.ACT_NONE
        fc_in.append(h)
        h = O.fc_fwd(h, f64(w), f64(b), act)
        fc_out.append(h)
    loss, dlogits = O.softmax_xent(h, labels)
    g = dlogits
    fc_grads = [None] * len(fc_params)
    for j in reversed(range(len(fc_params))):
        act = O.ACT_RELU if j + 1 < len(fc_params) else O.ACT_NONE
        w, _ = fc_params[j]
        dz, dx, dw, db = O.fc_bwd(fc_in[j], f64(w), fc_out[j], g, act, dz_dtype=np.float64)
        fc_grads[j] = (dw, db)
        g = dx
    g = g.reshape(a.shape)            # gradient wrt the last pooled activation
    conv_grads = [None] * len(conv_params)
    for i in reversed(range(len(conv_params))):
        C, K, pool = conv_spec[i]
        w, _ = conv_params[i]
        y = ys[i]
        if pool:
            dz = O.maxpool2x2_bwd(y, g, relu_mask_src=y)
        else:
            dz = np.where(y > 0.0, g, 0.0)
        xin = acts_in[i]
        sh = ConvShape(N=N, C=C, K=K, H=xin.shape[1], W=xin.shape[2], R=3, S=3, pad_h=1, pad_w=1)
        dw, db = O.conv_bwd_weights(sh, xin, dz, want_db=True)
        conv_grads[i] = (dw, db)
        if i > 0:
            g = O.conv_bwd_data(sh, dz, f64(w))
    new_conv = [(O.sgd_update(w, dw, lr), O.sgd_update(b, db, lr)) for (w, b), (dw, db) in zip(conv_params, conv_grads)]
    new_fc = [(O.sgd_update(w, dw, lr), O.sgd_update(b, db, lr)) for (w, b), (dw, db) in zip(fc_params, fc_grads)]
    return dict(loss=loss, logits=fc_out[-1], conv_grads=conv_grads, fc_grads=fc_grads, conv_params=new_conv,
                fc_params=new_fc, conv_out=ys)


def dnn_step(x, labels, params, lr):
    """Sigmoid hidden layers, linear output + softmax cross-entropy; the first
    layer skips backpropagation."""
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    h = f64(x)
    ins, outs = [], []
    n = len(params)
    for j, (w, b) in enumerate(params):
        act = O.ACT_SIGMOID if j + 1 < n else O.ACT_NONE
        ins.append(h)
        h = O.fc_fwd(h, f64(w), f64(b), act)
        outs.append(h)
    loss, g = O.softmax_xent(h, labels)
    grads = [None] * n
    for j in reversed(range(n)):
        act = O.ACT_SIGMOID if j + 1 < n else O.ACT_NONE
        dz, dx, dw, db = O.fc_bwd(ins[j], f64(params[j][0]), outs[j], g, act, dz_dtype=np.float64)
        grads[j] = (dw, db)
        g = dx
    new = [(O.sgd_update(w, dw, lr), O.sgd_update(b, db, lr)) for (w, b), (dw, db) in zip(params, grads)]
    return dict(loss=loss, logits=outs[-1], grads=grads, params=new)
