"""TEST INFRASTRUCTURE: the fp64 CPU oracle.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` /
``--impl reference`` legs of ``bench.py`` may import this package.  The CUDA
product path neither imports it nor shares code with it.

Every function here evaluates the plain definition of one step of the
training hot path in float64:

* convolution forward / backward-data / weight-gradient: Algorithm 1 and the
  two update rules printed after it in Sec. 2.1 (direct loops in
  ``pcl_oracle.c``; zero padding, cross-correlation, no kernel flip);
* fully-connected layers: the ``k_h = k_w = out_h = out_w = 1`` special case of
  the same loops (Sec. 2.1), evaluated by calling the convolution oracle;
* vanilla SGD ``w <- w - lr * dw`` (Sec. 1: the algorithm is not altered, no
  momentum or decay);
* the glue the VGG-A and DNN topologies need and the paper does not spell out
  (ReLU, sigmoid, 2x2/2 max-pool, softmax cross-entropy): textbook definitions.

Readings of the paper taken here (all listed again in the design notes):
the output of Algorithm 1 is indexed by the *output* feature map; the printed
``- 1`` offset is a pad of one and generalises to ``- pad``; weights are stored
K,R,S,C (layout is not part of the mathematics); a bias term and activations
are this build's additions; max-pool backward sends the gradient to the first
maximum in row-major window order.

Pins (see ``tests/test_oracle_*.py``): literal scatter-form transcription in the
paper's index order on tiny layers, adjoint identities, finite differences,
matmul / shift / all-ones special cases, torch.float64 conv2d and autograd;
the chained steps of ``networks.py`` against torch.float64 networks with
autograd and finite differences of their loss.
Parity unpinned: nothing in this package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpcl_oracle.so")
_lib = None

ACT_NONE, ACT_RELU, ACT_SIGMOID = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile pcl_oracle.c with gcc (building the checker is not using it)."""
    srcs = [os.path.join(_HERE, f) for f in ("pcl_oracle.c", "conv_loops.inc")]
    if not force and os.path.exists(_LIB_PATH):
        if all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in srcs):
            return _LIB_PATH
    cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB_PATH, srcs[0], "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB_PATH


class _ConvShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("N", "C", "K", "H", "W", "R", "S", "stride_h", "stride_w", "pad_h", "pad_w")]


@dataclass(frozen=True)
class ConvShape:
    N: int
    C: int
    K: int
    H: int
    W: int
    R: int
    S: int
    stride_h: int = 1
    stride_w: int = 1
    pad_h: int = 0
    pad_w: int = 0

    @property
    def P(self) -> int:
        span = self.H + 2 * self.pad_h - self.R
        return 0 if span < 0 else span // self.stride_h + 1

    @property
    def Q(self) -> int:
        span = self.W + 2 * self.pad_w - self.S
        return 0 if span < 0 else span // self.stride_w + 1

    def flops(self) -> int:
        """2*N*K*P*Q*C*R*S per pass (one third of Comp in Sec. 3.1)."""
        return 2 * self.N * self.K * self.P * self.Q * self.C * self.R * self.S

    def _c(self) -> _ConvShape:
        return _ConvShape(self.N, self.C, self.K, self.H, self.W, self.R, self.S,
                          self.stride_h, self.stride_w, self.pad_h, self.pad_w)


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().oracle_threads())


def _prep(a, dt):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=dt)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def _suffix_dtype(*arrays):
    """Pick the f32 or f64 instantiation: f64 only if every given array is f64."""
    arrs = [a for a in arrays if a is not None]
    if all(np.asarray(a).dtype == np.float64 for a in arrs):
        return "_f64", np.float64
    return "_f32", np.float32


def _idx(idx):
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    return idx, idx.ctypes.data_as(ctypes.c_void_p)


# --------------------------------------------------------------------------
# Convolution passes (Sec. 2.1)
# --------------------------------------------------------------------------
def conv_fwd(d: ConvShape, x, w, bias=None, act=ACT_NONE, at=None) -> np.ndarray:
    """y[n,p,q,k] = act(bias[k] + sum_{c,r,s} x[n,p*st+r-pad,q*st+s-pad,c] * w[k,r,s,c]).

    Algorithm 1.  x NHWC, w KRSC.  Returns float64 NPQK, or the values at the
    flat output indices ``at``.
    """
    lib = _load()
    suf, dt = _suffix_dtype(x, w, bias)
    x, xp = _prep(x, dt); w, wp = _prep(w, dt); bias, bp = _prep(bias, dt)
    assert x.size == d.N * d.H * d.W * d.C and w.size == d.K * d.R * d.S * d.C
    cd = d._c()
    if at is None:
        y = np.empty((d.N, d.P, d.Q, d.K), dtype=np.float64)
        getattr(lib, "oracle_conv_fwd" + suf)(ctypes.byref(cd), xp, wp, bp, ctypes.c_int(act),
                                              y.ctypes.data_as(ctypes.c_void_p))
        return y
    idx, ip = _idx(at)
    out = np.empty(idx.size, dtype=np.float64)
    getattr(lib, "oracle_conv_fwd_at" + suf)(ctypes.byref(cd), xp, wp, bp, ctypes.c_int(act), ip,
                                             ctypes.c_int64(idx.size),
                                             out.ctypes.data_as(ctypes.c_void_p))
    return out


def conv_bwd_data(d: ConvShape, dy, w, relu_mask_src=None, at=None) -> np.ndarray:
    """dx = the backpropagation rule of Sec. 2.1 in gather form, optionally
    zeroed where ``relu_mask_src <= 0``.  Returns float64 NHWC (or values at
    flat indices ``at``)."""
    lib = _load()
    suf, dt = _suffix_dtype(dy, w, relu_mask_src)
    dy, gp = _prep(dy, dt); w, wp = _prep(w, dt); m, mp = _prep(relu_mask_src, dt)
    assert dy.size == d.N * d.P * d.Q * d.K and w.size == d.K * d.R * d.S * d.C
    cd = d._c()
    if at is None:
        dx = np.empty((d.N, d.H, d.W, d.C), dtype=np.float64)
        getattr(lib, "oracle_conv_bwd_data" + suf)(ctypes.byref(cd), gp, wp, mp,
                                                   dx.ctypes.data_as(ctypes.c_void_p))
        return dx
    idx, ip = _idx(at)
    out = np.empty(idx.size, dtype=np.float64)
    getattr(lib, "oracle_conv_bwd_data_at" + suf)(ctypes.byref(cd), gp, wp, mp, ip,
                                                  ctypes.c_int64(idx.size),
                                                  out.ctypes.data_as(ctypes.c_void_p))
    return out


def conv_bwd_weights(d: ConvShape, x, dy, want_db=False, at=None):
    """dw[k,r,s,c] = sum_{n,p,q} x[n,p*st+r-pad,q*st+s-pad,c] * dy[n,p,q,k]
    (weight-gradient rule of Sec. 2.1) and db[k] = sum_{n,p,q} dy[n,p,q,k].
    Returns dw (float64 KRSC) or (dw, db); or values at flat KRSC indices ``at``."""
    lib = _load()
    suf, dt = _suffix_dtype(x, dy)
    x, xp = _prep(x, dt); dy, gp = _prep(dy, dt)
    assert x.size == d.N * d.H * d.W * d.C and dy.size == d.N * d.P * d.Q * d.K
    cd = d._c()
    if at is None:
        dw = np.empty((d.K, d.R, d.S, d.C), dtype=np.float64)
        db = np.empty(d.K, dtype=np.float64) if want_db else None
        getattr(lib, "oracle_conv_bwd_weights" + suf)(
            ctypes.byref(cd), xp, gp, dw.ctypes.data_as(ctypes.c_void_p),
            db.ctypes.data_as(ctypes.c_void_p) if want_db else None)
        return (dw, db) if want_db else dw
    idx, ip = _idx(at)
    out = np.empty(idx.size, dtype=np.float64)
    getattr(lib, "oracle_conv_bwd_weights_at" + suf)(ctypes.byref(cd), xp, gp, ip,
                                                     ctypes.c_int64(idx.size),
                                                     out.ctypes.data_as(ctypes.c_void_p))
    return out


# --------------------------------------------------------------------------
# Fully-connected layers: the 1x1-kernel, 1x1-map case of the loops above
# (Sec. 2.1).  w is [K, C]; y = act(x w^T + b).
# --------------------------------------------------------------------------
def _fc_shape(N, C, K) -> ConvShape:
    return ConvShape(N=N, C=C, K=K, H=1, W=1, R=1, S=1)


def fc_fwd(x, w, bias=None, act=ACT_NONE) -> np.ndarray:
    N, C = x.shape
    K = w.shape[0]
    return conv_fwd(_fc_shape(N, C, K), x, w, bias, act).reshape(N, K)


def act_grad(y, dy, act) -> np.ndarray:
    """dz = dy * act'(z) written in terms of the activation output y."""
    y = np.asarray(y, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    if act == ACT_NONE:
        return dy.copy()
    if act == ACT_RELU:
        return np.where(y > 0.0, dy, 0.0)
    if act == ACT_SIGMOID:
        return dy * y * (1.0 - y)
    raise ValueError(act)


def fc_bwd(x, w, y, dy, act=ACT_NONE, dz_dtype=np.float64):
    """Returns (dz, dx, dw, db): dz = dy * act'(y), dx = dz w, dw = dz^T x,
    db = sum_n dz (the 1x1 case of the two update rules of Sec. 2.1), all in
    float64.  A caller that compares against an implementation which stores dz
    in fp32 between the two contractions passes ``dz_dtype=np.float32``: dz is
    then rounded once before it is used."""
    N, C = x.shape
    K = w.shape[0]
    dz = act_grad(y, dy, act).astype(dz_dtype)
    sh = _fc_shape(N, C, K)
    if dz_dtype == np.float64:
        x = np.asarray(x, dtype=np.float64); w = np.asarray(w, dtype=np.float64)
    dx = conv_bwd_data(sh, dz, w).reshape(N, C)
    dw, db = conv_bwd_weights(sh, x, dz, want_db=True)
    return dz, dx, dw.reshape(K, C), db


# --------------------------------------------------------------------------
# SGD (Sec. 1: vanilla, hyper-parameters untouched)
# --------------------------------------------------------------------------
def sgd_update(w, dw, lr) -> np.ndarray:
    """w - lr*dw, with lr taken at fp32 precision as the product path receives it."""
    return np.asarray(w, dtype=np.float64) - float(np.float32(lr)) * np.asarray(dw, dtype=np.float64)


# --------------------------------------------------------------------------
# Glue the topologies need (textbook definitions; not in the paper's analysis)
# --------------------------------------------------------------------------
def maxpool2x2_fwd(x) -> np.ndarray:
    """2x2 window, stride 2, no padding, NHWC; H and W even."""
    x = np.asarray(x, dtype=np.float64)
    N, H, W, C = x.shape
    assert H % 2 == 0 and W % 2 == 0
    v = x.reshape(N, H // 2, 2, W // 2, 2, C)
    return v.max(axis=(2, 4))


def maxpool2x2_bwd(x, dy, relu_mask_src=None) -> np.ndarray:
    """Routes dy to the first maximum of each window in row-major window order
    ((0,0),(0,1),(1,0),(1,1)); then zeroes positions where relu_mask_src <= 0."""
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    N, H, W, C = x.shape
    v = x.reshape(N, H // 2, 2, W // 2, 2, C).transpose(0, 1, 3, 5, 2, 4).reshape(N, H // 2, W // 2, C, 4)
    arg = v.argmax(axis=-1)                       # first max in row-major order
    onehot = (arg[..., None] == np.arange(4)).astype(np.float64)
    g = onehot * dy[..., None]                    # N,P,Q,C,4
    dx = g.reshape(N, H // 2, W // 2, C, 2, 2).transpose(0, 1, 4, 2, 5, 3).reshape(N, H, W, C)
    if relu_mask_src is not None:
        dx = np.where(np.asarray(relu_mask_src, dtype=np.float64) > 0.0, dx, 0.0)
    return dx


def maxpool2x2_codes(x) -> np.ndarray:
    """Position code of each 2x2 window (one byte per pooled element): bits 0-1 = position of the window's first
    maximum in row-major window order (0: (0,0), 1: (0,1), 2: (1,0), 3: (1,1)), bit 2 set where that maximum
    is <= 0 (where a ReLU mask taken from x would zero the routed gradient)."""
    x = np.asarray(x, dtype=np.float64)
    N, H, W, C = x.shape
    v = x.reshape(N, H // 2, 2, W // 2, 2, C).transpose(0, 1, 3, 5, 2, 4).reshape(N, H // 2, W // 2, C, 4)
    arg = v.argmax(axis=-1)
    return (arg + 4 * (v.max(axis=-1) <= 0.0)).astype(np.uint8)


def maxpool2x2_bwd_codes(codes, dy, relu_mask: bool) -> np.ndarray:
    """Routes dy by position codes (maxpool2x2_codes): the coded position of each window gets dy, the other three 0;
    with relu_mask, windows whose code has bit 2 set get 0 everywhere."""
    codes = np.asarray(codes).astype(np.int64)
    dy = np.asarray(dy, dtype=np.float64)
    N, P, Q, C = dy.shape
    g = dy * (codes < 4) if relu_mask else dy
    onehot = ((codes & 3)[..., None] == np.arange(4)).astype(np.float64)
    return (onehot * g[..., None]).reshape(N, P, Q, C, 2, 2).transpose(0, 1, 4, 2, 5, 3).reshape(N, 2 * P, 2 * Q, C)


def softmax_xent(logits, labels):
    """loss = -(1/N) sum_n log softmax(z_n)[label_n];  dz = (softmax(z) - onehot)/N."""
    z = np.asarray(logits, dtype=np.float64)
    N, K = z.shape
    zs = z - z.max(axis=1, keepdims=True)
    e = np.exp(zs)
    sm = e / e.sum(axis=1, keepdims=True)
    lab = np.asarray(labels, dtype=np.int64)
    loss = -np.mean(zs[np.arange(N), lab] - np.log(e.sum(axis=1)))
    dz = sm.copy()
    dz[np.arange(N), lab] -= 1.0
    return float(loss), dz / N


# --------------------------------------------------------------------------
# Parity metric used everywhere: relative L2 and max-abs over RMS(reference)
# --------------------------------------------------------------------------
def parity_errors(got, ref):
    got = np.asarray(got, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    diff = got - ref
    ref_l2 = float(np.sqrt(np.sum(ref * ref)))
    rms = ref_l2 / np.sqrt(max(ref.size, 1))
    rel_l2 = float(np.sqrt(np.sum(diff * diff))) / ref_l2 if ref_l2 > 0 else float(np.sqrt(np.sum(diff * diff)))
    max_over_rms = float(np.max(np.abs(diff))) / rms if rms > 0 else float(np.max(np.abs(diff), initial=0.0))
    return rel_l2, max_over_rms
