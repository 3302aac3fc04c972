"""Seeded synthetic input tensors.

This module is the only code shared by the CPU oracle's callers and the CUDA
path's callers.  It draws numbers and nothing else: no convolution, GEMM,
activation or update arithmetic lives here.  Every tensor is a pure function of
``(BASE_SEED, tensor_id)`` so both sides see identical fp32 values without any
file being shipped around.

The tensors stand in for the image (ImageNet-1k) and speech (Switchboard)
minibatches of the paper's experiments (Sec. 5): only the shapes and the value
distributions are kept.
"""
from __future__ import annotations

import math
import zlib

import numpy as np

BASE_SEED = 160206709


def tensor_id(*parts) -> int:
    """Stable 32-bit id for a (config, layer, role, ...) tuple."""
    return zlib.crc32("/".join(str(p) for p in parts).encode())


def _gen(tid: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[BASE_SEED, int(tid)]))


def uniform(tid: int, shape, lo: float, hi: float) -> np.ndarray:
    g = _gen(tid)
    out = g.random(size=shape, dtype=np.float32)
    out *= np.float32(hi - lo)
    out += np.float32(lo)
    return out


def normal(tid: int, shape, std: float) -> np.ndarray:
    g = _gen(tid)
    out = g.standard_normal(size=shape, dtype=np.float32)
    out *= np.float32(std)
    return out


def labels(tid: int, n: int, classes: int) -> np.ndarray:
    g = _gen(tid)
    return g.integers(0, classes, size=n, dtype=np.int32)


def he_normal_conv(tid: int, K: int, R: int, S: int, C: int) -> np.ndarray:
    """KRSC weights, std sqrt(2 / (R*S*C))."""
    return normal(tid, (K, R, S, C), math.sqrt(2.0 / (R * S * C)))


def he_normal_fc(tid: int, K: int, C: int) -> np.ndarray:
    return normal(tid, (K, C), math.sqrt(2.0 / C))


def xavier_uniform_fc(tid: int, K: int, C: int) -> np.ndarray:
    a = math.sqrt(6.0 / (C + K))
    return uniform(tid, (K, C), -a, a)


# ---------------------------------------------------------------------------
# Workload tables (shapes only).  Layer tuples are
# (name, C, H, W, K, R, S, stride, pad).
# ---------------------------------------------------------------------------
CFG1 = dict(N=4, C=16, K=32, H=16, W=16, R=3, S=3, stride=1, pad=1)
CFG2 = dict(N=256, C=256, K=256, H=56, W=56, R=3, S=3, stride=1, pad=1)
CFG3_LAYERS = [
    ("C1", 3, 231, 231, 96, 11, 11, 4, 0),
    ("C2", 96, 24, 24, 256, 5, 5, 1, 0),
    ("C3", 256, 12, 12, 512, 3, 3, 1, 1),
    ("C4", 512, 12, 12, 1024, 3, 3, 1, 1),
    ("C5", 1024, 12, 12, 1024, 3, 3, 1, 1),
]
CFG4_DIMS = [440, 2048, 2048, 2048, 2048, 2048, 8192]
CFG4_N = 1024
VGGA_CONV = [  # (name, C, K, pool_after)
    ("conv1", 3, 64, True),
    ("conv2", 64, 128, True),
    ("conv3", 128, 256, False),
    ("conv4", 256, 256, True),
    ("conv5", 256, 512, False),
    ("conv6", 512, 512, True),
    ("conv7", 512, 512, False),
    ("conv8", 512, 512, True),
]
VGGA_FC = [(512 * 7 * 7, 4096), (4096, 4096), (4096, 1000)]
VGGA_HW = 224
VGGA_CLASSES = 1000


def conv_inputs(cfg: str, layer: str, N, C, H, W, K, R, S, P, Q, kind: str):
    """Return (x, w, dy) as fp32 NHWC / KRSC / NPQK arrays.

    kind == "unit":  everything uniform[-1, 1]            (config 1 recipe)
    kind == "train": x uniform[0,1], w He-normal, dy N(0, 1e-3)  (configs 2, 3)
    """
    if kind == "unit":
        x = uniform(tensor_id(cfg, layer, "x"), (N, H, W, C), -1.0, 1.0)
        w = uniform(tensor_id(cfg, layer, "w"), (K, R, S, C), -1.0, 1.0)
        dy = uniform(tensor_id(cfg, layer, "dy"), (N, P, Q, K), -1.0, 1.0)
    elif kind == "train":
        x = uniform(tensor_id(cfg, layer, "x"), (N, H, W, C), 0.0, 1.0)
        w = he_normal_conv(tensor_id(cfg, layer, "w"), K, R, S, C)
        dy = normal(tensor_id(cfg, layer, "dy"), (N, P, Q, K), 1e-3)
    else:
        raise ValueError(kind)
    return x, w, dy
