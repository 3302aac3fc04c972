"""Hybrid parallelism for fully-connected layers (Sec. 3.3 and 3.4).

The ranks are cut into G groups.  Inside a group the layer is model-parallel:
every rank holds the slice of the weights that belongs to its share of the
INPUT features, multiplies its slice of the activations with it, and a
part-reduce (reduce-scatter) over the group sums the partial outputs and leaves
each rank with its strip of the OUTPUT features -- exactly the slice the next
model-parallel layer needs as input.  In the backward pass a part-broadcast
(all-gather) of the strips of dz rebuilds the full gradient, from which every
rank forms the input gradient and the weight gradient of its own slice with no
further exchange.  Across groups the layer is data-parallel: each group works on
minibatch / G samples, and the ranks that hold the same slice in different
groups sum their weight gradients, update the strip they own and broadcast it
(the exchange of ``data_parallel.GradientExchange`` over that sub-group).

G is chosen by the paper's communication-volume model:
    comms_hybrid(G) = 2 * size * ifm * minibatch / G                  (model part; none if a group is one rank)
                    + size * ofm * ifm * (2 - overlap) * G / N        (data part; none if G == 1)
whose minimum over real G is G = sqrt(N * minibatch / ofm); here the best
divisor of N is taken.

Host logic only: the contractions are the library's FC kernels (injected as
``ops`` so that the CPU tests can run the same schedule with torch matmuls), the
collectives torch.distributed's.
"""
from __future__ import annotations

import math
from typing import List, Optional

import torch
import torch.distributed as dist

from .data_parallel import GradientExchange


def comm_volume(n_ranks: int, groups: int, minibatch: int, ifm: int, ofm: int, overlap: float = 0.0, size: int = 4,
                kernel: int = 1, spatial: int = 1) -> float:
    """Bytes a rank exchanges for one layer under G groups (Sec. 3.3); kernel = k_w * k_h, spatial = in_w * in_h."""
    g = groups
    model = 2.0 * size * ifm * spatial * (minibatch / g) if n_ranks // g > 1 else 0.0
    data = size * ofm * ifm * kernel * (2.0 - overlap) * g / n_ranks if g > 1 else 0.0
    return model + data


def choose_groups(n_ranks: int, minibatch: int, ifm: int, ofm: int, overlap: float = 0.0) -> int:
    """The divisor G of n_ranks (that also divides the minibatch) with the smallest communication volume; ties go to
    the smaller G (larger messages inside the group)."""
    best, best_v = 1, None
    for g in range(1, n_ranks + 1):
        if n_ranks % g or minibatch % g:
            continue
        v = comm_volume(n_ranks, g, minibatch, ifm, ofm, overlap)
        if best_v is None or v < best_v - 1e-9:
            best, best_v = g, v
    return best


def analytic_groups(n_ranks: int, minibatch: int, ofm: int) -> float:
    """The stationary point of comms_hybrid for a fully-connected layer without overlap: sqrt(N * minibatch / ofm)."""
    return math.sqrt(n_ranks * minibatch / ofm)


class TorchOps:
    """Plain torch contractions (CPU tests)."""

    @staticmethod
    def fwd(x, w):
        return x @ w.t()

    @staticmethod
    def bwd(dz, x, w, want_dx=True):
        return (dz @ w if want_dx else None), dz.t() @ x

    @staticmethod
    def sgd(w, dw, lr):
        w.sub_(lr * dw)


class LibraryOps:
    """The library's FC kernels on the current CUDA stream."""

    def __init__(self):
        from . import binding as B
        self.B = B
        self.ws = None

    def _ws(self, n, c, k):
        need = max(self.B.fc_workspace_bytes(n, c, k, self.B.PASS_BWD_DATA), self.B.fc_workspace_bytes(n, c, k, self.B.PASS_FWD), 256)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        return self.ws

    def fwd(self, x, w):
        n, c = x.shape
        k = w.shape[0]
        y = torch.empty(n, k, device=x.device)
        self.B.fc_fwd(n, c, k, x, w, None, y, self.B.ACT_NONE, self._ws(n, c, k))
        return y

    def bwd(self, dz, x, w, want_dx=True):
        n, c = x.shape
        k = w.shape[0]
        dx = torch.empty(n, c, device=x.device) if want_dx else None
        dw = torch.empty(k, c, device=x.device)
        self.B.fc_bwd(n, c, k, x, w, None, self.B.ACT_NONE, dz, dx, dw, None, self._ws(n, c, k))
        return dx, dw

    def sgd(self, w, dw, lr):
        self.B.sgd_update(w, dw, lr)


def _act(y, act):
    return torch.relu(y) if act == "relu" else torch.sigmoid(y) if act == "sigmoid" else y


def _act_grad(y, dy, act):
    return dy * (y > 0).to(dy.dtype) if act == "relu" else dy * y * (1 - y) if act == "sigmoid" else dy


class HybridFc:
    """One fully-connected layer y = act(x w^T + b) under hybrid parallelism.

    world ranks, G groups of M = world / G ranks; rank r is model rank m = r % M of group r // M.  It holds
    w[:, m-th slice of the C inputs] ([K][C/M]) and the m-th strip of the bias ([K/M]); its input is the m-th feature
    slice of the group's minibatch shard ([mb_group][C/M]) and its output the m-th strip of the outputs
    ([mb_group][K/M]).  C, K must be multiples of 4*M (and K/M of 4*G for the data-parallel strips)."""

    def __init__(self, C: int, K: int, groups: int, act: str = "none", lr: float = 0.01, ops=None, w_full=None, b_full=None,
                 dtype=torch.float32, device="cpu"):
        self.world = dist.get_world_size() if dist.is_initialized() else 1
        self.rank = dist.get_rank() if dist.is_initialized() else 0
        assert self.world % groups == 0
        self.G, self.M = groups, self.world // groups
        self.m, self.g = self.rank % self.M, self.rank // self.M
        assert C % (4 * self.M) == 0 and K % (4 * self.M) == 0
        self.C, self.K, self.act, self.lr = C, K, act, lr
        self.ops = ops or TorchOps()
        # sub-groups: every rank takes part in creating all of them (a torch.distributed requirement)
        self.model_group = self.data_group = None
        if self.world > 1:
            for gi in range(self.G):
                grp = dist.new_group([gi * self.M + i for i in range(self.M)])
                if gi == self.g:
                    self.model_group = grp
            for mi in range(self.M):
                grp = dist.new_group([gi * self.M + mi for gi in range(self.G)])
                if mi == self.m:
                    self.data_group = grp
        cs, ks = C // self.M, K // self.M
        # parameters of this rank in one flat store: [K][C/M] weights, then the bias strip (padded to 64 elements)
        n_w = K * cs
        n_b = (ks + 63) // 64 * 64
        self.params = torch.zeros(n_w + n_b, dtype=dtype, device=device)
        self.grads = torch.zeros_like(self.params)
        self.w = self.params[:n_w].view(K, cs)
        self.b = self.params[n_w:n_w + ks]
        self.dw = self.grads[:n_w].view(K, cs)
        self.db = self.grads[n_w:n_w + ks]
        if w_full is not None:
            self.w.copy_(w_full[:, self.m * cs:(self.m + 1) * cs])
        if b_full is not None:
            self.b.copy_(b_full[self.m * ks:(self.m + 1) * ks])
        # data-parallel exchange of this rank's slice among the G ranks that hold the same slice
        self.exchange = None
        if self.G > 1:
            assert n_w % (4 * self.G) == 0 and n_b % (4 * self.G) == 0
            self.exchange = GradientExchange(self.params, self.grads, [(0, n_w), (n_w, n_b)], lr, self.ops.sgd,
                                             self.data_group)
            assert self.exchange.world == self.G and self.exchange.rank == self.g

    # forward: partial products of the input slice, part-reduce over the group
    def forward(self, x_slice: torch.Tensor) -> torch.Tensor:
        self.x = x_slice
        partial = self.ops.fwd(x_slice, self.w)                      # [mb][K]: this slice's share of every output
        ks = self.K // self.M
        if self.M > 1:
            strip = torch.empty(partial.shape[0], ks, dtype=partial.dtype, device=partial.device)
            chunks = [partial[:, i * ks:(i + 1) * ks].contiguous() for i in range(self.M)]
            dist.reduce_scatter(strip, chunks, op=dist.ReduceOp.SUM, group=self.model_group)      # part-reduce
        else:
            strip = partial
        self.y = _act(strip + self.b, self.act)
        return self.y

    # backward: part-broadcast of dz, then local input and weight gradients of the slice
    def backward(self, dy_strip: torch.Tensor, want_dx: bool = True) -> Optional[torch.Tensor]:
        dz_strip = _act_grad(self.y, dy_strip, self.act).contiguous()
        self.db.copy_(dz_strip.sum(dim=0))
        if self.M > 1:
            parts = [torch.empty_like(dz_strip) for _ in range(self.M)]
            dist.all_gather(parts, dz_strip, group=self.model_group)                              # part-broadcast
            dz = torch.cat(parts, dim=1)
        else:
            dz = dz_strip
        dx, dw = self.ops.bwd(dz, self.x, self.w, want_dx)
        self.dw.copy_(dw)
        return dx

    def update(self):
        """Vanilla SGD on the slice, after summing the groups' gradients (each group's loss is its own mean)."""
        if self.exchange is not None:
            for j in (0, 1):
                self.exchange.gradient_ready(j)
                self.exchange.weights_free(j)
            self.exchange.wait_all()
        else:
            self.ops.sgd(self.params, self.grads, self.lr)
