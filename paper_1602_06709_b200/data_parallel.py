"""Data-parallel training step over several GPUs of one node (Sec. 3.1 and 3.4).

The minibatch is split over the ranks (one process per GPU); forward and
backward-data need no communication, and every layer's weight gradient needs
one exchange: the per-rank gradients are summed with a *part-reduce*
(reduce-scatter: rank r ends up with the sum of strip r), each rank applies the
SGD update to the strip it owns, and a *part-broadcast* (all-gather) hands every
rank the updated weights (Sec. 3.4).  A layer's part-reduce is issued on a second
stream as soon as that layer's weight gradient is complete (the weight gradient
runs before the layer's backpropagation for this reason, Sec. 3.1), its update
and part-broadcast once the layer's own backpropagation -- the last reader of
the old weights -- has been issued; all of it overlaps the backward pass of the
layers below, and the new weights are only waited for where they are needed,
before that layer's next forward pass (Sec. 3.1).

Plumbing only: the collectives are torch.distributed's (NCCL over NVLink on
GPUs; gloo in the CPU tests), the update is the library's SGD kernel on the
owned strip, and the step drivers of ``networks.py`` provide the per-layer
hooks.  No peer memory is ever handed to a kernel of this library.

The loss of every rank is the mean over its own shard, so the exchanged sum is
divided by the number of ranks inside the update (lr / world): the step equals
the single-process step on the whole minibatch, exactly so when the arithmetic
is exact (the CPU test uses integer-valued data to check bit equality).
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

STRIP_ALIGN = 4      # strips start on 16-byte boundaries


def strip_bounds(length: int, world: int, rank: int) -> Tuple[int, int]:
    """Strip `rank` of a bucket of `length` elements cut into `world` equal strips."""
    if length % (world * STRIP_ALIGN) != 0:
        raise ValueError(f"bucket length {length} is not a multiple of {world} strips x {STRIP_ALIGN} elements")
    s = length // world
    return rank * s, (rank + 1) * s


class GradientExchange:
    """Part-reduce, update of the owned strip, part-broadcast, bucket by bucket.

    params, grads: flat 1-D tensors of equal length (the parameter store of a step driver).
    buckets: (offset, length) per layer, in elements; every length a multiple of world * 4.
    sgd_fn(w_strip, dw_strip, lr): the update, in place on w_strip (the library's kernel on GPUs).
    """

    def __init__(self, params: torch.Tensor, grads: torch.Tensor, buckets: Sequence[Tuple[int, int]], lr: float,
                 sgd_fn: Callable[[torch.Tensor, torch.Tensor, float], None], group=None):
        assert params.dim() == 1 and params.shape == grads.shape
        self.params, self.grads, self.buckets, self.lr, self.sgd_fn, self.group = params, grads, list(buckets), lr, sgd_fn, group
        self.distributed = dist.is_available() and dist.is_initialized()
        self.world = dist.get_world_size(group) if self.distributed else 1
        self.rank = dist.get_rank(group) if self.distributed else 0
        self.cuda = params.is_cuda
        for off, length in self.buckets:
            strip_bounds(length, self.world, self.rank)                 # validates divisibility
            assert 0 <= off and off + length <= params.numel()
        # summed gradient of the owned strip of every bucket (a bucket's part-reduce and its update are separate steps)
        self.strip_off, total = [], 0
        for _, length in self.buckets:
            self.strip_off.append(total)
            total += length // self.world
        self.strip_grad = torch.empty(total if self.world > 1 else 0, dtype=grads.dtype, device=grads.device)
        if self.cuda:
            self.stream = torch.cuda.Stream()
            self.ready: List[Optional[torch.cuda.Event]] = [None] * len(self.buckets)

    # -- called by the step driver -------------------------------------------------------------------------------
    def gradient_ready(self, j: int):
        """Bucket j's gradient is complete on the current stream: start its part-reduce.  The layer's own
        backpropagation, which still reads the old weights, may follow on the current stream meanwhile."""
        off, length = self.buckets[j]
        lo, hi = strip_bounds(length, self.world, self.rank)
        if self.world == 1:
            return
        g = self.grads[off:off + length]
        if self.cuda:
            self._fork()
            with torch.cuda.stream(self.stream):
                dist.reduce_scatter_tensor(self.strip_grad[self.strip_off[j]:self.strip_off[j] + hi - lo], g,
                                           op=dist.ReduceOp.SUM, group=self.group)
        else:
            dist.reduce_scatter_tensor(self.strip_grad[self.strip_off[j]:self.strip_off[j] + hi - lo], g,
                                       op=dist.ReduceOp.SUM, group=self.group)

    def weights_free(self, j: int):
        """Nothing on the current stream reads bucket j's weights any more in this step (its backpropagation has
        been issued): update the owned strip and part-broadcast the new weights."""
        off, length = self.buckets[j]
        lo, hi = strip_bounds(length, self.world, self.rank)
        if self.cuda:
            self._fork()
            with torch.cuda.stream(self.stream):
                self._update(j, off, length, lo, hi)
                ev = torch.cuda.Event()
                ev.record(self.stream)
                self.ready[j] = ev
        else:
            self._update(j, off, length, lo, hi)

    def _fork(self):
        """The exchange stream continues from where the current stream stands."""
        here = torch.cuda.Event()
        here.record()
        self.stream.wait_event(here)

    def wait_weights(self, j: int):
        """Before bucket j's weights are read again (its next forward pass)."""
        if self.cuda and self.ready[j] is not None:
            torch.cuda.current_stream().wait_event(self.ready[j])
            self.ready[j] = None

    def wait_all(self):
        for j in range(len(self.buckets)):
            self.wait_weights(j)

    # -- one bucket ----------------------------------------------------------------------------------------------
    def _update(self, j, off, length, lo, hi):
        w = self.params[off:off + length]
        if self.world > 1:
            sg = self.strip_grad[self.strip_off[j]:self.strip_off[j] + hi - lo]            # filled by the part-reduce
            self.sgd_fn(w[lo:hi], sg, self.lr / self.world)                                 # the mean over the ranks' shards
            dist.all_gather_into_tensor(w, w[lo:hi], group=self.group)                       # part-broadcast (in place)
        else:
            self.sgd_fn(w, self.grads[off:off + length], self.lr)


class DataParallelStep:
    """One synchronous-SGD step of a step driver (networks.VggA / networks.Dnn, or anything with the same
    interface) with the gradient exchange overlapped layer by layer.  The driver must provide
    ``store.params`` / ``store.grads`` (flat), ``param_buckets()`` -> [(offset, length)] in layer order,
    ``forward(before_layer=f)`` calling f(j) before layer j reads its weights, and
    ``backward(after_layer=f, after_backprop=g)`` calling f(j) once layer j's weight and bias gradients are complete
    and g(j) once the layer's backpropagation (the last reader of its old weights) has been issued."""

    def __init__(self, net, sgd_fn=None, group=None):
        self.net = net
        if sgd_fn is None:
            from . import binding as B
            sgd_fn = lambda w, dw, lr: B.sgd_update(w, dw, lr)      # (on the current stream: the exchange's)
        self.exchange = GradientExchange(net.store.params, net.store.grads, net.param_buckets(), net.lr, sgd_fn, group)

    def step(self):
        self.net.forward(before_layer=self.exchange.wait_weights)
        self.net.backward(after_layer=self.exchange.gradient_ready, after_backprop=self.exchange.weights_free)

    def finish(self):
        """Makes the current stream wait for every outstanding weight update (before reading the parameters)."""
        self.exchange.wait_all()
