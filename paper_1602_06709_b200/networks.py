"""Step drivers for the two topologies the workloads name: the VGG-A CNN and
the 7-layer fully-connected DNN (Sec. 5).  A driver only owns device buffers
and calls the C ABI in order; all arithmetic happens in the library's kernels.

Per layer the backward pass computes the weight gradient first and the
backpropagated gradient second, and the first layer skips backpropagation
(Sec. 3.1).  Parameters and their gradients live in two flat buffers so that
the SGD update of the whole model is one kernel launch.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from . import binding as B
from . import inputs


def _align(n: int, a: int = 64) -> int:
    return (n + a - 1) // a * a


class _ParamStore:
    """Flat fp32 parameter and gradient buffers with 256-byte aligned views."""

    def __init__(self, shapes: List[tuple], device="cuda", tail=()):
        """tail: indices of the tensors laid out behind all others (the fused-update steps keep there what still takes
        the plain SGD launch: the biases and the first layer's few weights), in index order."""
        self.offsets = [0] * len(shapes)
        off = 0
        tail = sorted(set(tail))
        for i in [i for i in range(len(shapes)) if i not in tail] + tail:
            if tail and i == tail[0]:
                self.tail_offset = off
            self.offsets[i] = off
            off += _align(int(np.prod(shapes[i])))
        if not tail:
            self.tail_offset = off
        self.total = off
        self.shapes = shapes
        self.in_order = not tail
        self.params = torch.zeros(off, device=device)
        self.grads = torch.zeros(off, device=device)

    def view(self, buf, i):
        n = int(np.prod(self.shapes[i]))
        return buf[self.offsets[i]:self.offsets[i] + n].view(self.shapes[i])

    def p(self, i):
        return self.view(self.params, i)

    def g(self, i):
        return self.view(self.grads, i)

    def n_real(self) -> int:
        return sum(int(np.prod(s)) for s in self.shapes)

    def layer_buckets(self):
        """(offset, length) of every (weights, bias) pair: the unit of the data-parallel gradient exchange.  Every
        tensor starts on a 64-element boundary, so a bucket divides into 2, 4, 8 or 16 equal 16-byte aligned strips."""
        assert self.in_order, "the gradient exchange needs the (weights, bias) pairs side by side"
        out = []
        for i in range(0, len(self.shapes), 2):
            end = self.offsets[i + 2] if i + 2 < len(self.shapes) else self.total
            out.append((self.offsets[i], end - self.offsets[i]))
        return out


@dataclass
class _ConvLayer:
    name: str
    C: int
    K: int
    H: int
    W: int
    pool: bool
    desc: object = None

class _GraphStep:
    """A step is a fixed sequence of launches on fixed buffers, so it can be captured once into a CUDA graph and
    replayed with a single launch (the DNN step is ~45 short kernels: issued one by one, the host's launch rate
    bounds it).  One graph per input buffer: the host feed alternates between two."""

    _graphs = None

    def capture_step(self):
        """Call once, after construction (or after any eager steps).  The library's one-time setup (function
        attributes, its device status word) must not fall into the capture, so one eager step runs first, with the
        parameters put back afterwards."""
        saved = self.store.params.clone()
        self.step()
        torch.cuda.synchronize()
        self.store.params.copy_(saved)
        del saved
        self._graphs = {}
        for _ in range(2):
            g = torch.cuda.CUDAGraph()
            n0 = B.launch_count()
            with torch.cuda.graph(g):
                self.step()
            self.graph_launches = B.launch_count() - n0       # kernels one replay launches
            self._graphs[self.x.data_ptr()] = g
            self.x, self._alt_x = self._alt_x, self.x
            self.labels, self._alt_labels = self._alt_labels, self.labels

    def run_step(self):
        """step(), through the captured graph when there is one for the current input buffer."""
        g = self._graphs.get(self.x.data_ptr()) if self._graphs else None
        if g is None:
            self.step()
        else:
            g.replay()


class _HostFeed(_GraphStep):
    """Host-side input feed shared by the step drivers: the minibatch of a step is copied from pinned host
    memory, and the copy of the NEXT minibatch can run on a second stream while this step computes (two
    device input buffers that swap).  Buffers and call order only; no arithmetic of the method."""

    def _feed_init(self):
        self._alt_x = torch.empty_like(self.x)
        self._alt_labels = torch.empty_like(self.labels)
        self._copy_stream = torch.cuda.Stream()
        self._staged = None          # event: the alternate buffers hold the next minibatch

    def step_from_host(self, x_host, labels_host, next_x_host=None, next_labels_host=None) -> float:
        """The call a user makes: pinned host minibatch in, loss out.  If the previous call was given this
        minibatch as its `next_*` arguments, its copy has already been issued and only has to be waited for;
        `next_*` of this call start the copy of the following minibatch before the step is launched."""
        cur = torch.cuda.current_stream()
        if self._staged is not None:
            cur.wait_event(self._staged)
            self.x, self._alt_x = self._alt_x, self.x
            self.labels, self._alt_labels = self._alt_labels, self.labels
            self._staged = None
        else:
            self.x.copy_(x_host, non_blocking=True)
            self.labels.copy_(labels_host, non_blocking=True)
        if next_x_host is not None:
            # the alternate buffers were last read by the previous step, which has finished (its loss was read)
            with torch.cuda.stream(self._copy_stream):
                self._alt_x.copy_(next_x_host, non_blocking=True)
                self._alt_labels.copy_(next_labels_host, non_blocking=True)
                self._staged = torch.cuda.Event()
                self._staged.record(self._copy_stream)
        self.run_step()
        return float(self.loss.cpu().item())


class VggA(_HostFeed):
    """VGG configuration A: eight 3x3 pad-1 convolutions (64,128,256,256,512,512,
    512,512) each followed by ReLU, 2x2 max-pool after conv 1,2,4,6,8, then
    FC 25088-4096-4096-1000 and softmax cross-entropy."""

    def __init__(self, N: int, hw: int = inputs.VGGA_HW, conv=None, fc=None, classes: int = inputs.VGGA_CLASSES,
                 lr: float = 0.01, cfg: str = "cfg5", keep_unpooled: bool = False, fused_update: bool = False):
        """keep_unpooled: also store the full-resolution output of the pooled layers (self.y[i]).  The step never
        reads it (pooling backward and the ReLU mask go by the position codes), so by default it is neither
        allocated nor written where the convolution and the pooling run as one kernel."""
        # fused_update: every layer's weights but the first's are updated by the second pass (or epilogue) of their own
        # weight-gradient call (Sec. 3.1), after the layer's backpropagation has read the old ones; their gradients are
        # never stored, and update() is one small SGD launch over the biases and the first layer's weights.  Not for the
        # data-parallel step, which exchanges the gradients.
        self.fused_update = fused_update
        self.N, self.lr, self.classes = N, lr, classes
        conv = conv if conv is not None else inputs.VGGA_CONV
        self.convs: List[_ConvLayer] = []
        h = hw
        for name, C, K, pool in conv:
            L = _ConvLayer(name, C, K, h, h, pool)
            L.desc = B.conv_desc(N, C, K, h, h, 3, 3, 1, 1)
            self.convs.append(L)
            if pool:
                h //= 2
        self.flat = self.convs[-1].K * h * h
        if fc is None:
            fc = [(self.flat, 4096), (4096, 4096), (4096, classes)]
        assert fc[0][0] == self.flat and fc[-1][1] == classes
        self.fcs = fc
        shapes = []
        for L in self.convs:
            shapes += [(L.K, 3, 3, L.C), (L.K,)]
        for C, K in fc:
            shapes += [(K, C), (K,)]
        self.store = _ParamStore(shapes, tail=([0] + list(range(1, len(shapes), 2))) if fused_update else ())
        nconv = len(self.convs)
        for i, L in enumerate(self.convs):
            w = inputs.he_normal_conv(inputs.tensor_id(cfg, L.name, "w"), L.K, 3, 3, L.C)
            self.store.p(2 * i).copy_(torch.from_numpy(w))
        for j, (C, K) in enumerate(fc):
            w = inputs.he_normal_fc(inputs.tensor_id(cfg, f"fc{j + 1}", "w"), K, C)
            self.store.p(2 * (nconv + j)).copy_(torch.from_numpy(w))
        # activations and gradients
        dev = "cuda"
        self.x = torch.empty(N, hw, hw, self.convs[0].C, device=dev)
        self.y = [None if (L.pool and not keep_unpooled and B.conv_fwd_pool_is_fused(L.desc))
                  else torch.empty(N, L.H, L.W, L.K, device=dev) for L in self.convs]       # post-ReLU
        self.pooled = [torch.empty(N, L.H // 2, L.W // 2, L.K, device=dev) if L.pool else None for L in self.convs]
        # The first layer has no backward-data pass; where it is pooled and the library can take its weight gradient
        # straight from the pooled gradient and the position codes, its full-resolution dy is never formed either.
        self.first_from_pooled = bool(self.convs[0].pool and not keep_unpooled and
                                      B.conv_bwd_weights_pooled_is_fused(self.convs[0].desc))
        self.dy = [None if (i == 0 and self.first_from_pooled) else torch.empty(N, L.H, L.W, L.K, device=dev)
                   for i, L in enumerate(self.convs)]                                          # grad wrt pre-activation
        self.dpooled = [torch.empty(N, L.H // 2, L.W // 2, L.K, device=dev) if L.pool else None for L in self.convs]
        # position codes of the pooling windows (one byte per pooled element), written by the forward epilogue
        self.pool_codes = [torch.empty(N, L.H // 2, L.W // 2, L.K, dtype=torch.uint8, device=dev) if L.pool else None
                           for L in self.convs]
        self.fc_out = [torch.empty(N, K, device=dev) for _, K in fc]
        self.fc_dout = [torch.empty(N, K, device=dev) for _, K in fc]
        self.labels = torch.zeros(N, dtype=torch.int32, device=dev)
        self._feed_init()
        self.loss = torch.zeros(1, device=dev)
        ws = 0
        if self.first_from_pooled:
            ws = B.conv_bwd_weights_pooled_workspace_bytes(self.convs[0].desc)
        for L in self.convs:
            ws = max(ws, B.conv_workspace_bytes(L.desc, B.PASS_FWD), B.conv_workspace_bytes(L.desc, B.PASS_BWD_DATA),
                     B.conv_workspace_bytes(L.desc, B.PASS_BWD_WEIGHTS), B.conv_bwd_data_colsum_workspace_bytes(L.desc),
                     B.maxpool2x2_bwd_colsum_workspace_bytes(N, L.H, L.W, L.K))
        for C, K in fc:
            ws = max(ws, B.fc_workspace_bytes(N, C, K, B.PASS_BWD_DATA), B.fc_workspace_bytes(N, C, K, B.PASS_FWD))
        if fused_update:
            ws = max([ws] + [B.conv_bwd_weights_sgd_workspace_bytes(L.desc) for L in self.convs[1:]] +
                     [B.fc_bwd_fused_sgd_workspace_bytes(N, C, K) for C, K in fc])
        self.ws = torch.empty(max(ws, 256), dtype=torch.uint8, device=dev)
        # The first layer's forward call stages its few-channel input at the start of its workspace; with a workspace
        # of its own, kept until the backward pass, its weight gradient reads that copy instead of staging x again.
        self.ws_first = None
        if self.first_from_pooled and B.conv_staged_input_bytes(self.convs[0].desc) > 0:
            self.ws_first = torch.empty(max(256, B.conv_workspace_bytes(self.convs[0].desc, B.PASS_FWD)), dtype=torch.uint8,
                                        device=dev)
        self.conv_flops_fwd = [2 * N * L.K * L.H * L.W * L.C * 9 for L in self.convs]
        self.fc_flops_fwd = [2 * N * C * K for C, K in fc]

    # -- parameters ---------------------------------------------------------
    def conv_w(self, i): return self.store.p(2 * i)
    def conv_b(self, i): return self.store.p(2 * i + 1)
    def conv_dw(self, i): return self.store.g(2 * i)
    def conv_db(self, i): return self.store.g(2 * i + 1)
    def fc_w(self, j): return self.store.p(2 * (len(self.convs) + j))
    def fc_b(self, j): return self.store.p(2 * (len(self.convs) + j) + 1)
    def fc_dw(self, j): return self.store.g(2 * (len(self.convs) + j))
    def fc_db(self, j): return self.store.g(2 * (len(self.convs) + j) + 1)

    def layer_input(self, i):
        if i == 0:
            return self.x
        prev = self.convs[i - 1]
        return self.pooled[i - 1] if prev.pool else self.y[i - 1]

    # -- one training step --------------------------------------------------
    def param_buckets(self):
        return self.store.layer_buckets()        # conv layers first, then the FC layers: the order of forward()

    def forward(self, before_layer=None):
        """before_layer(j), if given, is called before layer j (convolutions, then FC layers) reads its weights."""
        for i, L in enumerate(self.convs):
            if before_layer:
                before_layer(i)
            if L.pool:      # conv -> ReLU -> 2x2 pool, the maxima taken in the convolution's epilogue
                B.conv_fwd_pool(L.desc, self.layer_input(i), self.conv_w(i), self.conv_b(i), self.y[i], self.pooled[i],
                                B.ACT_RELU, self.ws_first if (i == 0 and self.ws_first is not None) else self.ws,
                                pool_codes=self.pool_codes[i])
            else:
                B.conv_fwd(L.desc, self.layer_input(i), self.conv_w(i), self.conv_b(i), self.y[i], B.ACT_RELU, self.ws)
        a = self.pooled[-1].view(self.N, self.flat)
        for j, (C, K) in enumerate(self.fcs):
            if before_layer:
                before_layer(len(self.convs) + j)
            act = B.ACT_RELU if j + 1 < len(self.fcs) else B.ACT_NONE
            B.fc_fwd(self.N, C, K, a, self.fc_w(j), self.fc_b(j), self.fc_out[j], act, self.ws)
            a = self.fc_out[j]
        B.softmax_xent(self.N, self.classes, self.fc_out[-1], self.labels, self.loss, self.fc_dout[-1])

    def backward(self, after_layer=None, after_backprop=None):
        """after_layer(j), if given, is called once the weight and bias gradients of layer j are complete (its bias
        gradient comes out of the layer above's call, so it is complete by then too); after_backprop(j) once the
        layer's backpropagation, the last reader of its weights in this step, has been issued."""
        nfc = len(self.fcs)
        for j in reversed(range(nfc)):
            C, K = self.fcs[j]
            a = self.fc_out[j - 1] if j > 0 else self.pooled[-1].view(self.N, self.flat)
            dx = self.fc_dout[j - 1] if j > 0 else self.dpooled[-1].view(self.N, self.flat)
            # fc_dout[j] already is dz_j: the softmax gradient for the last layer, and for the others the layer above
            # folded this layer's ReLU gradient and bias gradient into its backpropagation kernel
            if self.fused_update:
                B.fc_bwd_fused_sgd(self.N, C, K, a, self.fc_w(j), None, B.ACT_NONE, self.fc_dout[j], dx,
                                   B.ACT_RELU if j > 0 else B.ACT_NONE, self.fc_db(j - 1) if j > 0 else None, self.lr,
                                   self.fc_db(j) if j + 1 == nfc else None, self.ws)
            else:
                B.fc_bwd_fused(self.N, C, K, a, self.fc_w(j), None, B.ACT_NONE, self.fc_dout[j], dx,
                               B.ACT_RELU if j > 0 else B.ACT_NONE, self.fc_db(j - 1) if j > 0 else None, self.fc_dw(j),
                               self.fc_db(j) if j + 1 == nfc else None, self.ws)
            if after_layer:
                after_layer(len(self.convs) + j)
            if after_backprop:
                after_backprop(len(self.convs) + j)
        for i in reversed(range(len(self.convs))):
            L = self.convs[i]
            # The bias gradient of layer i is the per-map sum of dy[i]; it is formed by whichever kernel writes
            # dy[i] (the pool backward here, or the backward-data pass of layer i+1 below), not by a separate pass.
            if i == 0 and self.first_from_pooled:
                # pooling backward, ReLU mask, bias gradient and weight gradient in one pass over the pooled gradient
                if self.ws_first is not None:
                    B.conv_bwd_weights_pooled_staged(L.desc, self.ws_first, self.dpooled[0], self.pool_codes[0], True,
                                                     self.conv_dw(0), self.conv_db(0), self.ws)
                else:
                    B.conv_bwd_weights_pooled(L.desc, self.layer_input(0), self.dpooled[0], self.pool_codes[0], True,
                                              self.conv_dw(0), self.conv_db(0), self.ws)
                if after_layer:
                    after_layer(0)
                if after_backprop:
                    after_backprop(0)
                continue
            if L.pool:   # gradient through the pool, then through the ReLU (fused mask), routed by the position codes
                B.maxpool2x2_bwd_codes(self.N, L.H, L.W, L.K, self.pool_codes[i], self.dpooled[i], True, self.dy[i],
                                       self.conv_db(i), self.ws)
            if not self.fused_update:      # (Sec. 3.1: the weight gradient first, so that its exchange can start)
                B.conv_bwd_weights(L.desc, self.layer_input(i), self.dy[i], self.conv_dw(i), None, True, self.ws)
                if after_layer:
                    after_layer(i)
            if i > 0:
                prev = self.convs[i - 1]
                if prev.pool:
                    B.conv_bwd_data(L.desc, self.dy[i], self.conv_w(i), None, self.dpooled[i - 1], self.ws)
                else:   # the layer's input is the previous ReLU output: fuse its mask (and its bias gradient)
                    B.conv_bwd_data_colsum(L.desc, self.dy[i], self.conv_w(i), self.y[i - 1], self.dy[i - 1],
                                           self.conv_db(i - 1), self.ws)
            if self.fused_update:          # the old weights have been read: gradient and update in one call
                if i > 0:
                    B.conv_bwd_weights_sgd(L.desc, self.layer_input(i), self.dy[i], self.conv_w(i), self.lr, None, self.ws)
                else:
                    B.conv_bwd_weights(L.desc, self.layer_input(i), self.dy[i], self.conv_dw(i), None, True, self.ws)
                if after_layer:
                    after_layer(i)
            if after_backprop:
                after_backprop(i)

    def update(self):
        t = self.store.tail_offset if self.fused_update else 0
        B.sgd_update(self.store.params[t:], self.store.grads[t:], self.lr)

    def step(self):
        self.forward()
        self.backward()
        self.update()



class Dnn(_HostFeed):
    """Fully-connected DNN: dims[0] inputs, sigmoid hidden layers, linear output
    layer with softmax cross-entropy (the 7-layer ASR network shape of Sec. 5.4)."""

    def __init__(self, N: int, dims=None, lr: float = 0.01, cfg: str = "cfg4", fused_update: bool = False):
        dims = dims if dims is not None else inputs.CFG4_DIMS
        self.N, self.dims, self.lr = N, dims, lr
        self.fused_update = fused_update      # (as in VggA: weights updated by their own weight-gradient call)
        self.layers = list(zip(dims[:-1], dims[1:]))
        shapes = []
        for C, K in self.layers:
            shapes += [(K, C), (K,)]
        self.store = _ParamStore(shapes, tail=list(range(1, len(shapes), 2)) if fused_update else ())
        for j, (C, K) in enumerate(self.layers):
            w = inputs.xavier_uniform_fc(inputs.tensor_id(cfg, f"fc{j + 1}", "w"), K, C)
            self.store.p(2 * j).copy_(torch.from_numpy(w))
        dev = "cuda"
        self.x = torch.empty(N, dims[0], device=dev)
        self.out = [torch.empty(N, K, device=dev) for _, K in self.layers]
        self.dout = [torch.empty(N, K, device=dev) for _, K in self.layers]
        self.labels = torch.zeros(N, dtype=torch.int32, device=dev)
        self._feed_init()
        self.loss = torch.zeros(1, device=dev)
        ws = max(max(B.fc_workspace_bytes(N, C, K, B.PASS_BWD_DATA), B.fc_workspace_bytes(N, C, K, B.PASS_FWD))
                 for C, K in self.layers)
        if fused_update:
            ws = max([ws] + [B.fc_bwd_fused_sgd_workspace_bytes(N, C, K) for C, K in self.layers])
        self.ws = torch.empty(max(ws, 256), dtype=torch.uint8, device=dev)
        self.fc_flops_fwd = [2 * N * C * K for C, K in self.layers]

    def w(self, j): return self.store.p(2 * j)
    def b(self, j): return self.store.p(2 * j + 1)
    def dw(self, j): return self.store.g(2 * j)
    def db(self, j): return self.store.g(2 * j + 1)

    def param_buckets(self):
        return self.store.layer_buckets()

    def forward(self, before_layer=None):
        a = self.x
        n = len(self.layers)
        for j, (C, K) in enumerate(self.layers):
            if before_layer:
                before_layer(j)
            act = B.ACT_SIGMOID if j + 1 < n else B.ACT_NONE
            B.fc_fwd(self.N, C, K, a, self.w(j), self.b(j), self.out[j], act, self.ws)
            a = self.out[j]
        B.softmax_xent(self.N, self.dims[-1], self.out[-1], self.labels, self.loss, self.dout[-1])

    def backward(self, after_layer=None, after_backprop=None):
        n = len(self.layers)
        for j in reversed(range(n)):
            C, K = self.layers[j]
            a = self.out[j - 1] if j > 0 else self.x
            dx = self.dout[j - 1] if j > 0 else None          # first layer: no backpropagation
            # dout[j] already is dz_j (the softmax gradient, or formed by the layer above together with db_j)
            if self.fused_update:
                B.fc_bwd_fused_sgd(self.N, C, K, a, self.w(j), None, B.ACT_NONE, self.dout[j], dx,
                                   B.ACT_SIGMOID if j > 0 else B.ACT_NONE, self.db(j - 1) if j > 0 else None, self.lr,
                                   self.db(j) if j + 1 == n else None, self.ws)
            else:
                B.fc_bwd_fused(self.N, C, K, a, self.w(j), None, B.ACT_NONE, self.dout[j], dx,
                               B.ACT_SIGMOID if j > 0 else B.ACT_NONE, self.db(j - 1) if j > 0 else None, self.dw(j),
                               self.db(j) if j + 1 == n else None, self.ws)
            if after_layer:
                after_layer(j)
            if after_backprop:
                after_backprop(j)

    def update(self):
        t = self.store.tail_offset if self.fused_update else 0
        B.sgd_update(self.store.params[t:], self.store.grads[t:], self.lr)

    def step(self):
        self.forward()
        self.backward()
        self.update()

