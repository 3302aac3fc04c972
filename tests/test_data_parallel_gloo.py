"""world_size-2 CPU (gloo) test of the data-parallel step (part-reduce / update of the owned strip / part-broadcast,
layer by layer): the partitioning, the hook order, and bit equality with the single-process step on the whole
minibatch (bitwise for the first step, whose sums are all exact; to 1e-12 afterwards).  The step driver here is a small linear network in plain torch on the CPU (test infrastructure standing in
for the CUDA drivers, which need a GPU) with integer-valued data, so that every sum is exact and equality is
bitwise; it uses the library's own parameter store, so the bucket layout is the real one."""
import os
import socket
import subprocess
import sys
import textwrap

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

NET = textwrap.dedent("""
    import torch
    from paper_1602_06709_b200 import networks

    class LinearNet:
        '''y = x W1^T + b1, then W2, b2; loss = mean over the local samples of 0.5 |y - t|^2.'''
        def __init__(self, x, t, dims, lr):
            self.x, self.t, self.lr = x, t, lr
            self.layers = list(zip(dims[:-1], dims[1:]))
            shapes = []
            for C, K in self.layers:
                shapes += [(K, C), (K,)]
            self.store = networks._ParamStore(shapes, device="cpu")
            # float64: the second step multiplies dyadic fractions of the first update; 53 bits keep every sum exact
            self.store.params = self.store.params.double(); self.store.grads = self.store.grads.double()
            g = torch.Generator().manual_seed(1)
            for j, (C, K) in enumerate(self.layers):
                self.store.p(2 * j).copy_(torch.randint(-2, 3, (K, C), generator=g).double())
                self.store.p(2 * j + 1).copy_(torch.randint(-2, 3, (K,), generator=g).double())
            self.log = []
        def param_buckets(self):
            return self.store.layer_buckets()
        def forward(self, before_layer=None):
            a = self.x
            self.acts = []
            for j in range(len(self.layers)):
                if before_layer:
                    before_layer(j)
                self.log.append(("fwd", j))
                self.acts.append(a)
                a = a @ self.store.p(2 * j).t() + self.store.p(2 * j + 1)
            self.y = a
        def backward(self, after_layer=None, after_backprop=None):
            g = (self.y - self.t) / self.x.shape[0]
            for j in reversed(range(len(self.layers))):
                self.store.g(2 * j).copy_(g.t() @ self.acts[j])          # weight gradient first (Sec. 3.1)
                self.store.g(2 * j + 1).copy_(g.sum(dim=0))
                self.log.append(("wgrad", j))
                if after_layer:
                    after_layer(j)
                if j > 0:
                    g = g @ self.store.p(2 * j)                           # reads the OLD weights
                self.log.append(("bprop", j))
                if after_backprop:
                    after_backprop(j)
        def plain_step(self):
            self.forward(); self.backward()
            self.store.params.sub_(self.lr * self.store.grads)

    def data(n):
        g = torch.Generator().manual_seed(7)
        return torch.randint(-3, 4, (n, 24), generator=g).double(), torch.randint(-8, 9, (n, 16), generator=g).double()
""")

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    from paper_1602_06709_b200 import replicas, data_parallel
    exec(open(sys.argv[1]).read())
    world = replicas.init("gloo")
    _, rank, _ = replicas.world()
    N, dims, lr = 16, [24, 40, 16], 2.0 ** -6
    x, t = data(N)
    shard = slice(rank * N // world, (rank + 1) * N // world)
    net = LinearNet(x[shard], t[shard], dims, lr)
    dp = data_parallel.DataParallelStep(net, sgd_fn=lambda w, dw, lr: w.sub_(lr * dw))
    assert dp.exchange.world == world and dp.exchange.rank == rank
    for off, length in net.param_buckets():
        lo, hi = data_parallel.strip_bounds(length, world, rank)
        assert (hi - lo) * world == length and lo %% 4 == 0
    ref = LinearNet(x, t, dims, lr)
    for step in range(3):
        dp.step(); dp.finish()
        ref.plain_step()
        if step == 0:       # every sum of the first step is exact (small integers, power-of-two scales): bit equality
            assert torch.equal(net.store.params, ref.store.params), "step 0: differs from the single-process step"
        else:               # later steps multiply dyadic fractions beyond 53 bits: equal up to the order of the sums
            assert torch.allclose(net.store.params, ref.store.params, rtol=1e-12, atol=0), f"step {step}"
    # every rank holds the same parameters
    both = [torch.zeros_like(net.store.params) for _ in range(world)]
    dist.all_gather(both, net.store.params)
    assert all(torch.equal(b, both[0]) for b in both)
    # order of one step: weight gradient of a layer before its backpropagation
    assert net.log[-4:] == [("wgrad", 1), ("bprop", 1), ("wgrad", 0), ("bprop", 0)]
    replicas.barrier(cuda=False)
    replicas.shutdown()
    print("rank", rank, "ok")
""") % ROOT


@pytest.mark.parametrize("world", [2, 4])
def test_data_parallel_step_equals_single_process_step(tmp_path, world):
    netfile = tmp_path / "net.py"
    netfile.write_text(NET)
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = []
    for rank in range(world):
        env = dict(os.environ, WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD, str(netfile)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_strips_partition_a_bucket():
    from paper_1602_06709_b200 import data_parallel as D
    for world in (1, 2, 4, 8, 16):
        covered = []
        for r in range(world):
            lo, hi = D.strip_bounds(64 * 7, world, r)
            assert lo % D.STRIP_ALIGN == 0
            covered += list(range(lo, hi))
        assert covered == list(range(64 * 7))
    with pytest.raises(ValueError):
        D.strip_bounds(100, 8, 0)


def test_single_process_exchange_is_the_plain_update():
    """Without a process group the exchange degenerates to the SGD update of every bucket: same result as one update
    of the whole store."""
    from paper_1602_06709_b200 import data_parallel as D
    g = torch.Generator().manual_seed(3)
    params = torch.randn(64 * 5, generator=g); grads = torch.randn(64 * 5, generator=g)
    want = params - 0.125 * grads
    ex = D.GradientExchange(params, grads, [(0, 128), (128, 64), (192, 128)], 0.125, lambda w, dw, lr: w.sub_(lr * dw))
    for j in (2, 1, 0):
        ex.gradient_ready(j); ex.weights_free(j)
    ex.wait_all()
    assert torch.equal(params, want)
