"""Hybrid parallelism for fully-connected layers (Sec. 3.3): the group-count model against its closed forms, and a
world_size-4 CPU (gloo) run of two chained layers under G = 2 groups x 2 model-parallel ranks (and the pure
model-parallel and pure data-parallel special cases) against the single-process layers on the whole minibatch, bit
for bit (integer-valued data: every sum is exact)."""
import math
import os
import socket
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_group_count_model_matches_the_closed_forms():
    from paper_1602_06709_b200 import hybrid as H
    # stationary point of comms_hybrid for a fully-connected layer (Sec. 3.3): G = sqrt(N * minibatch / ofm)
    assert H.analytic_groups(64, 256, 1024) == 4.0
    assert H.choose_groups(64, 256, 4096, 1024) == 4
    ifm = 4096
    v = H.comm_volume(64, 4, 256, ifm, 1024)
    assert v == 8 * ifm * (256 / 4 + 1024 * 4 / 64)                       # 8 * ifm * (minibatch/G + ofm*G/N)
    assert v < H.comm_volume(64, 1, 256, ifm, 1024) == 8 * ifm * 256      # pure model parallelism
    # pure data parallelism (every group one rank): only the weight exchange, size * ofm * ifm * 2
    assert H.comm_volume(64, 64, 256, ifm, 1024) == 4 * 1024 * ifm * 2
    # the printed rule: model parallelism beats data parallelism for a fully-connected layer whenever ofm > minibatch
    for ofm, mb in ((4096, 256), (1024, 2048)):
        model, data = H.comm_volume(16, 1, mb, 512, ofm), H.comm_volume(16, 16, mb, 512, ofm)
        assert (model < data) == (ofm > mb)
    # brute force over the divisors agrees with the choice, and the choice brackets the analytic optimum
    for n, mb, ofm in ((8, 256, 4096), (8, 1024, 2048), (16, 4096, 1024), (4, 256, 1000)):
        g = H.choose_groups(n, mb, 2048, ofm)
        vols = {d: H.comm_volume(n, d, mb, 2048, ofm) for d in range(1, n + 1) if n % d == 0 and mb % d == 0}
        assert vols[g] == min(vols.values())
        a = H.analytic_groups(n, mb, ofm)
        below = max([d for d in vols if d <= a] or [1]); above = min([d for d in vols if d >= a] or [n])
        assert g in (below, above, 1, n)


CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    from paper_1602_06709_b200 import replicas, hybrid
    world = replicas.init("gloo")
    _, rank, _ = replicas.world()
    G = int(sys.argv[1])
    M = world // G
    mb, dims, lr = 16, [32, 48, 16], 2.0 ** -5
    gen = torch.Generator().manual_seed(5)
    ri = lambda lo, hi, shape: torch.randint(lo, hi + 1, shape, generator=gen).double()
    x, t = ri(-2, 2, (mb, dims[0])), ri(-6, 6, (mb, dims[2]))
    w1, b1, w2, b2 = ri(-1, 1, (dims[1], dims[0])), ri(-2, 2, (dims[1],)), ri(-1, 1, (dims[2], dims[1])), ri(-2, 2, (dims[2],))
    # single-process reference: two layers (ReLU, then linear), loss = mean_n 0.5 |y - t|^2, one vanilla SGD step
    y1 = torch.relu(x @ w1.t() + b1); y2 = y1 @ w2.t() + b2
    d2 = (y2 - t) / mb
    dw2, db2 = d2.t() @ y1, d2.sum(0)
    d1 = (d2 @ w2) * (y1 > 0)
    dw1, db1 = d1.t() @ x, d1.sum(0)
    ref = [w1 - lr * dw1, b1 - lr * db1, w2 - lr * dw2, b2 - lr * db2]
    # hybrid: G groups of M ranks; group g takes samples g*mb/G .., model rank m the m-th feature slice
    g, m = rank // M, rank %% M
    rows = slice(g * mb // G, (g + 1) * mb // G)
    L1 = hybrid.HybridFc(dims[0], dims[1], G, "relu", lr, w_full=w1, b_full=b1, dtype=torch.float64)
    L2 = hybrid.HybridFc(dims[1], dims[2], G, "none", lr, w_full=w2, b_full=b2, dtype=torch.float64)
    assert (L1.G, L1.M, L1.g, L1.m) == (G, M, g, m)
    c0 = dims[0] // M
    a1 = L1.forward(x[rows, m * c0:(m + 1) * c0].contiguous())
    a2 = L2.forward(a1)
    k2 = dims[2] // M
    assert torch.equal(a2, y2[rows, m * k2:(m + 1) * k2])
    dy = (a2 - t[rows, m * k2:(m + 1) * k2]) / (mb // G)               # the group's own mean
    dx2 = L2.backward(dy)
    L1.backward(dx2, want_dx=False)
    L2.update(); L1.update()
    for L, (wr, br), (C, K) in ((L1, ref[0:2], dims[0:2]), (L2, ref[2:4], dims[1:3])):
        cs, ks = C // M, K // M
        assert torch.equal(L.w, wr[:, m * cs:(m + 1) * cs]), "weights slice differs from the single-process step"
        assert torch.equal(L.b, br[m * ks:(m + 1) * ks]), "bias strip differs from the single-process step"
    replicas.barrier(cuda=False)
    replicas.shutdown()
    print("rank", rank, "ok")
""") % ROOT


@pytest.mark.parametrize("groups", [2, 1, 4])      # hybrid; pure model parallelism; pure data parallelism
def test_hybrid_layers_equal_the_single_process_layers(groups):
    world = 4
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = []
    for rank in range(world):
        env = dict(os.environ, WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD, str(groups)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out
