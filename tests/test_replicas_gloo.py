"""world_size-2 CPU (gloo) test of the multi-replica plumbing bench.py uses for --gpus N."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np
    from paper_1602_06709_b200 import replicas, inputs
    n = replicas.init("gloo")
    w, rank, _ = replicas.world()
    assert n == 2 and w == 2
    replicas.barrier(cuda=False)
    slow = replicas.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    assert slow == 15.0, slow
    thr = replicas.whole_job_throughput(256, 4, n, slow)
    assert abs(thr - 256 * 4 * 2 / 0.015) < 1e-6
    # every rank draws its own minibatch shard: same recipe, different tensor id
    x = inputs.uniform(inputs.tensor_id("cfg5", "x", rank), (2, 8, 8, 3), 0.0, 1.0)
    import torch, torch.distributed as dist
    both = [torch.zeros(x.size, dtype=torch.float32) for _ in range(2)]
    dist.all_gather(both, torch.from_numpy(x.reshape(-1)))
    assert not torch.equal(both[0], both[1])
    assert torch.equal(both[rank], torch.from_numpy(x.reshape(-1)))
    replicas.barrier(cuda=False)
    replicas.shutdown()
    print("rank", rank, "ok")
""") % ROOT


def test_two_replicas_on_gloo(tmp_path):
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_is_a_no_op():
    from paper_1602_06709_b200 import replicas
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_throughput(10, 2, 1, 100.0) == 200.0
