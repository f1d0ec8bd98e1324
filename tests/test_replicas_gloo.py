"""The N > 1 host logic (replicas, barrier, max-over-ranks timing) on CPU with gloo, world size 2."""
import os
import socket
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist
    from paper_2310_17723_b200 import replicas, workloads as W
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, lr, w = replicas.rank_info()
    assert (r, lr, w) == (rank, rank, world)
    dist.barrier()
    fake_seconds = 1.0 + 0.5 * rank                       # rank 1 is the slow one
    tmax = replicas.max_over_ranks(fake_seconds, dist)
    x = W.activations(W.tiny_shape(), 1, tensor=replicas.batch_tensor_index(rank))
    dist.barrier()
    out.put((rank, tmax, float(x.sum()), replicas.job_throughput(96, 10, world, tmax)))
    dist.destroy_process_group()


def test_two_replicas_share_only_the_clock():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == 1.5                  # both see the slowest rank's time
    assert res[0][2] != res[1][2]                         # each replica drew its own batch
    assert res[0][3] == pytest.approx(2 * 96 * 10 / 1.5)  # whole-job units / s


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2310_17723_b200 import replicas
    assert replicas.max_over_ranks(0.25) == 0.25
    assert replicas.job_throughput(100, 4, 1, 2.0) == 200.0
