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


def test_bench_gpus_flag_starts_its_own_ranks():
    # `python bench.py --gpus 2` outside a torchrun environment launches two ranks itself; without GPUs they meet over
    # gloo.  --rendezvous-only runs the multi-rank plumbing (process group, barrier, max over ranks, rank 0's line)
    # without the CUDA workload.
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rendezvous-only"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                                # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["rendezvous"] == "ok"
    assert d["max_over_ranks"] == 2.0                               # rank 1 reported 2.0 s, rank 0 1.0 s
    assert d["value"] == pytest.approx(2 * 100 / 2.0)
