"""Host-side logic of the N > 1 benchmark path, run as two gloo ranks on CPU: the path does not
exchange data between GPUs (replicas only), so what is distributed is the timing reduction and
the assignment of simulated workers to ranks."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_1905_10988_b200 import timing
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    worst = timing.max_over_ranks(ms, dist, "cpu")
    total = timing.sum_over_ranks(1.0 + rank, dist, "cpu")
    ids = timing.replica_worker_ids(rank, 8)
    gathered = [None] * world
    dist.all_gather_object(gathered, ids)
    if rank == 0:
        out.put((worst, total, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_timing_reduction_and_worker_assignment_two_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    worst, total, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert worst == 15.0                        # the max over ranks, not the mean or rank 0's
    assert total == 3.0
    flat = [w for ids in gathered for w in ids]
    assert sorted(flat) == list(range(16))      # disjoint worker ids: independent random streams


def test_single_process_reductions_are_identity():
    from paper_1905_10988_b200 import timing
    assert timing.max_over_ranks(3.5) == 3.5
    assert timing.sum_over_ranks(2.0, None) == 2.0


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "1"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
