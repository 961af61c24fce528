"""Algorithm 1 with the master sharded over the ranks (paper_1905_10988_b200.sharded).

Host logic (shard plan, buffer slicing, order of the collectives) runs here as gloo ranks on CPU
with the oracle injected as the codec; on a GPU the same flow runs with the CUDA codec: as one
NCCL rank, and as four ranks emulated by host threads that exchange through host-side barriers
(no kernel waits on another).  Expected values come from the oracle on the whole vectors:
sum_i C_nat(g_i) in rank order, optionally followed by C_M = C_nat with the master's stream."""
import os
import socket
import sys
import threading

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle
from paper_1905_10988_b200.sharded import MASTER_WORKER_ID, NaturalAllReduce, ShardPlan

SEED = 0x5EED1905


def gradient(rank: int, d: int) -> np.ndarray:
    rng = np.random.default_rng(1000 + rank)
    x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 1, d)).astype(np.float32)
    x[rng.random(d) < 0.02] = 0.0
    return x


def expected(d: int, world: int, master_compress: bool) -> np.ndarray:
    planes = [oracle.nc_compress(gradient(r, d), SEED, r) for r in range(world)]
    total = oracle.nc_aggregate([p[0] for p in planes], [p[1] for p in planes], d)
    if not master_compress:
        return total
    e, s = oracle.nc_compress(total, SEED, MASTER_WORKER_ID)
    return oracle.nc_aggregate([e], [s], d)


def same_bits(a, b) -> bool:
    return np.array_equal(np.asarray(a, np.float32).view(np.uint32),
                          np.asarray(b, np.float32).view(np.uint32))


# ---- shard plan -------------------------------------------------------------------------------
@pytest.mark.parametrize("d,world", [(1, 1), (1, 4), (1024, 2), (1025, 2), (5000, 3),
                                     (25_557_032, 8), (2 ** 28, 64)])
def test_shard_plan_covers_every_coordinate_once(d, world):
    plan = ShardPlan(d, world)
    assert plan.shard % 1024 == 0 and plan.padded >= d
    assert plan.padded - d < world * 1024 + world          # no more than a tile per rank wasted
    hi_prev = 0
    for r in range(world):
        lo, hi = plan.owned(r)
        assert lo == hi_prev and lo <= hi <= d
        assert plan.first(r) % 1024 == 0
        hi_prev = hi
    assert hi_prev == d


def test_shard_plan_rejects_bad_arguments():
    with pytest.raises(ValueError):
        ShardPlan(0, 2)
    with pytest.raises(ValueError):
        ShardPlan(10, 65)


# ---- the oracle as codec (CPU tensors) --------------------------------------------------------
class OracleCodec:
    @staticmethod
    def nc_compress(x, d, seed, worker, exp, sign):
        e, s = oracle.nc_compress(x.numpy()[:d], seed, worker)
        exp.numpy()[:d] = e
        sign.numpy().view(np.uint32)[:s.size] = s

    @staticmethod
    def nc_aggregate(exps, signs, n, d, out):
        out.numpy()[:d] = oracle.nc_aggregate([e.numpy()[:d] for e in exps[:n]],
                                              [s.numpy().view(np.uint32) for s in signs[:n]], d)

    @staticmethod
    def nc_aggregate_compress_shard(exps, signs, n, d, first, seed, master, out_exp, out_sign):
        total = oracle.nc_aggregate([e.numpy()[:d] for e in exps[:n]],
                                    [s.numpy().view(np.uint32) for s in signs[:n]], d)
        e, s = oracle.nc_compress(total, seed, master, j0=first)
        out_exp.numpy()[:d] = e
        out_sign.numpy().view(np.uint32)[:s.size] = s


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _gloo_rank(rank, world, port, d, master_compress, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ar = NaturalAllReduce(d, dist, seed=SEED, master_compress=master_compress, device="cpu",
                          codec=OracleCodec)
    g = torch.from_numpy(gradient(rank, d))
    first = ar(g).numpy().copy()
    second = ar(g).numpy().copy()                   # buffers are reused: a second call agrees
    out.put((rank, first, second, ar.wire_bytes_per_rank()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,d,master_compress", [(2, 5000, False), (2, 5000, True),
                                                     (3, 7 * 1024 + 5, True), (2, 3, False)])
def test_gloo_ranks_reproduce_the_single_master_result(world, d, master_compress):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gloo_rank, args=(r, world, port, d, master_compress, out))
             for r in range(world)]
    for p in procs:
        p.start()
    got = [out.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    want = expected(d, world, master_compress)
    for rank, first, second, wire in got:
        assert same_bits(first, want), "rank %d differs from the single-master result" % rank
        assert same_bits(second, want)
        assert wire["codes_out"] < wire["uncompressed_ring_allreduce"]


# ---- CUDA codec -------------------------------------------------------------------------------
@pytest.mark.gpu
def test_aggregate_compress_shards_side_by_side_equal_the_whole_vector():
    import paper_1905_10988_b200 as nc
    d, n = 6 * 1024 + 37, 3
    xs = [torch.from_numpy(gradient(r, d)).cuda() for r in range(n)]
    exps = [torch.zeros(nc.nc_exp_bytes(d) + 1024, dtype=torch.uint8, device="cuda") for _ in xs]
    signs = [torch.zeros(nc.nc_sign_bytes(d) + 128, dtype=torch.uint8, device="cuda") for _ in xs]
    for r in range(n):
        nc.nc_compress(xs[r], d, SEED, r, exps[r], signs[r])
    whole_e = torch.zeros(nc.nc_exp_bytes(d), dtype=torch.uint8, device="cuda")
    whole_s = torch.zeros(nc.nc_sign_bytes(d), dtype=torch.uint8, device="cuda")
    nc.nc_aggregate_compress(exps, signs, n, d, SEED, 77, whole_e, whole_s)
    parts_e = torch.full_like(whole_e, 0xCD)
    parts_s = torch.full_like(whole_s, 0xCD)
    for first, length in ((0, 2048), (2048, 3072), (5120, d - 5120)):
        nc.nc_aggregate_compress_shard([e[first:] for e in exps], [s[first // 8:] for s in signs],
                                       n, length, first, SEED, 77, parts_e[first:],
                                       parts_s[first // 8:])
    torch.cuda.synchronize()
    assert torch.equal(parts_e, whole_e) and torch.equal(parts_s, whole_s)
    # and against the oracle
    planes = [oracle.nc_compress(x.cpu().numpy(), SEED, r) for r, x in enumerate(xs)]
    total = oracle.nc_aggregate([p[0] for p in planes], [p[1] for p in planes], d)
    e, s = oracle.nc_compress(total, SEED, 77)
    assert np.array_equal(whole_e.cpu().numpy()[:d], e)
    assert np.array_equal(whole_s.cpu().numpy().view(np.uint32)[:s.size], s)
    with pytest.raises(nc.NatcompError):
        nc.nc_aggregate_compress_shard(exps, signs, n, 64, 512, SEED, 77, parts_e, parts_s)


class ThreadFabric:
    """The two collectives of the flow among `world` host threads of one process that share one
    device and one stream: a thread publishes its tensor, waits at a host barrier, copies its
    part of everybody's tensor.  Stream order equals enqueue order, so no device-side wait."""

    def __init__(self, world):
        self.world = world
        self.local = threading.local()
        self.barrier = threading.Barrier(world)
        self.slots = [None] * world
        self.group = type("group", (), {"WORLD": None})     # what dist.group.WORLD stands for

    def get_rank(self, group=None):
        return self.local.rank

    def get_world_size(self, group=None):
        return self.world

    def _publish(self, t):
        self.slots[self.local.rank] = t
        self.barrier.wait()

    def all_to_all_single(self, out, inp, group=None):
        self._publish(inp)
        n = inp.numel() // self.world
        r = self.local.rank
        for i in range(self.world):
            out[i * n:(i + 1) * n].copy_(self.slots[i][r * n:(r + 1) * n])
        self.barrier.wait()

    def all_gather_into_tensor(self, out, inp, group=None):
        self._publish(inp)
        n = inp.numel()
        for i in range(self.world):
            out[i * n:(i + 1) * n].copy_(self.slots[i])
        self.barrier.wait()


@pytest.mark.gpu
@pytest.mark.parametrize("master_compress", [False, True])
@pytest.mark.parametrize("world,d", [(4, 300_000), (3, 5 * 1024 + 1)])
def test_cuda_codec_four_emulated_ranks(world, d, master_compress):
    fabric = ThreadFabric(world)
    results, errors = [None] * world, []

    def run(rank):
        try:
            fabric.local.rank = rank
            torch.cuda.set_device(0)
            ar = NaturalAllReduce(d, fabric, seed=SEED, master_compress=master_compress)
            g = torch.from_numpy(gradient(rank, d)).cuda()
            ar(g)
            out = ar(g)
            torch.cuda.synchronize()
            results[rank] = out.cpu().numpy()
        except Exception as e:                                  # surfaces in the main thread
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    want = expected(d, world, master_compress)
    for r in range(world):
        assert same_bits(results[r], want), "rank %d" % r


class ThreadSymmetricMemory:
    """Stands in for symmetric memory among the host threads of ThreadFabric: every rank's
    buffer is an ordinary tensor on the one device, get_buffer(i) hands out rank i's, and the
    barrier is the host barrier (all ranks enqueue on one stream, so what was enqueued before
    the barrier runs before what is enqueued after it).  The aggregate kernel then reads the
    other ranks' planes in place, exactly as it reads peer-mapped memory."""

    def __init__(self, fabric):
        self.fabric = fabric
        self.buffers = {}

    def empty(self, *shape, dtype, device):
        return torch.empty(*shape, dtype=dtype, device=device)

    def rendezvous(self, tensor, group=None):
        owner = self
        rank = self.fabric.local.rank
        self.buffers.setdefault(tensor.numel(), [None] * self.fabric.world)[rank] = tensor
        self.fabric.barrier.wait()

        class Handle:
            def barrier(self, channel=0):
                owner.fabric.barrier.wait()

            def get_buffer(self, i, shape, dtype):
                n = 1
                for v in shape:
                    n *= v
                return owner.buffers[tensor.numel()][i][:n].view(dtype)

        return Handle()


@pytest.mark.gpu
@pytest.mark.parametrize("world,d", [(4, 300_000), (3, 5 * 1024 + 1)])
def test_cuda_codec_peer_transport_emulated_ranks(world, d):
    """The "peer" transport with more than one rank: plane slicing, the order of the two barriers
    and the in-place reads of the other ranks' buffers, for C_nat (with and without the master's
    compression) and for D_nat.  Results must equal the single-master result bit for bit."""
    off = bucket_table(d)
    fabric = ThreadFabric(world)
    symm = ThreadSymmetricMemory(fabric)
    results, errors = [None] * world, []

    def run(rank):
        try:
            fabric.local.rank = rank
            torch.cuda.set_device(0)
            g = torch.from_numpy(gradient(rank, d)).cuda()
            outs = []
            for master_compress in (False, True):
                ar = NaturalAllReduce(d, fabric, seed=SEED, transport="peer",
                                      master_compress=master_compress, symm_mem=symm)
                ar(g)
                outs.append(ar(g).cpu().numpy())         # the second call reuses every buffer
            ad = DitherAllReduce(d, off, fabric, p=0, s=4, seed=SEED, transport="peer",
                                 symm_mem=symm)
            ad(g)
            outs.append(ad(g).cpu().numpy())
            torch.cuda.synchronize()
            results[rank] = outs
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    want = [expected(d, world, False), expected(d, world, True),
            expected_dither(d, world, off, 0, 4)]
    for r in range(world):
        for got, ref in zip(results[r], want):
            assert same_bits(got, ref), "rank %d" % r


@pytest.mark.gpu
@pytest.mark.parametrize("transport", ["collective", "peer"])
def test_cuda_codec_one_nccl_rank(transport):
    d = 200_000
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(_free_port())
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    try:
        for master_compress in (False, True):
            ar = NaturalAllReduce(d, dist, seed=SEED, transport=transport,
                                  master_compress=master_compress, device="cuda:0")
            out = ar(torch.from_numpy(gradient(0, d)).cuda())
            torch.cuda.synchronize()
            assert same_bits(out.cpu().numpy(), expected(d, 1, master_compress))
        off = bucket_table(d)
        ad = DitherAllReduce(d, off, dist, p=0, s=4, seed=SEED, transport=transport,
                             device="cuda:0")
        out = ad(torch.from_numpy(gradient(0, d)).cuda())
        torch.cuda.synchronize()
        assert same_bits(out.cpu().numpy(), expected_dither(d, 1, off, 0, 4))
    finally:
        dist.destroy_process_group()


# ---- D_nat over the sharded master -------------------------------------------------------------
from paper_1905_10988_b200.sharded import DitherAllReduce, shard_bucket_table


def bucket_table(d: int):
    rng = np.random.default_rng(d)
    cuts = sorted(set(int(v) for v in rng.integers(1, d, 7)) | {d // 2})
    off = [0] + cuts + [d]
    off.insert(3, off[3])                         # one empty bucket
    return off


def expected_dither(d: int, world: int, off, p: int, s: int) -> np.ndarray:
    parts = [oracle.nd_compress(gradient(r, d), off, p, s, SEED, r) for r in range(world)]
    return oracle.nd_aggregate([q[0] for q in parts], [q[1] for q in parts],
                               [q[2] for q in parts], off, s, d)


def test_shard_bucket_table_cuts_the_global_table():
    off = [0, 100, 100, 3000, 5000]
    assert shard_bucket_table(off, 0, 2048) == (0, [0, 100, 100, 2048])
    assert shard_bucket_table(off, 2048, 4096) == (2, [0, 952, 2048])
    assert shard_bucket_table(off, 4096, 5000) == (3, [0, 904])
    assert shard_bucket_table(off, 5000, 5000) == (0, [0])
    assert shard_bucket_table([0, 10], 0, 10) == (0, [0, 10])
    # every coordinate of every range lands in the bucket the global table gives it
    off = bucket_table(7000)
    for world in (1, 2, 3, 5):
        plan = ShardPlan(7000, world)
        for r in range(world):
            lo, hi = plan.owned(r)
            b0, local = shard_bucket_table(off, lo, hi)
            assert local[0] == 0 and local[-1] == hi - lo
            for j in range(lo, hi, 97):
                want = max(b for b in range(len(off) - 1) if off[b] <= j and j < off[b + 1])
                got = b0 + max(k for k in range(len(local) - 1)
                               if local[k] <= j - lo and j - lo < local[k + 1])
                assert got == want


class OracleDitherCodec:
    @staticmethod
    def nd_workspace_bytes(d, B):
        return 16

    @staticmethod
    def nd_compress(x, d, off, B, p, s, seed, worker, norms, level, sign, ws, wsb):
        nrm, lv, sg = oracle.nd_compress(x.numpy()[:d], off.numpy().astype(np.uint64), p, s, seed,
                                         worker)
        norms.numpy()[:] = nrm
        level.numpy()[:lv.size] = lv
        sign.numpy().view(np.uint32)[:sg.size] = sg

    @staticmethod
    def nd_aggregate(norms, levels, signs, n, d, off, B, s, out):
        out.numpy()[:d] = oracle.nd_aggregate(
            [a.numpy()[:B] for a in norms[:n]], [a.numpy()[:(d + 1) // 2] for a in levels[:n]],
            [a.numpy().view(np.uint32) for a in signs[:n]], off.numpy().astype(np.uint64), s, d)


def _gloo_dither_rank(rank, world, port, d, p, s, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ar = DitherAllReduce(d, bucket_table(d), dist, p=p, s=s, seed=SEED, device="cpu",
                         codec=OracleDitherCodec)
    g = torch.from_numpy(gradient(rank, d))
    ar(g)
    out.put((rank, ar(g).numpy().copy()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,d,p,s", [(2, 6000, 2, 8), (3, 5 * 1024 + 77, 0, 4), (2, 900, 1, 3)])
def test_gloo_ranks_reproduce_the_single_master_dither_sum(world, d, p, s):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gloo_dither_rank, args=(r, world, port, d, p, s, out))
             for r in range(world)]
    for q in procs:
        q.start()
    got = [out.get(timeout=180) for _ in range(world)]
    for q in procs:
        q.join(timeout=180)
        assert q.exitcode == 0
    want = expected_dither(d, world, bucket_table(d), p, s)
    for rank, res in got:
        assert same_bits(res, want), "rank %d differs from the single-master result" % rank


@pytest.mark.gpu
@pytest.mark.parametrize("world,d,p,s", [(4, 300_000, 0, 4), (3, 5 * 1024 + 1, 0, 8),
                                         (4, 300_000, 2, 8)])
def test_cuda_codec_dither_emulated_ranks(world, d, p, s):
    import paper_1905_10988_b200 as nc
    off = bucket_table(d)
    fabric = ThreadFabric(world)
    results, errors = [None] * world, []

    def run(rank):
        try:
            fabric.local.rank = rank
            torch.cuda.set_device(0)
            ar = DitherAllReduce(d, off, fabric, p=p, s=s, seed=SEED)
            g = torch.from_numpy(gradient(rank, d)).cuda()
            ar(g)
            out = ar(g)
            torch.cuda.synchronize()
            results[rank] = out.cpu().numpy()
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    for r in range(1, world):
        assert same_bits(results[r], results[0])
    if p == 0:
        # the max-norm is exact, so the codes and the sum are the oracle's bit for bit
        assert same_bits(results[0], expected_dither(d, world, off, p, s))
    else:
        # p = 2: the norm may differ in the last place, so compare with one GPU aggregating the
        # same W vectors as simulated workers (the same kernels, unsharded)
        B = len(off) - 1
        offd = torch.tensor(off, dtype=torch.int64, device="cuda")
        u8 = dict(dtype=torch.uint8, device="cuda")
        norms = [torch.zeros(B, dtype=torch.float32, device="cuda") for _ in range(world)]
        levels = [torch.zeros(nc.nd_level_bytes(d), **u8) for _ in range(world)]
        signs = [torch.zeros(nc.nc_sign_bytes(d), **u8) for _ in range(world)]
        wsb = nc.nd_workspace_bytes(d, B)
        ws = torch.empty(wsb, **u8)
        for r in range(world):
            nc.nd_compress(torch.from_numpy(gradient(r, d)).cuda(), d, offd, B, p, s, SEED, r,
                           norms[r], levels[r], signs[r], ws, wsb)
        single = torch.empty(d, dtype=torch.float32, device="cuda")
        nc.nd_aggregate(norms, levels, signs, world, d, offd, B, s, single)
        torch.cuda.synchronize()
        assert same_bits(results[0], single.cpu().numpy())
        want = expected_dither(d, world, off, p, s)
        assert np.allclose(results[0], want, rtol=0, atol=1e-5 * np.abs(want).max() + 1e-30) or \
            np.mean(results[0] != want) < 1e-3


@pytest.mark.gpu
def test_allreduce_bench_runs_with_one_rank():
    import json
    import subprocess
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(_free_port()))
    r = subprocess.run([sys.executable, "-m", "paper_1905_10988_b200.allreduce_bench",
                        "--log2-d", "20", "--iters", "2"], env=env, cwd=ROOT,
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert [l["variant"] for l in lines] == ["nccl_allreduce_fp32", "natural_allreduce",
                                             "natural_allreduce_master_compress",
                                             "dither_allreduce_p2_s8"]
    assert all(l["ms"] > 0 and l["n_gpus"] == 1 for l in lines)
