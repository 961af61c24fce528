"""Algorithm 1 with the master's work split over the GPUs of one node: every rank is a worker
(Delta_i = C_nat(g_i)) and the master of one contiguous range of coordinates.

    compress        each rank codes its whole vector once (9 bits per entry); the random stream is
                    indexed by the position in the whole vector, so nothing depends on the split
    exchange        rank r needs the codes of its range from every rank: either an all-to-all of
                    the two code planes over NCCL ("collective"), or no copy at all: the aggregate
                    kernel reads the peers' planes in place through peer-mapped pointers
                    ("peer", plain loads over NVLink; planes live in symmetric memory)
    aggregate       nc_aggregate over the n = world code shards in rank order 0..world-1: the
                    same sum, bit for bit, as one GPU aggregating n simulated workers
    return          all-gather of the fp32 range, or, with master compression (g = C_M(Delta),
                    C_M = C_nat), of its 9-bit code followed by one decode launch

All arithmetic runs in the library's kernels; this module only owns buffers, slices them and
calls the collectives.  `codec` is the module that provides nc_compress, nc_aggregate and
nc_aggregate_compress_shard (the CUDA binding unless a test injects another).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

TILE = 1024                      # shards start on a tile boundary: 16-byte aligned plane slices
MASTER_WORKER_ID = 0xFFFF0000    # stream id of C_M, outside the range of worker ranks


@dataclass(frozen=True)
class ShardPlan:
    """Equal shards of a whole number of tiles; the last ranks' shards may reach past d (their
    surplus entries are coded as zeros and dropped at the end)."""
    d: int
    world: int

    def __post_init__(self):
        if self.d < 1 or self.world < 1 or self.world > 64:
            raise ValueError("need d >= 1 and 1 <= world <= 64")

    @property
    def shard(self) -> int:
        per = -(-self.d // self.world)
        return -(-per // TILE) * TILE

    @property
    def padded(self) -> int:
        return self.shard * self.world

    def first(self, rank: int) -> int:
        return rank * self.shard

    def owned(self, rank: int):
        """[lo, hi) of the coordinates inside [0, d) that rank aggregates (empty if lo == hi)."""
        lo = min(self.first(rank), self.d)
        return lo, min(lo + self.shard, self.d)


class NaturalAllReduce:
    """sum_i C_nat(g_i) over the ranks of `group`, every rank receiving the full result.

    transport = "collective": code planes move by all_to_all_single.
    transport = "peer":       planes are allocated in symmetric memory and read in place by the
                              aggregate kernel (needs CUDA peer access between all ranks).
    """

    def __init__(self, d: int, dist, group=None, *, seed: int = 0, transport: str = "collective",
                 master_compress: bool = False, device=None, codec=None, symm_mem=None):
        if transport not in ("collective", "peer"):
            raise ValueError("transport must be 'collective' or 'peer'")
        if codec is None:
            from . import binding as codec          # fails loudly without the built library
        self.codec = codec
        self.dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.plan = ShardPlan(d, self.world)
        self.seed = seed
        self.transport = transport
        self.master_compress = master_compress
        self.device = torch.device(device if device is not None else "cuda")
        P, S = self.plan.padded, self.plan.shard
        dev = self.device
        self._symm = None
        if transport == "peer":
            if symm_mem is None:      # `symm_mem`: what provides empty() and rendezvous()
                import torch.distributed._symmetric_memory as symm_mem
            # one allocation for both planes: exponents, then sign bytes
            self._send = symm_mem.empty(P + P // 8, dtype=torch.uint8, device=dev)
            self._send.zero_()
            self._symm = symm_mem.rendezvous(self._send, group if group is not None
                                             else dist.group.WORLD)
        else:
            self._send = torch.zeros(P + P // 8, dtype=torch.uint8, device=dev)
            self._recv = torch.empty(P + P // 8, dtype=torch.uint8, device=dev)
        self.exp_send = self._send[:P]
        self.sign_send = self._send[P:]
        if master_compress:
            self._mine = torch.empty(S + S // 8, dtype=torch.uint8, device=dev)
            self._all = torch.empty(P + P // 8, dtype=torch.uint8, device=dev)
        else:
            self._out_shard = torch.empty(S, dtype=torch.float32, device=dev)
        self.out = torch.empty(P, dtype=torch.float32, device=dev)

    # ---- the exchange: where rank r finds the codes of its range, one (exp, sign) per rank ----
    def _shards_by_collective(self):
        P, S, W = self.plan.padded, self.plan.shard, self.world
        exp_recv, sign_recv = self._recv[:P], self._recv[P:]
        self.dist.all_to_all_single(exp_recv, self.exp_send, group=self.group)
        self.dist.all_to_all_single(sign_recv, self.sign_send, group=self.group)
        exps = [exp_recv[i * S:(i + 1) * S] for i in range(W)]
        signs = [sign_recv[i * (S // 8):(i + 1) * (S // 8)] for i in range(W)]
        return exps, signs

    def _shards_in_peer_memory(self):
        P, S, W, r = self.plan.padded, self.plan.shard, self.world, self.rank
        self._symm.barrier(channel=0)               # every rank's planes are written
        exps, signs = [], []
        for i in range(W):
            buf = self._symm.get_buffer(i, (P + P // 8,), torch.uint8)
            exps.append(buf[r * S:(r + 1) * S])
            signs.append(buf[P + r * (S // 8):P + (r + 1) * (S // 8)])
        return exps, signs

    def __call__(self, g: torch.Tensor) -> torch.Tensor:
        plan, W, r, c = self.plan, self.world, self.rank, self.codec
        if g.numel() != plan.d or g.dtype != torch.float32:
            raise ValueError("expected an fp32 vector of %d entries" % plan.d)
        P, S = plan.padded, plan.shard
        c.nc_compress(g, plan.d, self.seed, r, self.exp_send, self.sign_send)
        if self.transport == "peer":
            exps, signs = self._shards_in_peer_memory()
        else:
            exps, signs = self._shards_by_collective()
        if self.master_compress:
            my_exp, my_sign = self._mine[:S], self._mine[S:]
            c.nc_aggregate_compress_shard(exps, signs, W, S, plan.first(r), self.seed,
                                          MASTER_WORKER_ID, my_exp, my_sign)
            if self.transport == "peer":
                self._symm.barrier(channel=1)       # peers have read my planes: free to rewrite
            all_exp, all_sign = self._all[:P], self._all[P:]
            self.dist.all_gather_into_tensor(all_exp, my_exp, group=self.group)
            self.dist.all_gather_into_tensor(all_sign, my_sign, group=self.group)
            c.nc_aggregate([all_exp], [all_sign], 1, plan.d, self.out)
        else:
            c.nc_aggregate(exps, signs, W, S, self._out_shard)
            if self.transport == "peer":
                self._symm.barrier(channel=1)
            self.dist.all_gather_into_tensor(self.out, self._out_shard, group=self.group)
        return self.out[:plan.d]

    def wire_bytes_per_rank(self) -> dict:
        """Bytes a rank sends per call (its own shard stays local)."""
        P, S, W = self.plan.padded, self.plan.shard, self.world
        planes = (P + P // 8) * (W - 1) // W
        back = (S + S // 8 if self.master_compress else 4 * S) * (W - 1)
        return {"codes_out": planes, "result_out": back,
                "uncompressed_ring_allreduce": 2 * 4 * P * (W - 1) // W}


def shard_bucket_table(bucket_off, first: int, stop: int):
    """The buckets that overlap the coordinates [first, stop) of the whole vector, as the
    aggregate call of that range needs them: (index of the first overlapping bucket, offsets
    relative to `first`, clipped to the range).  Empty buckets inside the range are kept (their
    offsets repeat); stop <= first gives (0, [0])."""
    if stop <= first:
        return 0, [0]
    B = len(bucket_off) - 1
    b0 = 0
    while b0 + 1 < B and bucket_off[b0 + 1] <= first:
        b0 += 1
    local = [0]
    b = b0
    while b < B and bucket_off[b] < stop:
        local.append(min(bucket_off[b + 1], stop) - first)
        b += 1
    return b0, local


class DitherAllReduce:
    """sum_i D_nat^{p,s}(g_i) over the ranks of `group` with the master's work split as in
    NaturalAllReduce.  Every rank codes its whole vector (per-bucket norms, level nibbles, sign
    bits; the rounding stream is indexed by the position in the whole vector), the norms of all
    ranks are all-gathered (W * B floats), the level and sign planes of a rank's range are
    fetched from every rank (all-to-all or peer pointers), and nd_aggregate runs on the range
    with the bucket table cut to it.  Buckets are never split between compressing ranks, so no
    partial norms are exchanged; a bucket that straddles two ranges is simply decoded by both
    with the same norm."""

    def __init__(self, d: int, bucket_off, dist, group=None, *, p: int = 2, s: int = 8,
                 seed: int = 0, transport: str = "collective", device=None, codec=None,
                 symm_mem=None):
        if transport not in ("collective", "peer"):
            raise ValueError("transport must be 'collective' or 'peer'")
        bucket_off = [int(v) for v in bucket_off]
        if bucket_off[0] != 0 or bucket_off[-1] != d or any(
                a > b for a, b in zip(bucket_off, bucket_off[1:])):
            raise ValueError("bucket_off must ascend from 0 to d")
        if codec is None:
            from . import binding as codec
        self.codec = codec
        self.dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)
        self.plan = ShardPlan(d, self.world)
        self.p, self.s, self.seed = p, s, seed
        self.transport = transport
        self.device = torch.device(device if device is not None else "cuda")
        self.B = len(bucket_off) - 1
        P, S, dev = self.plan.padded, self.plan.shard, self.device
        nbytes = P // 2 + P // 8                      # level nibbles, then sign bytes
        self._symm = None
        if transport == "peer":
            if symm_mem is None:
                import torch.distributed._symmetric_memory as symm_mem
            self._send = symm_mem.empty(nbytes, dtype=torch.uint8, device=dev)
            self._send.zero_()
            self._symm = symm_mem.rendezvous(self._send, group if group is not None
                                             else dist.group.WORLD)
        else:
            self._send = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
            self._recv = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.level_send = self._send[:P // 2]
        self.sign_send = self._send[P // 2:]
        self.off_dev = torch.tensor(bucket_off, dtype=torch.int64, device=dev)
        self.norms_mine = torch.zeros(self.B, dtype=torch.float32, device=dev)
        self.norms_all = torch.zeros(self.world * self.B, dtype=torch.float32, device=dev)
        self.ws_bytes = int(codec.nd_workspace_bytes(d, self.B))
        self.ws = torch.empty(max(self.ws_bytes, 16), dtype=torch.uint8, device=dev)
        lo, hi = self.plan.owned(self.rank)
        self.owned_len = hi - lo
        self.b0, local = shard_bucket_table(bucket_off, lo, hi)
        self.off_local = torch.tensor(local, dtype=torch.int64, device=dev)
        self.B_local = len(local) - 1
        self._out_shard = torch.zeros(S, dtype=torch.float32, device=dev)
        self.out = torch.empty(P, dtype=torch.float32, device=dev)

    def _planes_of_my_range(self):
        P, S, W, r = self.plan.padded, self.plan.shard, self.world, self.rank
        if self.transport == "peer":
            self._symm.barrier(channel=0)
            levels, signs = [], []
            for i in range(W):
                buf = self._symm.get_buffer(i, (P // 2 + P // 8,), torch.uint8)
                levels.append(buf[r * (S // 2):(r + 1) * (S // 2)])
                signs.append(buf[P // 2 + r * (S // 8):P // 2 + (r + 1) * (S // 8)])
            return levels, signs
        level_recv, sign_recv = self._recv[:P // 2], self._recv[P // 2:]
        self.dist.all_to_all_single(level_recv, self.level_send, group=self.group)
        self.dist.all_to_all_single(sign_recv, self.sign_send, group=self.group)
        return ([level_recv[i * (S // 2):(i + 1) * (S // 2)] for i in range(W)],
                [sign_recv[i * (S // 8):(i + 1) * (S // 8)] for i in range(W)])

    def __call__(self, g: torch.Tensor) -> torch.Tensor:
        plan, W, r, c = self.plan, self.world, self.rank, self.codec
        if g.numel() != plan.d or g.dtype != torch.float32:
            raise ValueError("expected an fp32 vector of %d entries" % plan.d)
        c.nd_compress(g, plan.d, self.off_dev, self.B, self.p, self.s, self.seed, r,
                      self.norms_mine, self.level_send, self.sign_send, self.ws, self.ws_bytes)
        self.dist.all_gather_into_tensor(self.norms_all, self.norms_mine, group=self.group)
        levels, signs = self._planes_of_my_range()
        if self.owned_len > 0:
            norms = [self.norms_all[i * self.B + self.b0:(i + 1) * self.B] for i in range(W)]
            c.nd_aggregate(norms, levels, signs, W, self.owned_len, self.off_local, self.B_local,
                           self.s, self._out_shard)
        if self.transport == "peer":
            self._symm.barrier(channel=1)
        self.dist.all_gather_into_tensor(self.out, self._out_shard, group=self.group)
        return self.out[:plan.d]
