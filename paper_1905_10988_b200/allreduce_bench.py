"""Times the compressed all-reduce of `sharded.py` against NCCL's fp32 all-reduce on the ranks of
one node (one process per GPU):

    python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 \
        --master-port P -m paper_1905_10988_b200.allreduce_bench [--log2-d 25] [--transport peer]

Every rank holds one seeded gradient of d fp32 entries.  Timed with CUDA events on the device after
warm-up, max over ranks; rank 0 prints one JSON line per variant.  The NCCL line is the
uncompressed reference point (it computes the exact fp32 sum, the compressed variants compute
sum_i C(g_i)); what is compared is time and bytes on the wire, not values.
"""
from __future__ import annotations

import argparse
import json
import os

import torch
import torch.distributed as dist

from . import workloads
from .sharded import DitherAllReduce, NaturalAllReduce


def _time(fn, iters: int, device) -> float:
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    dist.barrier()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    t = torch.tensor([e0.elapsed_time(e1) / iters], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--log2-d", type=int, default=0,
                    help="vector length 2^LOG2_D (default: the ResNet-50-shaped 25,557,032)")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--transport", default="collective", choices=["collective", "peer"])
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29531")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=device)
    try:
        sizes = workloads.resnet50_tensor_sizes()
        if args.log2_d:
            d = 1 << args.log2_d
            off = [0, d]
            g = torch.randn(d, device=device,
                            generator=torch.Generator(device=device).manual_seed(2000 + rank))
        else:
            off = workloads.offsets_from_sizes(sizes)
            d = off[-1]
            g = workloads.config2_vector(rank, device, sizes)
        plain = g.clone()
        variants = [
            ("nccl_allreduce_fp32", lambda: dist.all_reduce(plain), 8.0 * d * (world - 1) / world),
        ]
        nat = NaturalAllReduce(d, dist, transport=args.transport, device=device)
        natm = NaturalAllReduce(d, dist, transport=args.transport, master_compress=True,
                                device=device)
        dith = DitherAllReduce(d, off, dist, p=2, s=8, transport=args.transport, device=device)
        wire = nat.wire_bytes_per_rank()
        wirem = natm.wire_bytes_per_rank()
        variants += [
            ("natural_allreduce", lambda: nat(g), wire["codes_out"] + wire["result_out"]),
            ("natural_allreduce_master_compress", lambda: natm(g),
             wirem["codes_out"] + wirem["result_out"]),
            ("dither_allreduce_p2_s8", lambda: dith(g),
             (0.625 * nat.plan.padded * (world - 1) / world) + 4.0 * nat.plan.shard * (world - 1)),
        ]
        for name, fn, sent in variants:
            ms = _time(fn, args.iters, device)
            if rank == 0:
                print(json.dumps({"variant": name, "n_gpus": world, "d": d, "ms": round(ms, 4),
                                  "Gelem_per_s": round(d / ms / 1e6, 2),
                                  "bytes_sent_per_rank": int(sent),
                                  "transport": args.transport if name != "nccl_allreduce_fp32"
                                  else "nccl"}), flush=True)
    finally:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
