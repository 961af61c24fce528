"""Seeded synthetic inputs for the five benchmark workloads.

This module only draws numbers and lays out bucket tables; it contains none of the
method's arithmetic, so both the CUDA path and the test oracle may be fed from it.
The gradients the paper compresses came from training runs that are not available;
these generators reproduce their shapes (worker counts, tensor sizes, value ranges).

Each worker's vector is drawn from torch.Generator(device).manual_seed(1000 * config + worker)
on the requested device; a test that needs identical bytes on host and device
generates once and copies.
"""
from __future__ import annotations

import math
from typing import List, Tuple

import torch

P_INF = 0  # encoding of p = infinity in the C ABI


def resnet50_tensor_sizes() -> List[int]:
    """Parameter-tensor sizes of ResNet-50 in definition order (161 tensors, 25,557,032 entries)."""
    sizes: List[int] = []

    def conv(cin, cout, k):
        sizes.append(cout * cin * k * k)

    def bn(c):
        sizes.extend([c, c])

    conv(3, 64, 7)
    bn(64)
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for blk in range(blocks):
            conv(inplanes, planes, 1)
            bn(planes)
            conv(planes, planes, 3)
            bn(planes)
            conv(planes, planes * 4, 1)
            bn(planes * 4)
            if blk == 0:
                conv(inplanes, planes * 4, 1)
                bn(planes * 4)
            inplanes = planes * 4
    sizes.append(2048 * 1000)
    sizes.append(1000)
    return sizes


def offsets_from_sizes(sizes: List[int]) -> List[int]:
    off = [0]
    for s in sizes:
        off.append(off[-1] + int(s))
    return off


def bert_large_bucket_sizes() -> List[int]:
    """d = 335,141,888 in 25 MiB buckets: 51 of 6,553,600 entries and one of 908,288."""
    return [6_553_600] * 51 + [908_288]


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def config1_vector(worker: int, d: int = 1 << 20, device="cpu") -> torch.Tensor:
    """N(0, 1e-3^2) with 1 % exact zeros (alternating +0 / -0) and 0.1 % exact powers of two."""
    g = _gen(device, 1000 * 1 + worker)
    x = torch.randn(d, generator=g, device=device, dtype=torch.float32) * 1e-3
    u = torch.rand(d, generator=g, device=device, dtype=torch.float32)
    k = torch.randint(-24, 1, (d,), generator=g, device=device)
    sgn = torch.randint(0, 2, (d,), generator=g, device=device).to(torch.float32) * 2.0 - 1.0
    pow2 = sgn * torch.pow(torch.tensor(2.0, device=device), k.to(torch.float32))
    is_zero = u < 0.01
    is_pow2 = (u >= 0.01) & (u < 0.011)
    idx = torch.arange(d, device=device)
    zeros = torch.where(idx % 2 == 0, torch.tensor(0.0, device=device),
                        torch.tensor(-0.0, device=device))
    x = torch.where(is_pow2, pow2, x)
    x = torch.where(is_zero, zeros, x)
    return x.contiguous()


def bucketed_gaussian(sizes: List[int], seed: int, device="cpu") -> torch.Tensor:
    """Tensor l has entries N(0, sigma_l^2), sigma_l = 10^U(-5, -2) (log-uniform)."""
    g = _gen(device, seed)
    B = len(sizes)
    log_sigma = torch.rand(B, generator=g, device=device, dtype=torch.float32) * 3.0 - 5.0
    sigma = torch.pow(torch.tensor(10.0, device=device), log_sigma)
    d = sum(sizes)
    x = torch.randn(d, generator=g, device=device, dtype=torch.float32)
    per_elem = torch.repeat_interleave(sigma, torch.tensor(sizes, device=device))
    return (x * per_elem).contiguous()


def config2_vector(worker: int, device="cpu", sizes=None) -> torch.Tensor:
    """ResNet-50-shaped gradient of one worker (configs 2 and 3 share these buffers)."""
    if sizes is None:
        sizes = resnet50_tensor_sizes()
    return bucketed_gaussian(sizes, 1000 * 2 + worker, device)


def config4_vector(worker: int, d: int = 335_141_888, device="cpu") -> torch.Tensor:
    """1e-4 * Student-t(nu = 3): Z / sqrt((Z1^2 + Z2^2 + Z3^2) / 3)."""
    g = _gen(device, 1000 * 4 + worker)
    z = torch.randn(d, generator=g, device=device, dtype=torch.float32)
    chi = torch.zeros(d, device=device, dtype=torch.float32)
    for _ in range(3):
        zz = torch.randn(d, generator=g, device=device, dtype=torch.float32)
        chi.addcmul_(zz, zz)
        del zz
    chi.div_(3.0).sqrt_()
    z.div_(chi).mul_(1e-4)
    return z.contiguous()


def config5_vector(worker: int, d: int = 1 << 28, device="cpu") -> torch.Tensor:
    """N(0, 1) entries."""
    g = _gen(device, 1000 * 5 + worker)
    return torch.randn(d, generator=g, device=device, dtype=torch.float32).contiguous()


KEEP_1PCT_THRESHOLD = 42_949_673  # round(0.01 * 2^32): selection probability of config 5
KEEP_1PCT_SCALE = 100.0


def small_bucket_table(d: int, seed: int) -> List[int]:
    """A ragged bucket table over [0, d): tiny, unaligned and large buckets mixed (tests)."""
    g = torch.Generator().manual_seed(int(seed))
    off = [0]
    while off[-1] < d:
        kind = int(torch.randint(0, 4, (1,), generator=g))
        if kind == 0:
            step = int(torch.randint(1, 9, (1,), generator=g))
        elif kind == 1:
            step = int(torch.randint(9, 200, (1,), generator=g))
        elif kind == 2:
            step = int(torch.randint(200, 5000, (1,), generator=g))
        else:
            step = int(torch.randint(5000, 40000, (1,), generator=g))
        off.append(min(d, off[-1] + step))
    return off


def describe() -> Tuple[str, ...]:
    return (
        "c1: d=2^20, n=4, N(0,1e-3^2) + 1% zeros + 0.1% powers of two",
        "c2: ResNet-50-shaped, d=25,557,032 in 161 buckets, n=8, sigma_l log-uniform [1e-5,1e-2]",
        "c3: same buffers, D_nat^{2,8}",
        "c4: d=335,141,888 in 25 MiB buckets, n=16, 1e-4 * Student-t(3)",
        "c5: d=2^28, n=8, N(0,1), keep 1% then D_nat^{inf,4}",
    )


assert math.isclose(KEEP_1PCT_THRESHOLD / 2 ** 32, 0.01, rel_tol=1e-8)
