"""Benchmark plumbing shared by bench.py and its tests: rank reduction of timings and the
end-to-end (host buffers) variant of a step.  None of the method's arithmetic lives here."""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The slowest rank's value (multi-GPU numbers are reported as the max over ranks)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist=None, device="cpu") -> float:
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def replica_worker_ids(rank: int, n_workers: int):
    """Replicas are independent: rank r simulates workers r*n .. r*n + n - 1."""
    return [rank * n_workers + w for w in range(n_workers)]


def e2e_host_steps(nc, hp, steps: int, max_pinned_buffers: int = 0) -> dict:
    """Runs `steps` steps with the inputs in pinned host memory: every step copies the n
    gradient vectors host -> device through the C ABI, runs the whole step, and copies the
    step's results (`hp.outputs`) back to pinned host memory.  Returns ms per step and bytes moved.
    `hp` provides n, d, x (list of n device vectors), outputs (device vectors) and step().
    max_pinned_buffers > 0 limits the distinct pinned input buffers (they are then uploaded in
    turn: same bytes per step, less host memory; for several ranks sharing one host).

    Three streams and two sets of device input buffers: the upload of step i + 1 runs while the
    kernels of step i work on the other set and while the results of step i (and i - 1) go back
    (PCIe is full duplex).  An upload waits until the kernels that last read its buffer set are
    done, the kernels of a step wait for their upload and for the download of the previous
    results.  The timed region runs from the first upload to the end of the last download."""
    n, d = hp.n, hp.d
    host_x = []
    try:
        for w in range(n if max_pinned_buffers <= 0 else min(n, max_pinned_buffers)):
            host_x.append(torch.empty(d, dtype=torch.float32, pin_memory=True))
    except RuntimeError:
        # the host cannot pin n vectors: keep what it could, at least two, and upload them in turn
        # (the bytes moved per step stay the same)
        while len(host_x) > 2 and len(host_x) > n // 4:
            host_x.pop()
        if not host_x:
            raise
    for w, buf in enumerate(host_x):
        buf.copy_(hp.x[w])
    outputs = list(hp.outputs)
    host_out = [torch.empty(d, dtype=torch.float32, pin_memory=True) for _ in outputs]
    sets = [hp.x, [torch.empty_like(t) for t in hp.x]]
    torch.cuda.synchronize()
    s_up = torch.cuda.Stream()
    s_main = torch.cuda.Stream()
    s_out = torch.cuda.Stream()
    state = {"downloaded": None, "computed": [None, None], "i": 0}

    def one_step():
        b = state["i"] & 1
        state["i"] += 1
        with torch.cuda.stream(s_up):
            if state["computed"][b] is not None:
                s_up.wait_event(state["computed"][b])       # the set's last readers are done
            for w in range(n):
                nc.nc_copy_to_device(sets[b][w], host_x[w % len(host_x)], 4 * d)
            uploaded = torch.cuda.Event()
            uploaded.record(s_up)
        with torch.cuda.stream(s_main):
            s_main.wait_event(uploaded)
            if state["downloaded"] is not None:
                s_main.wait_event(state["downloaded"])      # outputs may be overwritten now
            hp.x = sets[b]
            hp.step()
            computed = torch.cuda.Event()
            computed.record(s_main)
            state["computed"][b] = computed
        with torch.cuda.stream(s_out):
            s_out.wait_event(computed)
            for dst, src in zip(host_out, outputs):
                nc.nc_copy_to_host(dst, src, 4 * d)
            state["downloaded"] = torch.cuda.Event()
            state["downloaded"].record(s_out)

    one_step()                                   # warm-up (both buffer sets)
    one_step()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(s_up)
    for _ in range(steps):
        one_step()
    e1.record(s_out)
    torch.cuda.synchronize()
    hp.x = sets[0]
    ms = e0.elapsed_time(e1) / steps
    # outside the timed region: what arrived on the host is what the device holds
    arrived = all(torch.equal(dst, src.cpu()) for dst, src in zip(host_out, outputs))
    return {"ms_per_step": ms, "h2d_bytes_per_step": 4 * d * n,
            "d2h_bytes_per_step": 4 * d * len(outputs), "steps": steps,
            "results_arrived": arrived, "distinct_pinned_input_buffers": len(host_x),
            "overlap": "upload of step i+1 overlaps the kernels and the download of step i"}
