"""Multi-GPU bookkeeping of the benchmark: the path shards by prefix group with
no exchange step, so ranks only agree on the timing (max over ranks) and add
up the work they did.  Works on any torch.distributed backend (NCCL on GPUs,
gloo in the CPU tests)."""
from __future__ import annotations


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws an independent batch of the same shape."""
    return int(base_seed) + int(rank)


def aggregate(ms: float, flops: float, device="cpu"):
    """(max over ranks of ms, sum over ranks of flops).  No-op without a process group."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), float(flops)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    f = torch.tensor([flops], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t[0]), float(f[0])


def whole_job_tflops(ms: float, flops: float, device="cpu") -> float:
    ms_max, flops_all = aggregate(ms, flops, device)
    return flops_all / (ms_max * 1e-3) / 1e12
