"""Candidate sharding across GPUs.

Candidates are independent given the prefix cache (each one reads the shared prefix K/V and
its own suffix K/V only), so the multi-GPU path splits the candidate dimension, replicates
the small prefix cache on every rank and needs no collective on the data path -- the paper's
data-parallel case, where every rank keeps the prefix caches of its local batch and no
all-gather of caches takes place (Appendix G.6).  The helpers here are host-side only.
"""
from __future__ import annotations

import torch


def candidate_range(B: int, world: int, rank: int) -> tuple[int, int]:
    """Half-open range of candidates owned by `rank`: contiguous, sizes differ by at most one."""
    if not (0 <= rank < world) or B < 0:
        raise ValueError("bad rank/world/B")
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_inputs(t: dict, world: int, rank: int) -> dict:
    """Slice the per-candidate tensors of an input dict; the prefix tensors are replicated."""
    lo, hi = candidate_range(t["q"].shape[0], world, rank)
    out = {}
    for k, v in t.items():
        out[k] = v if k.startswith("prefix_") else v[lo:hi].contiguous()
    return out


def max_over_ranks(values, device=None):
    """Element-wise max of a list of floats over all ranks (timings are reported as the slowest rank's)."""
    import torch.distributed as dist
    x = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(x, op=dist.ReduceOp.MAX)
    return x.tolist()
