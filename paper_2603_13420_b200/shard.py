"""Candidate sharding across GPUs.

Candidates are independent given the prefix cache (each one reads the shared prefix K/V and
its own suffix K/V only), so the multi-GPU path splits the candidate dimension, replicates
the small prefix cache on every rank and needs no collective on the data path -- the paper's
data-parallel case, where every rank keeps the prefix caches of its local batch and no
all-gather of caches takes place (Appendix G.6).  The one exchange step belongs to the optional
gradients of the shared prefix cache: they are sums over ALL candidates, so each rank's
`pskv_attn_bwd_prefix` result covers only its own candidates and the ranks' results are summed
(`allreduce_prefix_gradients`, one all-reduce of 2 * Hkv * P * d values).  The helpers here are
host-side only.
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


def allreduce_prefix_gradients(dk_prefix: torch.Tensor, dv_prefix: torch.Tensor):
    """Sum the per-rank gradients of the shared prefix cache over all ranks, in place (NCCL on CUDA
    tensors, gloo on CPU tensors).  The sum is taken in fp32: a bf16 all-reduce would round once per
    rank.  No-op without an initialised process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1):
        return dk_prefix, dv_prefix
    both = torch.stack([dk_prefix.to(torch.float32), dv_prefix.to(torch.float32)])
    dist.all_reduce(both, op=dist.ReduceOp.SUM)
    dk_prefix.copy_(both[0])
    dv_prefix.copy_(both[1])
    return dk_prefix, dv_prefix
