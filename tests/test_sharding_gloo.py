"""The N > 1 path on CPU: two gloo ranks shard the candidates, each evaluates its shard against
a replicated prefix cache (here with the oracle standing in for the device), and the gathered
result equals the unsharded one -- no collective is needed on the data path.  The optional
gradients of the shared prefix cache are the exception: sums over all candidates, so the ranks'
partial results meet in one all-reduce."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_13420_b200 import shard
from paper_2603_13420_b200.inputs import Workload, make_inputs


def test_candidate_ranges_partition_the_batch():
    for B in (0, 1, 5, 8, 512, 513):
        for world in (1, 2, 3, 8):
            covered = []
            for r in range(world):
                lo, hi = shard.candidate_range(B, world, r)
                assert 0 <= lo <= hi <= B
                covered += list(range(lo, hi))
            assert covered == list(range(B))
            sizes = [shard.candidate_range(B, world, r) for r in range(world)]
            assert max(h - l for l, h in sizes) - min(h - l for l, h in sizes) <= 1
    with pytest.raises(ValueError):
        shard.candidate_range(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        w = Workload("shard", 7, B=5, Hq=4, Hkv=2, d=64, P=19, S=6)
        t = make_inputs(w)                      # same seed on every rank: same global batch
        mine = shard.shard_inputs(t, world, rank)
        assert mine["prefix_k"].data_ptr() == t["prefix_k"].data_ptr()  # replicated, not sliced
        f = {k: v.to(torch.float64).numpy() for k, v in mine.items()}
        out, lse = oracle.attn_fwd(f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], w.scale)
        gathered = [None] * world
        dist.all_gather_object(gathered, (rank, out, lse))
        slow = shard.max_over_ranks([1.0 + rank, 5.0 - rank])
        # prefix-cache gradients: each rank's covers its own candidates; one all-reduce sums them
        gen = torch.Generator(device="cpu")
        gen.manual_seed(11)
        dout_full = torch.randn(t["q"].shape, generator=gen, dtype=torch.float64).numpy()
        lo, hi = shard.candidate_range(t["q"].shape[0], world, rank)
        pk_g, pv_g = oracle.attn_bwd_prefix(dout_full[lo:hi], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"],
                                            f["suffix_v"], w.scale)
        dkp, dvp = torch.from_numpy(pk_g).to(torch.float32), torch.from_numpy(pv_g).to(torch.float32)
        shard.allreduce_prefix_gradients(dkp, dvp)
        if rank == 0:
            full = {k: v.to(torch.float64).numpy() for k, v in t.items()}
            ro, rl = oracle.attn_fwd(full["q"], full["prefix_k"], full["prefix_v"], full["suffix_k"],
                                     full["suffix_v"], w.scale)
            go = np.concatenate([g[1] for g in sorted(gathered, key=lambda g: g[0])], axis=0)
            gl = np.concatenate([g[2] for g in sorted(gathered, key=lambda g: g[0])], axis=0)
            ret["ok"] = bool(np.array_equal(go, ro) and np.array_equal(gl, rl))
            fk, fv = oracle.attn_bwd_prefix(dout_full, full["q"], full["prefix_k"], full["prefix_v"], full["suffix_k"],
                                            full["suffix_v"], w.scale)
            ret["prefix_grad_err"] = float(max(np.max(np.abs(dkp.numpy() - fk)), np.max(np.abs(dvp.numpy() - fv))))
            ret["max"] = slow
    finally:
        dist.destroy_process_group()


def test_two_rank_candidate_sharding_matches_unsharded():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
    assert ret["ok"] is True
    assert ret["max"] == [2.0, 5.0]
    assert ret["prefix_grad_err"] < 1e-5   # fp32 all-reduce of fp64-computed partial sums
