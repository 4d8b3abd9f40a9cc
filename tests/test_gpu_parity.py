"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2603_13420_b200 as pskv
from paper_2603_13420_b200.inputs import WORKLOADS, Workload, make_inputs

import parity

pytestmark = pytest.mark.gpu


def wl(name, **kw):
    return dataclasses.replace(WORKLOADS[name], **kw)


# ---------------------------------------------------------------- the five configurations, reduced B
# (sizes the oracle finishes in seconds; each spans several 128-row tiles and ends in a ragged tail)

def test_c0_tiny_forward_full():
    parity.fwd_parity(WORKLOADS["C0"])


@pytest.mark.parametrize("name,B", [("C1", 7), ("C2", 5), ("C3", 3), ("C4", 5)])
def test_forward_reduced_candidates(name, B):
    parity.fwd_parity(wl(name, B=B))


@pytest.mark.parametrize("name,B", [("C4", 5), ("C0", 8), ("C2", 3), ("C3", 2)])
def test_backward_reduced_candidates(name, B):
    parity.bwd_parity(wl(name, B=B, backward=True))


# ---------------------------------------------------------------- full sizes, sampled candidates

@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_forward_full_size_sampled(name):
    w = WORKLOADS[name]
    rng = np.random.default_rng(w.seed)
    cand = sorted(set([0, w.B - 1] + rng.integers(0, w.B, size=4).tolist()))
    parity.fwd_parity(w, cand=cand)


def test_backward_full_size_sampled():
    w = WORKLOADS["C4"]
    rng = np.random.default_rng(w.seed)
    cand = sorted(set([0, w.B - 1] + rng.integers(0, w.B, size=4).tolist()))
    parity.bwd_parity(w, cand=cand)


def test_benchmark_step_full_size_sampled():
    """The exact launches the benchmark's headline times: forward and backward of the GQA layer at
    B = 512, sampled candidates against the oracle."""
    w = wl("C2", backward=True)
    rng = np.random.default_rng(w.seed + 7)
    cand = sorted(set([0, 1, w.B - 1] + rng.integers(0, w.B, size=4).tolist()))
    t = make_inputs(w, with_dout=True)
    parity.fwd_parity(w, t=t, cand=cand)
    parity.bwd_parity(w, t=t, cand=cand)


@pytest.mark.parametrize("name,B", [("C3", 64), ("C2", 64)])
def test_backward_many_tiles_per_cta_sampled(name, B):
    """Backward with several tiles per persistent CTA, so that the prefix K/V rings of the query-side kernel
    wrap across tiles: the long-prefix shape (K and V streaming, 512 tiles for 148 CTAs) and the GQA layer
    shape (K resident, V streaming, 768 tiles).  Sampled candidates against the oracle."""
    w = wl(name, B=B, backward=True)
    rng = np.random.default_rng(w.seed + 11)
    cand = sorted(set([0, B // 2, B - 1] + rng.integers(0, B, size=2).tolist()))
    parity.bwd_parity(w, cand=cand)


# ---------------------------------------------------------------- edge cases and odd shapes

EDGE = [
    # B, Hq, Hkv, S, P, d
    (1, 1, 1, 1, 0, 64),      # a single query that sees only itself
    (3, 4, 4, 8, 0, 128),     # no prefix: plain causal attention per candidate
    (2, 4, 2, 1, 40, 128),    # one suffix token
    (5, 7, 1, 3, 37, 64),     # n_rep = 7, odd S, P not a multiple of 16
    (4, 8, 2, 13, 100, 128),  # odd S with GQA
    (2, 4, 4, 200, 16, 64),   # suffix longer than prefix
    (1, 32, 8, 48, 256, 128), # one candidate of the GQA layer
    (9, 4, 1, 24, 333, 128),  # prefix not a multiple of any tile
    (3, 2, 2, 16, 1, 128),    # one prefix token
    # shapes the tensor-core kernels take (S a multiple of 8)
    (3, 8, 2, 16, 300, 128),  # prefix blocks streamed through the 2-stage ring (d = 128)
    (2, 4, 4, 24, 600, 64),   # prefix blocks streamed through the 4-stage ring (d = 64)
    (5, 7, 1, 8, 37, 64),     # n_rep = 7, partial prefix block
    (6, 4, 2, 128, 20, 64),   # S = 128: a tile is half of one candidate's group
    (3, 2, 2, 72, 50, 128),   # rows per candidate (72) force 72-row tiles
    (40, 4, 4, 8, 16, 128),   # sixteen candidates share one tile
    (37, 2, 1, 40, 129, 128), # ragged last tile, prefix one key past a block
    (2, 8, 2, 64, 64, 128),   # 256 rows per group: two full row tiles of the suffix-gradient kernel, 64 keys
    (2, 8, 1, 40, 32, 128),   # 320 rows per group: two and a half row tiles, n_rep = 8
    (300, 4, 4, 16, 48, 128), # more groups than SMs: every persistent CTA walks over several groups
    # suffixes beyond one key block (forward: tiles inside one candidate, suffix keys in 128-key blocks)
    (2, 8, 2, 256, 100, 128), # 1024 rows per group, two suffix blocks, causal limit inside each
    (1, 8, 2, 512, 0, 128),   # one sequence, no prefix: plain causal self-attention (a prefix prefill)
    (2, 4, 4, 131, 20, 128),  # a prime row count per group: no tiling, general kernels
    (2, 8, 2, 48, 16384, 128),  # a long prefix: 128 key blocks streamed per tile
    (3, 4, 4, 16, 4099, 64),    # long prefix with a ragged last block, head dim 64
]


@pytest.mark.parametrize("shape", EDGE)
def test_forward_edge_shapes(shape):
    B, Hq, Hkv, S, P, d = shape
    w = Workload("edge", 100 + sum(shape), B=B, Hq=Hq, Hkv=Hkv, d=d, P=P, S=S)
    parity.fwd_parity(w, strict_abs=(P + S >= 128))


@pytest.mark.parametrize("shape", EDGE)
def test_backward_edge_shapes(shape):
    B, Hq, Hkv, S, P, d = shape
    w = Workload("edge", 200 + sum(shape), B=B, Hq=Hq, Hkv=Hkv, d=d, P=P, S=S, backward=True)
    parity.bwd_parity(w)


def test_outlier_key_channels_and_large_scores():
    """Large score spread (outlier channels x8 and a 4x scale): exponents far from zero without any
    max subtraction in the tensor-core kernel."""
    w = wl("C2", B=3)
    t = make_inputs(w)
    out, lse, _ = parity.run_fwd_gpu(t, 4 * w.scale)
    ref_out, ref_lse = parity.oracle_fwd(t, 4 * w.scale)
    parity.check_tensor("out", parity.to_f64(out), ref_out, max_abs=4e-2, mean_abs=4e-3,
                        max_rel_of_max=2e-2, mean_rel_of_mean=2e-2)
    parity.check_lse(parity.to_f64(lse), ref_lse)


def _extreme_inputs(kind):
    """Rows whose exponents leave the range the tensor-core kernel handles without a running max:
    they must come back from the redo pass (max subtraction) with the same accuracy."""
    w = Workload("extreme", 777, B=6, Hq=4, Hkv=2, d=128, P=96, S=16)
    t = make_inputs(w)
    q = t["q"].float()
    if kind == "huge":        # scores of +-600 nats in a few rows
        q[1, 2, 3] *= 60.0
        q[4, 0, :] *= 45.0
    elif kind == "negative":  # every score of two rows far below zero (row sums underflow)
        for name in ("prefix_k", "suffix_k"):
            k = t[name].float()
            k[..., 0] = 4.0                     # all keys share a component ...
            t[name] = k.to(torch.bfloat16)
        q[2, 0, 5, 0] = -600.0                  # ... which these queries oppose strongly
        q[2, 1, 15, 0] = -450.0
    return w, dict(t, q=q.to(torch.bfloat16))


@pytest.mark.parametrize("kind", ["huge", "negative"])
def test_rows_outside_the_safe_exponent_range_are_redone(kind):
    w, t = _extreme_inputs(kind)
    out, lse, _ = parity.run_fwd_gpu(t, w.scale)
    ref_out, ref_lse = parity.oracle_fwd(t, w.scale)
    parity.check_tensor("out", parity.to_f64(out), ref_out)
    parity.check_lse(parity.to_f64(lse), ref_lse)
    assert np.abs(ref_lse).max() > 100.0   # the case really is extreme


def test_overflowing_rows_do_not_poison_the_next_tile_through_the_shared_staging_buffer():
    """Head layout of the GQA layer with S = 40: the output staging buffer shares its memory with the
    suffix V buffer, a CTA walks over five tiles, and every fifth tile holds ONE candidate (40 suffix keys
    in a 48-row block, so rows 40..47 of the buffer keep what the previous tile staged there).  Rows
    40..47 and 120..127 of the tile before it overflow (scores of several hundred nats): what they stage
    must be finite, or the next tile's value contraction turns every one of its rows into NaN."""
    w = Workload("alias", 4242, B=64, Hq=32, Hkv=8, d=128, P=256, S=40)
    assert pskv.pskv_kernel_family(0, w.B, w.Hq, w.Hkv, w.S, w.P, w.d) == 1
    t = make_inputs(w)
    q = t["q"].float()
    for g in (0, 5):                       # two KV heads; tile 3 of a head = rows 384..511 of its row list
        q[2, 4 * g + 2, 24:32] *= 60.0     # tile rows 40..47  (candidate 2, third head of the group)
        q[3, 4 * g + 0, 24:32] *= 60.0     # tile rows 120..127 (candidate 3, first head of the group)
    t["q"] = q.to(torch.bfloat16)
    out, lse, _ = parity.run_fwd_gpu(t, w.scale)   # (checks that nothing is NaN or unwritten)
    cand = [1, 2, 3, 4]                    # the overflowing candidates and the one-candidate tile behind them
    ref_out, ref_lse = parity.oracle_fwd(t, w.scale, cand)
    parity.check_tensor("out", parity.to_f64(out[cand]), ref_out, max_abs=4e-2, mean_abs=4e-3)
    parity.check_lse(parity.to_f64(lse[cand]), ref_lse)
    assert np.abs(ref_lse).max() > 100.0


# ---------------------------------------------------------------- properties that hold at any size

def test_candidate_permutation_equivariance():
    """Permuting the candidates permutes the results.  A candidate's position decides which rows
    share its tile and where its suffix keys sit inside the key block, i.e. the fp32 summation
    order, so equality holds up to one rounding of the bf16 result, not bit for bit."""
    w = wl("C1", B=12)
    t = make_inputs(w)
    out0, lse0, _ = parity.run_fwd_gpu(t, w.scale)
    perm = torch.randperm(w.B, generator=torch.Generator().manual_seed(5))
    t2 = dict(t, q=t["q"][perm].contiguous(), suffix_k=t["suffix_k"][perm].contiguous(),
              suffix_v=t["suffix_v"][perm].contiguous())
    out1, lse1, _ = parity.run_fwd_gpu(t2, w.scale)
    a, b = out1.cpu().float(), out0.cpu()[perm].float()
    assert torch.all((a - b).abs() <= 2.0 ** -7 * torch.maximum(a.abs(), b.abs()) + 1e-6)
    assert torch.all((lse1.cpu() - lse0.cpu()[perm]).abs() <= 1e-5)


def test_prefix_is_shared_not_copied():
    """Changing the one prefix tensor changes every candidate's result: there is no per-candidate copy."""
    w = wl("C1", B=6)
    t = make_inputs(w)
    out0, _, _ = parity.run_fwd_gpu(t, w.scale)
    t2 = dict(t, prefix_v=(t["prefix_v"].float() + 1.0).to(torch.bfloat16))
    out1, _, _ = parity.run_fwd_gpu(t2, w.scale)
    diff = (out1.float() - out0.float()).abs().amax(dim=(1, 2, 3))
    assert torch.all(diff > 0.1)


def test_results_do_not_depend_on_workspace_contents_or_repeat():
    w = wl("C4", B=4, backward=True)
    t = make_inputs(w, with_dout=True)
    a = [x.clone() for x in parity.run_bwd_gpu(t, w.scale)]
    b = [x.clone() for x in parity.run_bwd_gpu(t, w.scale)]
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_runs_on_a_side_stream():
    w = WORKLOADS["C0"]
    t = make_inputs(w)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        out, lse, _ = parity.run_fwd_gpu(t, w.scale)
    s.synchronize()
    ref_out, _ = parity.oracle_fwd(t, w.scale)
    parity.check_tensor("out", parity.to_f64(out), ref_out, strict_abs=True)


def test_status_word_is_clean_after_normal_calls():
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
