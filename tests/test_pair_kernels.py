"""GPU parity of the CTA-pair kernels (two SMs share every MMA) against the fp64 oracle, through the
C ABI, plus bit-level agreement checks against the single-CTA kernels where both take a shape."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2603_13420_b200 as pskv
from paper_2603_13420_b200.inputs import WORKLOADS, Workload, make_inputs

import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _pairs_on():
    """The pair kernels are opt-in; every test of this file runs with them switched on."""
    pskv.pskv_enable_cta_pairs(True)
    yield
    pskv.pskv_enable_cta_pairs(False)

# B, Hq, Hkv, S, P: shapes the pair forward takes (head dim 128, a KV head's rows a multiple of 256,
# every 256-row pair tile touching the same number of candidates)
PAIR_SHAPES = [
    (4, 32, 8, 48, 256),    # the GQA layer shape: 192 rows per candidate, two candidates per pair tile
    (8, 8, 2, 48, 256),     # the same geometry with two KV heads: prefix reloaded per head
    (6, 8, 2, 32, 100),     # 128 rows per candidate, partial prefix block (tail of 100 -> 128 keys)
    (4, 8, 2, 64, 37),      # 256 rows per candidate: one candidate per pair tile, its keys split in halves
    (16, 8, 1, 16, 256),    # n_rep = 8, short suffix: 32 suffix keys per pair tile
    (4, 8, 2, 32, 0),       # no prefix: causal attention per candidate on pairs
    (6, 16, 4, 32, 130),    # prefix one key pair past a block: a 32-key tail block
    (8, 8, 1, 16, 384),     # three resident prefix blocks
    (64, 32, 8, 48, 256),   # several pair tiles per CTA pair, KV heads change inside a CTA's range
    (600, 8, 1, 32, 200),   # one KV head, many tiles per pair: long persistent walk, buffer parities wrap
]


def _w(shape, seed, **kw):
    B, Hq, Hkv, S, P = shape
    return Workload("pair", seed, B=B, Hq=Hq, Hkv=Hkv, d=128, P=P, S=S, **kw)


@pytest.mark.parametrize("shape", PAIR_SHAPES)
def test_pair_forward_matches_oracle(shape):
    w = _w(shape, 300 + sum(shape))
    assert pskv.pskv_kernel_family(0, w.B, w.Hq, w.Hkv, w.S, w.P, w.d) == 2
    cand = None
    if w.B > 64:
        rng = np.random.default_rng(w.seed)
        cand = sorted(set([0, 1, w.B - 2, w.B - 1] + rng.integers(0, w.B, size=6).tolist()))
    parity.fwd_parity(w, cand=cand, strict_abs=(w.P + w.S >= 128))


def test_pair_forward_outliers_and_redo_rows():
    """Outlier key channels, and rows whose exponent range forces the max-subtracting redo pass."""
    w = dataclasses.replace(WORKLOADS["C2"], B=8)
    t = make_inputs(w)
    q = t["q"].float()
    q[1, 2, 3] *= 60.0    # scores of several hundred nats
    q[5, 31, 47] *= -60.0
    q[6, 0, 0] *= 45.0
    t["q"] = q.to(torch.bfloat16)
    assert pskv.pskv_kernel_family(0, w.B, w.Hq, w.Hkv, w.S, w.P, w.d) == 2
    out, lse, _ = parity.run_fwd_gpu(t, w.scale)
    ref_out, ref_lse = parity.oracle_fwd(t, w.scale)
    parity.check_tensor("out", parity.to_f64(out), ref_out, max_abs=4e-2, mean_abs=4e-3,
                        max_rel_of_max=2e-2, mean_rel_of_mean=2e-2)
    parity.check_lse(parity.to_f64(lse), ref_lse)


def test_pair_and_single_cta_kernels_agree():
    """Same shape through both kernel families: same tiling of the key blocks, so the results agree to
    the last bits of bf16 (they are not required to be bit-identical: the row sums are added up in a
    different order and the MMAs accumulate 256-row instructions)."""
    w = dataclasses.replace(WORKLOADS["C2"], B=16)
    t = make_inputs(w)
    try:
        out2, lse2, _ = parity.run_fwd_gpu(t, w.scale)
        pskv.pskv_enable_cta_pairs(False)
        assert pskv.pskv_kernel_family(0, w.B, w.Hq, w.Hkv, w.S, w.P, w.d) == 1
        out1, lse1, _ = parity.run_fwd_gpu(t, w.scale)
    finally:
        pskv.pskv_enable_cta_pairs(True)  # (the fixture switches them off again)
    a, b = parity.to_f64(out1), parity.to_f64(out2)
    assert np.max(np.abs(a - b)) <= 2e-2 * max(1.0, float(np.max(np.abs(a))))
    assert np.mean(np.abs(a - b)) <= 1e-4
    assert np.max(np.abs(parity.to_f64(lse1) - parity.to_f64(lse2))) <= 1e-4


def test_pair_forward_full_size_sampled():
    """The launch the benchmark times (B = 512 of the GQA layer), sampled candidates."""
    w = WORKLOADS["C2"]
    rng = np.random.default_rng(w.seed + 1)
    cand = sorted(set([0, 1, w.B - 1] + rng.integers(0, w.B, size=5).tolist()))
    parity.fwd_parity(w, cand=cand)
