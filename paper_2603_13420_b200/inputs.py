"""Seeded synthetic workloads for shared-prefix attention.

This module serves both the CUDA path and the CPU oracle's tests.  It holds
no attention arithmetic: only the workload table and the random draws.

Workload shapes follow the structure of the paper's attack-scoring loop
(Sec. 4.1, Table 1, Table 8, Appendix A): 7B/8B-class attention heads
(32 query heads, 32 or 8 KV heads, head dim 128), one instruction prefix
shared by hundreds of candidates, and a short per-candidate suffix+target
block behind it.  Values are iid N(0,1) drawn in fp32 from a seeded CPU
generator in the fixed order q, prefix_k, prefix_v, suffix_k, suffix_v, dout
and rounded to bf16 (round-to-nearest-even).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

SEED_BASE = 260313420
OUTLIER_CHANNELS = (5, 37, 69, 101)
OUTLIER_GAIN = 8.0


@dataclass(frozen=True)
class Workload:
    name: str
    index: int
    B: int
    Hq: int
    Hkv: int
    d: int
    P: int
    S: int
    backward: bool = False
    outlier_keys: bool = False
    note: str = ""

    @property
    def n_rep(self) -> int:
        return self.Hq // self.Hkv

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def seed(self) -> int:
        return SEED_BASE + self.index

    def with_candidates(self, B: int) -> "Workload":
        return replace(self, B=B)


WORKLOADS = {
    "C0": Workload("C0", 0, B=8, Hq=4, Hkv=4, d=64, P=32, S=8, note="tiny correctness"),
    "C1": Workload("C1", 1, B=512, Hq=32, Hkv=32, d=128, P=160, S=40,
                   note="Llama-2-7B-shaped MHA layer, 20 suffix + 20 target tokens"),
    "C2": Workload("C2", 2, B=512, Hq=32, Hkv=8, d=128, P=256, S=48, outlier_keys=True,
                   note="Llama-3-8B-shaped GQA layer, 4 outlier key channels x8"),
    "C3": Workload("C3", 3, B=256, Hq=32, Hkv=8, d=128, P=2048, S=32,
                   note="long-prefix stress"),
    "C4": Workload("C4", 4, B=128, Hq=32, Hkv=32, d=128, P=160, S=40, backward=True,
                   note="gradient path on the Llama-2-7B shape"),
}


def _randn_bf16(gen: torch.Generator, shape, outliers: bool = False) -> torch.Tensor:
    x = torch.randn(shape, generator=gen, dtype=torch.float32)
    if outliers:
        for c in OUTLIER_CHANNELS:
            if c < shape[-1]:
                x[..., c] *= OUTLIER_GAIN
    return x.to(torch.bfloat16)


def make_inputs(w: Workload, seed: int | None = None, candidates: int | None = None,
                with_dout: bool | None = None) -> dict:
    """CPU bf16 tensors for workload ``w``.

    ``candidates`` draws only the first few candidates' worth of data for the
    per-candidate tensors; because candidates are drawn as whole tensors the
    result is NOT a prefix of the full draw, so callers that compare two
    implementations must hand both the same dict.
    """
    B = w.B if candidates is None else int(candidates)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed if seed is None else int(seed))
    t = {}
    t["q"] = _randn_bf16(gen, (B, w.Hq, w.S, w.d))
    t["prefix_k"] = _randn_bf16(gen, (w.Hkv, w.P, w.d), w.outlier_keys)
    t["prefix_v"] = _randn_bf16(gen, (w.Hkv, w.P, w.d))
    t["suffix_k"] = _randn_bf16(gen, (B, w.Hkv, w.S, w.d), w.outlier_keys)
    t["suffix_v"] = _randn_bf16(gen, (B, w.Hkv, w.S, w.d))
    if w.backward if with_dout is None else with_dout:
        t["dout"] = _randn_bf16(gen, (B, w.Hq, w.S, w.d))
    return t


def checksum(t: torch.Tensor) -> int:
    """Order-independent 64-bit sum of the raw 16-bit patterns (to show two programs saw the same data)."""
    bits = t.contiguous().view(torch.int16).to(torch.int64) & 0xFFFF
    return int(bits.sum().item())


def fwd_flops(w: Workload) -> float:
    """Algorithmic forward flops: causal-visible multiply-adds only, 4*d per (row, key) pair."""
    rows = w.B * w.Hq * w.S
    return 4.0 * w.d * rows * (w.P + (w.S + 1) / 2.0)


def bwd_flops(w: Workload) -> float:
    """Algorithmic backward flops: 3 contractions on prefix keys (no prefix gradients), 5 on suffix keys."""
    rows = w.B * w.Hq * w.S
    return rows * (6.0 * w.d * w.P + 10.0 * w.d * (w.S + 1) / 2.0)


def fwd_bytes(w: Workload) -> float:
    """Algorithmic forward HBM bytes: every input read once, every output written once."""
    q = w.B * w.Hq * w.S * w.d * 2
    skv = 2 * w.B * w.Hkv * w.S * w.d * 2
    pkv = 2 * w.Hkv * w.P * w.d * 2
    lse = w.B * w.Hq * w.S * 4
    return float(q + skv + pkv + q + lse)


def bwd_bytes(w: Workload) -> float:
    """Algorithmic backward HBM bytes: q, dout, out, lse, K/V in; dq, dk_suffix, dv_suffix out."""
    q = w.B * w.Hq * w.S * w.d * 2
    skv = 2 * w.B * w.Hkv * w.S * w.d * 2
    pkv = 2 * w.Hkv * w.P * w.d * 2
    lse = w.B * w.Hq * w.S * 4
    return float(3 * q + lse + skv + pkv + q + skv)


def kernel_work(w: Workload) -> dict:
    """Algorithmic flops and HBM bytes per launch of each kernel of the tensor-core path
    (every input read once, every output written once; recomputed scores are not counted)."""
    rows = w.B * w.Hq * w.S
    q = rows * w.d * 2
    skv = 2 * w.B * w.Hkv * w.S * w.d * 2
    pkv = 2 * w.Hkv * w.P * w.d * 2
    vis = (w.S + 1) / 2.0
    return {
        "tc_fwd_kernel": {"flops": fwd_flops(w), "bytes": fwd_bytes(w)},
        "tc_bwd_dq_kernel": {"flops": rows * 6.0 * w.d * (w.P + vis), "bytes": float(3 * q + 8 * rows + skv + pkv)},
        # (reads q, dout and out -- it also forms D = <dout, out> --, lse and the suffix K/V; writes D and the gradients)
        "tc_bwd_dkv_kernel": {"flops": rows * (4.0 * w.d * vis + 2.0 * w.d), "bytes": float(3 * q + 8 * rows + 2 * skv)},
        "bwd_dkv_mma_kernel": {"flops": rows * 4.0 * w.d * vis, "bytes": float(2 * q + 8 * rows + 2 * skv)},
        "simt_row_dot_kernel": {"flops": rows * 2.0 * w.d, "bytes": float(2 * q + 4 * rows)},
    }
