"""Seeded random shapes through every call shape (full suffix, decode-shaped, ragged decode) against the
fp64 oracle: sizes on and around the tiling boundaries (suffix and cache lengths 1..300, prefixes 0..600,
1..7 query heads per KV head, both head dims), so that each geometry the planner can pick -- resident or
streamed prefix, whole-candidate tiles, tiles inside one candidate, the general kernels -- is met."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity


def shape(rng):
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4]))
    n_rep = int(rng.choice([1, 2, 4, 7]))
    Skv = int(rng.choice([1, 3, 8, 16, 24, 40, 48, 64, 100, 128, 130, 200, 256, 300]))
    decode = rng.random() < 0.5
    Sq = int(rng.integers(1, Skv + 1)) if decode else Skv
    if decode and rng.random() < 0.5:
        Sq = min(int(rng.choice([1, 2, 4, 8])), Skv)
    P = int(rng.choice([0, 1, 17, 64, 128, 129, 200, 256, 300, 600]))
    B = int(rng.integers(1, 40))
    while B * Hkv * n_rep * Sq * (P + Skv) * d > 4e8 and B > 1:   # keeps the oracle to a fraction of a second
        B = max(1, B // 2)
    ragged = decode and rng.random() < 0.6
    return B, Hkv * n_rep, Hkv, Sq, Skv, P, d, decode, ragged


CASES = [shape(np.random.default_rng(4200 + i)) for i in range(36)]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
def test_random_shape_matches_the_oracle(case):
    B, Hq, Hkv, Sq, Skv, P, d, decode, ragged = case
    gen = torch.Generator(device="cpu")
    gen.manual_seed(sum(int(x) for x in case) + 17)
    draw = lambda *s: torch.randn(s, generator=gen, dtype=torch.float32).to(torch.bfloat16)
    q, pk, pv = draw(B, Hq, Sq, d), draw(Hkv, P, d), draw(Hkv, P, d)
    sk, sv, do = draw(B, Hkv, Skv, d), draw(B, Hkv, Skv, d), draw(B, Hq, Sq, d)
    lens = torch.randint(Sq, Skv + 1, (B,), generator=gen, dtype=torch.int32) if ragged else None
    if ragged:
        for b in range(B):
            sk[b, :, int(lens[b]):] = 3.0e4
            sv[b, :, int(lens[b]):] = -3.0e4
    scale = 1 / math.sqrt(d)
    dev = lambda x: None if x is None or x.numel() == 0 else x.cuda()
    if decode:
        out, lse = pskv.pskv_attn_fwd_decode(q.cuda(), dev(pk), dev(pv), sk.cuda(), sv.cuda(), dev(lens), scale)
        dq, dk, dv = pskv.pskv_attn_bwd_decode(do.cuda(), q.cuda(), dev(pk), dev(pv), sk.cuda(), sv.cuda(), dev(lens),
                                               out, lse, scale)
    else:
        out, lse = pskv.pskv_attn_fwd(q.cuda(), dev(pk), dev(pv), sk.cuda(), sv.cuda(), scale)
        dq, dk, dv = pskv.pskv_attn_bwd(do.cuda(), q.cuda(), dev(pk), dev(pv), sk.cuda(), sv.cuda(), out, lse, scale)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    f = lambda x: x.to(torch.float64).numpy()
    nl = None if lens is None else lens.numpy()
    ro, rl = oracle.attn_fwd_decode(f(q), f(pk), f(pv), f(sk), f(sv), scale, nl)
    rq, rk, rv = oracle.attn_bwd_decode(f(do), f(q), f(pk), f(pv), f(sk), f(sv), scale, nl)
    parity.check_tensor("out", parity.to_f64(out), ro, strict_abs=False)
    parity.check_lse(parity.to_f64(lse), rl)
    parity.check_tensor("dq", parity.to_f64(dq), rq)
    parity.check_tensor("dk_suffix", parity.to_f64(dk), rk)
    parity.check_tensor("dv_suffix", parity.to_f64(dv), rv)


def multi_shape(rng):
    d = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4]))
    n_rep = int(rng.choice([1, 2, 4]))
    S = int(rng.choice([8, 16, 24, 32, 40, 48, 64]))
    Bp = int(rng.choice([2, 3, 4, 5, 8]))
    Kq = int(rng.choice([1, 2, 4, 8, 16]))
    Pmax = int(rng.choice([16, 64, 100, 128, 129, 256, 300, 600]))
    lens = [int(rng.integers(0, Pmax + 1)) for _ in range(Bp)]
    lens[int(rng.integers(0, Bp))] = Pmax
    form = "one" if rng.random() < 0.7 else "passes"
    return Bp * Kq, Bp, Hkv * n_rep, Hkv, S, Pmax, d, tuple(lens), form


MULTI_CASES = [multi_shape(np.random.default_rng(5200 + i)) for i in range(24)]


@pytest.mark.gpu
@pytest.mark.parametrize("case", MULTI_CASES)
def test_random_multi_instruction_shape_matches_the_oracle(case, monkeypatch):
    """Several instructions with random true prefix lengths (empty ones and whole padded key blocks included),
    in the one-launch form where the shape allows it and in per-instruction passes."""
    B, Bp, Hq, Hkv, S, Pmax, d, lens, form = case
    pskv.pskv_set_multi_form(form)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(B + 3 * Bp + 5 * S + 7 * Pmax + sum(lens))
    draw = lambda *s: torch.randn(s, generator=gen, dtype=torch.float32).to(torch.bfloat16)
    q, pk, pv = draw(B, Hq, S, d), draw(Bp, Hkv, Pmax, d), draw(Bp, Hkv, Pmax, d)
    sk, sv, do = draw(B, Hkv, S, d), draw(B, Hkv, S, d), draw(B, Hq, S, d)
    for i, n in enumerate(lens):
        pk[i, :, : Pmax - n] = 3.0e4
        pv[i, :, : Pmax - n] = -3.0e4
    scale = 1 / math.sqrt(d)
    out, lse = pskv.pskv_attn_fwd_multi(q.cuda(), pk.cuda(), pv.cuda(), lens, sk.cuda(), sv.cuda(), scale)
    dq, dk, dv = pskv.pskv_attn_bwd_multi(do.cuda(), q.cuda(), pk.cuda(), pv.cuda(), lens, sk.cuda(), sv.cuda(),
                                          out, lse, scale)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    f = lambda x: x.to(torch.float64).numpy()
    mask = oracle.left_padding_mask(lens, Pmax)
    ro, rl = oracle.attn_fwd_multi(f(q), f(pk), f(pv), mask, f(sk), f(sv), scale)
    rq, rk, rv = oracle.attn_bwd_multi(f(do), f(q), f(pk), f(pv), mask, f(sk), f(sv), scale)
    parity.check_tensor("out", parity.to_f64(out), ro, strict_abs=False)
    parity.check_lse(parity.to_f64(lse), rl)
    parity.check_tensor("dq", parity.to_f64(dq), rq)
    parity.check_tensor("dk_suffix", parity.to_f64(dk), rk)
    parity.check_tensor("dv_suffix", parity.to_f64(dv), rv)
