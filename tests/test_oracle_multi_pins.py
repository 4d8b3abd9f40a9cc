"""Pins for the multi-instruction oracle (Sec. 4.3: one left-padded prefix cache per instruction,
reused by that instruction's candidates; padding excluded from attention).  None of them re-types the
oracle's own formula: they go through a library attention routine on the padded sequence with an
explicit attention mask, through library autograd, or through invariants."""
import math

import numpy as np
import pytest
import torch

import oracle


def rnd(rng, *shape):
    return rng.standard_normal(shape)


def make(rng, B, Bp, Hq, Hkv, S, Pmax, d, lens):
    return dict(q=rnd(rng, B, Hq, S, d), pk=rnd(rng, Bp, Hkv, Pmax, d), pv=rnd(rng, Bp, Hkv, Pmax, d),
                sk=rnd(rng, B, Hkv, S, d), sv=rnd(rng, B, Hkv, S, d),
                mask=oracle.left_padding_mask(lens, Pmax), lens=list(lens))


def fwd(t, scale):
    return oracle.attn_fwd_multi(t["q"], t["pk"], t["pv"], t["mask"], t["sk"], t["sv"], scale)


def library_padded_sequence(t, scale, grads=False, dout=None):
    """Every candidate's PADDED sequence [prefix (Pmax, with padding) ; suffix (S)] through torch's fp64
    scaled_dot_product_attention with an explicit boolean mask: causal, and padded prefix positions
    hidden as keys (the model's standard attention_mask)."""
    q, pk, pv, sk, sv, mask = (torch.from_numpy(np.asarray(t[k], dtype=np.float64)) for k in ("q", "pk", "pv", "sk", "sv", "mask"))
    B, Hq, S, d = q.shape
    Bp, Hkv, Pmax, _ = pk.shape
    Kq, n_rep = B // Bp, Hq // Hkv
    if grads:
        q.requires_grad_(True); sk.requires_grad_(True); sv.requires_grad_(True)
    inst = torch.arange(B) // Kq
    kfull = torch.cat([pk[inst], sk], dim=2).repeat_interleave(n_rep, dim=1)   # [B,Hq,Pmax+S,d]
    vfull = torch.cat([pv[inst], sv], dim=2).repeat_interleave(n_rep, dim=1)
    T = Pmax + S
    key_ok = torch.cat([mask[inst].bool(), torch.ones(B, S, dtype=torch.bool)], dim=1)  # [B,T]
    rows = torch.arange(S)[:, None] + Pmax
    causal = torch.arange(T)[None, :] <= rows                                           # [S,T]
    attn_mask = (causal[None, None] & key_ok[:, None, None, :])                         # [B,1,S,T]
    o = torch.nn.functional.scaled_dot_product_attention(q, kfull, vfull, attn_mask=attn_mask, scale=scale)
    if not grads:
        return o.numpy()
    (o * torch.from_numpy(dout)).sum().backward()
    return q.grad.numpy(), sk.grad.numpy(), sv.grad.numpy()


CASES = [
    # B, Bp, Hq, Hkv, S, Pmax, d, lens
    (6, 3, 4, 4, 5, 9, 8, (9, 4, 1)),
    (4, 2, 8, 2, 6, 7, 16, (7, 3)),      # GQA n_rep = 4
    (6, 3, 2, 1, 3, 5, 8, (0, 5, 2)),    # an instruction with an empty prefix
    (5, 1, 4, 2, 4, 6, 8, (6,)),         # one instruction, no padding: the single-prefix layout
]


@pytest.mark.parametrize("case", CASES)
def test_multi_equals_library_attention_with_padding_mask(case):
    rng = np.random.default_rng(21)
    t = make(rng, *case)
    scale = 1.0 / math.sqrt(case[6])
    out, lse = fwd(t, scale)
    ref = library_padded_sequence(t, scale)
    assert np.max(np.abs(out - ref)) < 1e-12
    # lse against a library logsumexp over the visible scores of a few rows
    B, Bp, Hq, Hkv, S, Pmax, d, lens = case
    Kq, n_rep = B // Bp, Hq // Hkv
    for (b, h, i) in [(0, 0, 0), (B - 1, Hq - 1, S - 1), (B // 2, Hq // 2, S // 2)]:
        inst, g = b // Kq, h // n_rep
        keys = np.concatenate([t["pk"][inst, g][t["mask"][inst] == 1], t["sk"][b, g, : i + 1]], axis=0)
        s = torch.from_numpy(scale * keys @ t["q"][b, h, i])
        assert abs(float(torch.logsumexp(s, dim=0)) - lse[b, h, i]) < 1e-12


def test_multi_reduces_to_single_prefix_calls_on_the_unpadded_caches():
    """Each instruction's candidates equal a single-prefix evaluation on that instruction's real tokens
    (the claim behind reusing one cache per instruction)."""
    rng = np.random.default_rng(22)
    B, Bp, Hq, Hkv, S, Pmax, d = 6, 3, 4, 2, 4, 8, 8
    lens = (8, 5, 2)
    t = make(rng, B, Bp, Hq, Hkv, S, Pmax, d, lens)
    out, lse = fwd(t, 0.3)
    Kq = B // Bp
    for i in range(Bp):
        sl = slice(i * Kq, (i + 1) * Kq)
        o1, l1 = oracle.attn_fwd(t["q"][sl], t["pk"][i][:, Pmax - lens[i]:], t["pv"][i][:, Pmax - lens[i]:],
                                 t["sk"][sl], t["sv"][sl], 0.3)
        assert np.max(np.abs(out[sl] - o1)) < 1e-12 and np.max(np.abs(lse[sl] - l1)) < 1e-12


def test_padding_contents_do_not_matter():
    rng = np.random.default_rng(23)
    case = (4, 2, 4, 4, 3, 6, 8, (2, 4))
    t = make(rng, *case)
    out, lse = fwd(t, 0.5)
    t2 = dict(t)
    t2["pk"] = t["pk"].copy(); t2["pv"] = t["pv"].copy()
    for i, n in enumerate(t["lens"]):
        t2["pk"][i, :, : 6 - n] = 1e6 * rnd(rng, 4, 6 - n, 8)
        t2["pv"][i, :, : 6 - n] = -1e6
    out2, lse2 = fwd(t2, 0.5)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_instruction_permutation_equivariance():
    rng = np.random.default_rng(24)
    B, Bp, Hq, Hkv, S, Pmax, d = 6, 3, 2, 2, 3, 5, 8
    t = make(rng, B, Bp, Hq, Hkv, S, Pmax, d, (5, 1, 3))
    out, lse = fwd(t, 0.4)
    perm = [2, 0, 1]
    Kq = B // Bp
    cand = np.concatenate([np.arange(p * Kq, (p + 1) * Kq) for p in perm])
    t2 = dict(q=t["q"][cand], sk=t["sk"][cand], sv=t["sv"][cand], pk=t["pk"][perm], pv=t["pv"][perm],
              mask=t["mask"][perm])
    out2, lse2 = fwd(t2, 0.4)
    assert np.array_equal(out2, out[cand]) and np.array_equal(lse2, lse[cand])


@pytest.mark.parametrize("case", CASES[:3])
def test_multi_backward_matches_library_autograd(case):
    rng = np.random.default_rng(25)
    t = make(rng, *case)
    B, Bp, Hq, Hkv, S, Pmax, d, lens = case
    do = rnd(rng, B, Hq, S, d)
    scale = 0.37
    dq, dk, dv = oracle.attn_bwd_multi(do, t["q"], t["pk"], t["pv"], t["mask"], t["sk"], t["sv"], scale)
    rq, rk, rv = library_padded_sequence(t, scale, grads=True, dout=do)
    assert np.max(np.abs(dq - rq)) < 1e-12
    assert np.max(np.abs(dk - rk)) < 1e-12
    assert np.max(np.abs(dv - rv)) < 1e-12


def test_multi_rejects_bad_arguments():
    rng = np.random.default_rng(26)
    t = make(rng, 4, 2, 2, 2, 3, 4, 8, (4, 2))
    with pytest.raises(ValueError):
        oracle.attn_fwd_multi(t["q"], t["pk"], t["pv"], t["mask"][:1], t["sk"], t["sv"], 0.5)
    with pytest.raises(RuntimeError):  # candidates not a multiple of instructions
        oracle.attn_fwd_multi(t["q"][:3], t["pk"], t["pv"], t["mask"], t["sk"][:3], t["sv"][:3], 0.5)
