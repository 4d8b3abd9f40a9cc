"""Pins for the decode-shaped oracle (token-by-token suffix growth: only the last Sq of a candidate's
suffix_len[b] cached suffix tokens are queries; Eq. 2's causal mask, shifted).  None re-types the oracle's
formula: they go through a library attention routine with an explicit mask on the whole buffer, library
autograd, the already pinned full-suffix oracle (a decode step is the tail of a full evaluation), or
invariants (what lies past suffix_len is ignored; ragged batches are independent candidates)."""
import math

import numpy as np
import pytest
import torch

import oracle


def rnd(rng, *shape):
    return rng.standard_normal(shape)


def make(rng, B, Hq, Hkv, Sq, Skv, P, d, lens):
    return dict(q=rnd(rng, B, Hq, Sq, d), pk=rnd(rng, Hkv, P, d), pv=rnd(rng, Hkv, P, d),
                sk=rnd(rng, B, Hkv, Skv, d), sv=rnd(rng, B, Hkv, Skv, d),
                lens=None if lens is None else np.asarray(lens, dtype=np.int32))


def fwd(t, scale):
    return oracle.attn_fwd_decode(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale, t["lens"])


def library_masked(t, scale, grads=False, dout=None):
    """torch's fp64 scaled_dot_product_attention over [prefix ; whole suffix buffer] with an explicit
    boolean mask: suffix key j is visible to query i of candidate b iff j <= len_b - Sq + i."""
    q, pk, pv, sk, sv = (torch.from_numpy(np.asarray(t[k], dtype=np.float64)) for k in ("q", "pk", "pv", "sk", "sv"))
    B, Hq, Sq, d = q.shape
    Hkv, P, _ = pk.shape
    Skv = sk.shape[2]
    n_rep = Hq // Hkv
    lens = torch.full((B,), Skv, dtype=torch.long) if t["lens"] is None else torch.from_numpy(t["lens"]).long()
    if grads:
        q.requires_grad_(True); sk.requires_grad_(True); sv.requires_grad_(True)
    kfull = torch.cat([pk[None].expand(B, -1, -1, -1), sk], dim=2).repeat_interleave(n_rep, dim=1)
    vfull = torch.cat([pv[None].expand(B, -1, -1, -1), sv], dim=2).repeat_interleave(n_rep, dim=1)
    j = torch.arange(Skv)[None, None, :]
    pos = (lens[:, None] - Sq + torch.arange(Sq)[None, :])[:, :, None]        # [B,Sq,1]
    sfx_ok = j <= pos                                                          # [B,Sq,Skv]
    mask = torch.cat([torch.ones(B, Sq, P, dtype=torch.bool), sfx_ok], dim=2)[:, None]  # [B,1,Sq,P+Skv]
    o = torch.nn.functional.scaled_dot_product_attention(q, kfull, vfull, attn_mask=mask, scale=scale)
    if not grads:
        return o.numpy()
    (o * torch.from_numpy(dout)).sum().backward()
    return q.grad.numpy(), sk.grad.numpy(), sv.grad.numpy()


CASES = [
    # B, Hq, Hkv, Sq, Skv, P, d, lens
    (3, 4, 4, 1, 6, 5, 8, None),            # one new token per candidate
    (4, 8, 2, 2, 7, 9, 16, (7, 2, 5, 3)),   # GQA, ragged
    (3, 2, 1, 3, 5, 0, 8, (3, 5, 4)),       # no prefix at all
    (2, 4, 2, 4, 4, 6, 8, None),            # Sq == Skv: the full-suffix operator
]


@pytest.mark.parametrize("case", CASES)
def test_decode_equals_library_attention_with_shifted_causal_mask(case):
    rng = np.random.default_rng(31)
    t = make(rng, *case)
    scale = 1.0 / math.sqrt(case[6])
    out, lse = fwd(t, scale)
    assert np.max(np.abs(out - library_masked(t, scale))) < 1e-12
    B, Hq, Hkv, Sq, Skv, P, d, lens = case
    n_rep = Hq // Hkv
    for (b, h, i) in [(0, 0, 0), (B - 1, Hq - 1, Sq - 1), (B // 2, Hq // 2, Sq // 2)]:
        L = Skv if lens is None else lens[b]
        keys = np.concatenate([t["pk"][h // n_rep], t["sk"][b, h // n_rep, : L - Sq + i + 1]], axis=0)
        s = torch.from_numpy(scale * keys @ t["q"][b, h, i])
        assert abs(float(torch.logsumexp(s, dim=0)) - lse[b, h, i]) < 1e-12


def test_decode_with_all_tokens_as_queries_is_the_full_suffix_operator():
    rng = np.random.default_rng(32)
    t = make(rng, 3, 4, 2, 5, 5, 7, 8, None)
    out, lse = fwd(t, 0.3)
    o1, l1 = oracle.attn_fwd(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.3)
    assert np.array_equal(out, o1) and np.array_equal(lse, l1)


@pytest.mark.parametrize("Sq,L", [(1, 6), (2, 6), (3, 4)])
def test_decode_step_is_the_tail_of_a_full_suffix_evaluation(Sq, L):
    """Growing the suffix token by token must give, for the new tokens, exactly the rows a full
    evaluation of the L-token suffix gives for its last Sq positions (the point of caching)."""
    rng = np.random.default_rng(33)
    B, Hq, Hkv, P, d, Skv = 3, 4, 2, 5, 8, 8
    q_full = rnd(rng, B, Hq, L, d)
    t = make(rng, B, Hq, Hkv, Sq, Skv, P, d, [L] * B)
    t["q"] = q_full[:, :, L - Sq:]
    out, lse = fwd(t, 0.41)
    o1, l1 = oracle.attn_fwd(q_full, t["pk"], t["pv"], t["sk"][:, :, :L], t["sv"][:, :, :L], 0.41)
    assert np.max(np.abs(out - o1[:, :, L - Sq:])) < 1e-13
    assert np.max(np.abs(lse - l1[:, :, L - Sq:])) < 1e-13
    # and the gradients equal those of the full evaluation with zero upstream gradient on the old rows
    do = rnd(rng, B, Hq, Sq, d)
    do_full = np.zeros((B, Hq, L, d)); do_full[:, :, L - Sq:] = do
    dq, dk, dv = oracle.attn_bwd_decode(do, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.41, t["lens"])
    fq, fk, fv = oracle.attn_bwd(do_full, q_full, t["pk"], t["pv"], t["sk"][:, :, :L], t["sv"][:, :, :L], 0.41)
    assert np.max(np.abs(dq - fq[:, :, L - Sq:])) < 1e-13
    assert np.max(np.abs(dk[:, :, :L] - fk)) < 1e-13 and np.max(np.abs(dv[:, :, :L] - fv)) < 1e-13
    assert not dk[:, :, L:].any() and not dv[:, :, L:].any()


def test_rows_past_suffix_len_are_never_read():
    rng = np.random.default_rng(34)
    case = (4, 4, 2, 2, 6, 5, 8, (2, 6, 4, 3))
    t = make(rng, *case)
    out, lse = fwd(t, 0.5)
    t2 = dict(t)
    t2["sk"] = t["sk"].copy(); t2["sv"] = t["sv"].copy()
    for b, n in enumerate(case[7]):
        t2["sk"][b, :, n:] = np.nan
        t2["sv"][b, :, n:] = np.inf
    out2, lse2 = fwd(t2, 0.5)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)
    do = rnd(rng, 4, 4, 2, 8)
    g1 = oracle.attn_bwd_decode(do, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5, t["lens"])
    g2 = oracle.attn_bwd_decode(do, t2["q"], t2["pk"], t2["pv"], t2["sk"], t2["sv"], 0.5, t2["lens"])
    for a, b_ in zip(g1, g2):
        assert np.array_equal(a, b_)


def test_ragged_batch_equals_candidates_evaluated_alone():
    rng = np.random.default_rng(35)
    case = (3, 4, 2, 2, 7, 4, 8, (7, 2, 5))
    t = make(rng, *case)
    out, lse = fwd(t, 0.7)
    for b, n in enumerate(case[7]):
        o1, l1 = oracle.attn_fwd_decode(t["q"][b:b + 1], t["pk"], t["pv"], t["sk"][b:b + 1, :, :n],
                                        t["sv"][b:b + 1, :, :n], 0.7)
        assert np.array_equal(out[b:b + 1], o1) and np.array_equal(lse[b:b + 1], l1)


@pytest.mark.parametrize("case", CASES[:3])
def test_decode_backward_matches_library_autograd(case):
    rng = np.random.default_rng(36)
    t = make(rng, *case)
    B, Hq, Hkv, Sq, Skv, P, d, lens = case
    do = rnd(rng, B, Hq, Sq, d)
    scale = 0.37
    dq, dk, dv = oracle.attn_bwd_decode(do, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale, t["lens"])
    rq, rk, rv = library_masked(t, scale, grads=True, dout=do)
    assert np.max(np.abs(dq - rq)) < 1e-12
    assert np.max(np.abs(dk - rk)) < 1e-12
    assert np.max(np.abs(dv - rv)) < 1e-12


def test_decode_rejects_bad_arguments():
    rng = np.random.default_rng(37)
    t = make(rng, 2, 2, 2, 2, 4, 3, 8, (4, 3))
    with pytest.raises(RuntimeError):   # fewer cached tokens than queries
        oracle.attn_fwd_decode(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5, [1, 4])
    with pytest.raises(RuntimeError):   # more cached tokens than the buffer holds
        oracle.attn_fwd_decode(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5, [5, 4])
    with pytest.raises(ValueError):
        oracle.attn_fwd_decode(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5, [4])
    with pytest.raises(RuntimeError):   # Sq > Skv
        oracle.attn_fwd_decode(rnd(rng, 2, 2, 5, 8), t["pk"], t["pv"], t["sk"], t["sv"], 0.5)
