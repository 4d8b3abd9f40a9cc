"""Pins for the oracle's gradients of the shared prefix cache (summed over all candidates): library
autograd through the library attention on the full sequences with ONE shared prefix leaf, central finite
differences of the pinned forward, and the sum-over-candidates structure."""
import numpy as np
import pytest
import torch

import oracle


def rnd(rng, *shape):
    return rng.standard_normal(shape)


def make(rng, B, Hq, Hkv, S, P, d):
    return dict(q=rnd(rng, B, Hq, S, d), pk=rnd(rng, Hkv, P, d), pv=rnd(rng, Hkv, P, d),
                sk=rnd(rng, B, Hkv, S, d), sv=rnd(rng, B, Hkv, S, d))


def prefix_grads(t, do, scale, dl=None):
    return oracle.attn_bwd_prefix(do, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale, dl)


@pytest.mark.parametrize("shape", [(3, 4, 2, 5, 6, 8), (2, 6, 2, 3, 4, 4), (4, 2, 2, 1, 3, 8)])
def test_prefix_gradients_match_library_autograd_with_a_shared_prefix_leaf(shape):
    rng = np.random.default_rng(61)
    B, Hq, Hkv, S, P, d = shape
    n_rep = Hq // Hkv
    t = make(rng, *shape)
    do = rnd(rng, B, Hq, S, d)
    scale = 0.45
    dk, dv = prefix_grads(t, do, scale)
    pk = torch.from_numpy(t["pk"]).requires_grad_(True)
    pv = torch.from_numpy(t["pv"]).requires_grad_(True)
    q, sk, sv = (torch.from_numpy(t[k]) for k in ("q", "sk", "sv"))
    kfull = torch.cat([pk.expand(B, Hkv, P, d), sk], dim=2).repeat_interleave(n_rep, dim=1)
    vfull = torch.cat([pv.expand(B, Hkv, P, d), sv], dim=2).repeat_interleave(n_rep, dim=1)
    qfull = torch.cat([torch.zeros(B, Hq, P, d, dtype=torch.float64), q], dim=2)
    o = torch.nn.functional.scaled_dot_product_attention(qfull, kfull, vfull, is_causal=True, scale=scale)
    (o[:, :, P:] * torch.from_numpy(do)).sum().backward()
    assert np.max(np.abs(dk - pk.grad.numpy())) < 1e-11
    assert np.max(np.abs(dv - pv.grad.numpy())) < 1e-11


def test_prefix_gradients_match_central_finite_differences_with_an_lse_gradient():
    rng = np.random.default_rng(62)
    shape = (2, 4, 2, 3, 3, 4)
    t = make(rng, *shape)
    do, dl = rnd(rng, 2, 4, 3, 4), rnd(rng, 2, 4, 3)
    scale = 0.6
    dk, dv = prefix_grads(t, do, scale, dl)

    def loss(tt):
        out, lse = oracle.attn_fwd(tt["q"], tt["pk"], tt["pv"], tt["sk"], tt["sv"], scale)
        return float(np.sum(out * do) + np.sum(lse * dl))

    eps = 1e-6
    for name, grad in (("pk", dk), ("pv", dv)):
        fd = np.empty_like(grad)
        it = np.nditer(t[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            tp = dict(t)
            x = t[name].copy(); x[idx] += eps; tp[name] = x
            up = loss(tp)
            x = t[name].copy(); x[idx] -= eps; tp[name] = x
            fd[idx] = (up - loss(tp)) / (2 * eps)
        assert np.max(np.abs(fd - grad)) < 1e-7 * max(1.0, np.max(np.abs(grad))), name


def test_prefix_gradients_are_the_sum_over_candidates_evaluated_alone():
    rng = np.random.default_rng(63)
    B, Hq, Hkv, S, P, d = 4, 4, 2, 3, 5, 8
    t = make(rng, B, Hq, Hkv, S, P, d)
    do = rnd(rng, B, Hq, S, d)
    dk, dv = prefix_grads(t, do, 0.5)
    sk_ = np.zeros_like(dk); sv_ = np.zeros_like(dv)
    for b in range(B):
        one = dict(q=t["q"][b:b + 1], pk=t["pk"], pv=t["pv"], sk=t["sk"][b:b + 1], sv=t["sv"][b:b + 1])
        a, c = prefix_grads(one, do[b:b + 1], 0.5)
        sk_ += a; sv_ += c
    assert np.max(np.abs(dk - sk_)) < 1e-12 and np.max(np.abs(dv - sv_)) < 1e-12
    # no prefix, no gradient: shapes with P = 0 return empty arrays
    e = make(rng, 2, 2, 2, 3, 0, 4)
    a, c = prefix_grads(e, rnd(rng, 2, 2, 3, 4), 0.5)
    assert a.shape == (2, 0, 4) and c.shape == (2, 0, 4)


def test_dv_prefix_sums_to_the_prefix_probability_mass_times_dout():
    """With dout = 1 everywhere, sum_j dv_prefix[g, j, c] = sum over rows of head group g of the probability
    mass the row puts on the prefix (the same for every column c)."""
    rng = np.random.default_rng(64)
    B, Hq, Hkv, S, P, d = 3, 2, 1, 2, 4, 4
    t = make(rng, B, Hq, Hkv, S, P, d)
    _, dv = prefix_grads(t, np.ones((B, Hq, S, d)), 0.7)
    _, lse = oracle.attn_fwd(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.7)
    mass = 0.0
    for b in range(B):
        for h in range(Hq):
            for i in range(S):
                s = 0.7 * t["pk"][0] @ t["q"][b, h, i]
                mass += float(np.sum(np.exp(s - lse[b, h, i])))
    assert np.max(np.abs(dv.sum(axis=1)[0] - mass)) < 1e-12
