"""Pins for the oracle's backward with a gradient on the log-sum-exp output
(L = sum(out * dout) + sum(lse * dlse)).  Central finite differences of the pinned forward, library
autograd through a library logsumexp, and the structural facts: with dlse = 0 it is the plain backward,
lse sends nothing to the values, and the lse term alone is linear in dlse."""
import numpy as np
import pytest
import torch

import oracle


def rnd(rng, *shape):
    return rng.standard_normal(shape)


def make(rng, B, Hq, Hkv, S, P, d):
    return dict(q=rnd(rng, B, Hq, S, d), pk=rnd(rng, Hkv, P, d), pv=rnd(rng, Hkv, P, d),
                sk=rnd(rng, B, Hkv, S, d), sv=rnd(rng, B, Hkv, S, d))


def bwd_lse(t, do, dl, scale):
    return oracle.attn_bwd_lse(do, dl, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale)


def loss(t, do, dl, scale):
    out, lse = oracle.attn_fwd(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale)
    return float(np.sum(out * do) + np.sum(lse * dl))


@pytest.mark.parametrize("shape", [(2, 4, 2, 3, 4, 4), (1, 2, 2, 4, 0, 4), (2, 3, 1, 2, 3, 4)])
def test_lse_gradient_matches_central_finite_differences(shape):
    rng = np.random.default_rng(41)
    t = make(rng, *shape)
    do = rnd(rng, *t["q"].shape)
    dl = rnd(rng, *t["q"].shape[:3])
    scale = 0.6
    dq, dk, dv = bwd_lse(t, do, dl, scale)
    eps = 1e-6
    for name, grad in (("q", dq), ("sk", dk), ("sv", dv)):
        fd = np.empty_like(grad)
        base = t[name]
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            tp = dict(t)
            x = base.copy(); x[idx] += eps; tp[name] = x
            up = loss(tp, do, dl, scale)
            x = base.copy(); x[idx] -= eps; tp[name] = x
            dn = loss(tp, do, dl, scale)
            fd[idx] = (up - dn) / (2 * eps)
        err = np.max(np.abs(fd - grad))
        assert err < 1e-7 * max(1.0, np.max(np.abs(grad))), (name, err)


def test_lse_gradient_matches_library_autograd():
    """Scores by a library matmul, lse by the library logsumexp over the visible keys, out by the library
    softmax: torch fp64 autograd of sum(out*dout) + sum(lse*dlse)."""
    rng = np.random.default_rng(42)
    B, Hq, Hkv, S, P, d = 3, 4, 2, 5, 6, 8
    n_rep = Hq // Hkv
    t = make(rng, B, Hq, Hkv, S, P, d)
    do, dl = rnd(rng, B, Hq, S, d), rnd(rng, B, Hq, S)
    scale = 0.45
    dq, dk, dv = bwd_lse(t, do, dl, scale)
    q = torch.from_numpy(t["q"]).requires_grad_(True)
    sk = torch.from_numpy(t["sk"]).requires_grad_(True)
    sv = torch.from_numpy(t["sv"]).requires_grad_(True)
    pk, pv = torch.from_numpy(t["pk"]), torch.from_numpy(t["pv"])
    kfull = torch.cat([pk.expand(B, Hkv, P, d), sk], dim=2).repeat_interleave(n_rep, dim=1)
    vfull = torch.cat([pv.expand(B, Hkv, P, d), sv], dim=2).repeat_interleave(n_rep, dim=1)
    s = scale * q @ kfull.transpose(-1, -2)                                   # [B,Hq,S,P+S]
    visible = torch.arange(P + S)[None, :] <= (torch.arange(S)[:, None] + P)
    s = s.masked_fill(~visible, float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    out = torch.softmax(s, dim=-1) @ vfull
    ((out * torch.from_numpy(do)).sum() + (lse * torch.from_numpy(dl)).sum()).backward()
    assert np.max(np.abs(dq - q.grad.numpy())) < 1e-12
    assert np.max(np.abs(dk - sk.grad.numpy())) < 1e-12
    assert np.max(np.abs(dv - sv.grad.numpy())) < 1e-12


def test_zero_lse_gradient_is_the_plain_backward_and_values_get_nothing_from_lse():
    rng = np.random.default_rng(43)
    t = make(rng, 2, 4, 2, 4, 5, 8)
    do, dl = rnd(rng, 2, 4, 4, 8), rnd(rng, 2, 4, 4)
    plain = oracle.attn_bwd(do, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], 0.5)
    zero = bwd_lse(t, do, np.zeros_like(dl), 0.5)
    for a, b in zip(plain, zero):
        assert np.array_equal(a, b)
    with_l = bwd_lse(t, do, dl, 0.5)
    assert np.array_equal(with_l[2], plain[2])          # dv_suffix: lse does not depend on V
    # the lse term is linear: gradients with (dout, 2 dlse) minus (dout, dlse) equal the lse-only part
    two = bwd_lse(t, do, 2 * dl, 0.5)
    only = bwd_lse(t, np.zeros_like(do), dl, 0.5)
    assert np.max(np.abs((two[0] - with_l[0]) - only[0])) < 1e-12
    assert np.max(np.abs((two[1] - with_l[1]) - only[1])) < 1e-12


def test_lse_only_gradient_of_a_query_is_the_expected_key():
    """d lse / d q = scale * sum_j p_j k_j: with one visible key it is scale * that key."""
    rng = np.random.default_rng(44)
    t = make(rng, 1, 1, 1, 1, 0, 8)
    dq, dk, dv = bwd_lse(t, np.zeros((1, 1, 1, 8)), np.ones((1, 1, 1)), 0.7)
    assert np.max(np.abs(dq[0, 0, 0] - 0.7 * t["sk"][0, 0, 0])) < 1e-14
    assert np.max(np.abs(dk[0, 0, 0] - 0.7 * t["q"][0, 0, 0])) < 1e-14
    assert not dv.any()
