"""Pins for the fp64 oracle: everything here compares it with something that is
not the oracle -- a library attention routine on the duplicated full sequence,
closed forms, invariances that follow from Eq. 2, and finite differences."""
import math

import numpy as np
import pytest
import torch

import oracle


def rnd(rng, *shape):
    return rng.standard_normal(shape)


def make(rng, B, Hq, Hkv, S, P, d):
    return dict(q=rnd(rng, B, Hq, S, d), pk=rnd(rng, Hkv, P, d), pv=rnd(rng, Hkv, P, d),
                sk=rnd(rng, B, Hkv, S, d), sv=rnd(rng, B, Hkv, S, d))


def fwd(t, scale):
    return oracle.attn_fwd(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale)


def bwd(t, do, scale):
    return oracle.attn_bwd(do, t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale)


def library_full_sequence(t, scale, rng):
    """No-cache evaluation: every candidate's full prefix+suffix sequence through
    torch's fp64 scaled_dot_product_attention with a causal mask; the prefix
    positions get arbitrary queries, and only the last S rows are kept."""
    B, Hq, S, d = t["q"].shape
    Hkv, P, _ = t["pk"].shape
    n_rep = Hq // Hkv
    kfull = np.concatenate([np.broadcast_to(t["pk"], (B, Hkv, P, d)), t["sk"]], axis=2)
    vfull = np.concatenate([np.broadcast_to(t["pv"], (B, Hkv, P, d)), t["sv"]], axis=2)
    kfull = np.repeat(kfull, n_rep, axis=1)
    vfull = np.repeat(vfull, n_rep, axis=1)
    qfull = np.concatenate([rnd(rng, B, Hq, P, d), t["q"]], axis=2)
    o = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(qfull), torch.from_numpy(kfull), torch.from_numpy(vfull),
        is_causal=True, scale=scale)
    return o[:, :, P:, :].numpy()


SHAPES = [
    # B, Hq, Hkv, S, P, d
    (3, 4, 4, 5, 7, 8),
    (2, 8, 2, 6, 9, 16),     # GQA n_rep=4
    (2, 7, 1, 3, 4, 8),      # GQA n_rep=7
    (1, 2, 2, 9, 0, 8),      # no prefix: plain causal attention
    (4, 4, 4, 1, 12, 8),     # single suffix token
    (8, 4, 4, 8, 32, 64),    # the tiny-correctness config's shape
]


@pytest.mark.parametrize("shape", SHAPES)
def test_equals_no_cache_full_sequence_library_attention(shape):
    rng = np.random.default_rng(1)
    t = make(rng, *shape)
    scale = 1.0 / math.sqrt(shape[-1])
    out, _ = fwd(t, scale)
    ref = library_full_sequence(t, scale, rng)
    assert np.max(np.abs(out - ref)) < 1e-12


@pytest.mark.parametrize("shape", SHAPES)
def test_lse_matches_library_logsumexp_on_visible_scores(shape):
    B, Hq, Hkv, S, P, d = shape
    rng = np.random.default_rng(2)
    t = make(rng, *shape)
    scale = 0.37
    _, lse = fwd(t, scale)
    n_rep = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            g = h // n_rep
            keys = np.concatenate([t["pk"][g], t["sk"][b, g]], axis=0)
            s = torch.from_numpy(scale * t["q"][b, h] @ keys.T)
            for i in range(S):
                ref = torch.logsumexp(s[i, : P + i + 1], dim=0).item()
                assert abs(lse[b, h, i] - ref) < 1e-12


def test_zero_queries_give_running_mean_and_log_count():
    rng = np.random.default_rng(3)
    B, Hq, Hkv, S, P, d = 2, 4, 2, 5, 6, 8
    t = make(rng, B, Hq, Hkv, S, P, d)
    t["q"][:] = 0.0
    out, lse = fwd(t, 0.5)
    for b in range(B):
        for h in range(Hq):
            g = h // 2
            vfull = np.concatenate([t["pv"][g], t["sv"][b, g]], axis=0)
            for i in range(S):
                n = P + i + 1
                assert np.allclose(out[b, h, i], vfull[:n].mean(axis=0), atol=1e-13)
                assert abs(lse[b, h, i] - math.log(n)) < 1e-13


def test_constant_values_give_constant_output():
    rng = np.random.default_rng(4)
    t = make(rng, 2, 4, 2, 5, 6, 8)
    t["pv"][:] = 1.0
    t["sv"][:] = 1.0
    out, _ = fwd(t, 0.3)
    assert np.max(np.abs(out - 1.0)) < 1e-13


def test_key_shift_leaves_out_and_shifts_lse():
    rng = np.random.default_rng(5)
    B, Hq, Hkv, S, P, d = 2, 4, 2, 5, 6, 8
    t = make(rng, B, Hq, Hkv, S, P, d)
    u = rnd(rng, d)
    scale = 0.41
    out0, lse0 = fwd(t, scale)
    t2 = dict(t, pk=t["pk"] + u, sk=t["sk"] + u)
    out1, lse1 = fwd(t2, scale)
    assert np.max(np.abs(out1 - out0)) < 1e-12
    shift = scale * np.einsum("bhsd,d->bhs", t["q"], u)
    assert np.max(np.abs(lse1 - lse0 - shift)) < 1e-12


def test_one_prefix_one_suffix_token_is_logistic():
    rng = np.random.default_rng(6)
    d = 8
    t = make(rng, 3, 2, 2, 1, 1, d)
    scale = 0.7
    out, lse = fwd(t, scale)
    for b in range(3):
        for h in range(2):
            s_p = scale * t["q"][b, h, 0] @ t["pk"][h, 0]
            s_s = scale * t["q"][b, h, 0] @ t["sk"][b, h, 0]
            delta = s_s - s_p
            sig = 1.0 / (1.0 + math.exp(-delta))
            ref = sig * t["sv"][b, h, 0] + (1.0 - sig) * t["pv"][h, 0]
            assert np.allclose(out[b, h, 0], ref, atol=1e-13)
            assert abs(lse[b, h, 0] - (s_p + math.log1p(math.exp(delta)))) < 1e-13


def test_hand_computed_two_key_case():
    # q=(1,0), prefix key (ln 3, 0) value (1,0); suffix key (0,5) value (0,1); scale 1:
    # scores ln3 and 0 -> weights 3/4 and 1/4, lse = ln 4.
    q = np.array([[[[1.0, 0.0]]]])
    pk = np.array([[[math.log(3.0), 0.0]]])
    pv = np.array([[[1.0, 0.0]]])
    sk = np.array([[[[0.0, 5.0]]]])
    sv = np.array([[[[0.0, 1.0]]]])
    out, lse = oracle.attn_fwd(q, pk, pv, sk, sv, 1.0)
    assert np.allclose(out[0, 0, 0], [0.75, 0.25], atol=1e-15)
    assert abs(lse[0, 0, 0] - math.log(4.0)) < 1e-15


def test_prefix_split_invariance():
    """Moving the last t prefix tokens into every candidate's suffix leaves the last S rows unchanged."""
    rng = np.random.default_rng(7)
    B, Hq, Hkv, S, P, d, tmove = 3, 4, 2, 4, 7, 8, 3
    t = make(rng, B, Hq, Hkv, S, P, d)
    scale = 0.33
    out0, lse0 = fwd(t, scale)
    tail_k = np.broadcast_to(t["pk"][:, P - tmove:], (B, Hkv, tmove, d))
    tail_v = np.broadcast_to(t["pv"][:, P - tmove:], (B, Hkv, tmove, d))
    t2 = dict(q=np.concatenate([rnd(rng, B, Hq, tmove, d), t["q"]], axis=2),
              pk=t["pk"][:, : P - tmove], pv=t["pv"][:, : P - tmove],
              sk=np.concatenate([tail_k, t["sk"]], axis=2),
              sv=np.concatenate([tail_v, t["sv"]], axis=2))
    out1, lse1 = fwd(t2, scale)
    assert np.max(np.abs(out1[:, :, tmove:] - out0)) < 1e-12
    assert np.max(np.abs(lse1[:, :, tmove:] - lse0)) < 1e-12


def test_candidate_permutation_equivariance():
    rng = np.random.default_rng(8)
    t = make(rng, 5, 4, 2, 4, 6, 8)
    perm = np.array([3, 0, 4, 1, 2])
    out0, lse0 = fwd(t, 0.3)
    t2 = dict(t, q=t["q"][perm], sk=t["sk"][perm], sv=t["sv"][perm])
    out1, lse1 = fwd(t2, 0.3)
    assert np.array_equal(out1, out0[perm])
    assert np.array_equal(lse1, lse0[perm])
    do = rnd(rng, *t["q"].shape)
    g0 = bwd(t, do, 0.3)
    g1 = bwd(t2, do[perm], 0.3)
    for a, b_ in zip(g0, g1):
        assert np.array_equal(b_, a[perm])


def test_gqa_equals_mha_with_repeated_kv_heads():
    rng = np.random.default_rng(9)
    B, Hq, Hkv, S, P, d = 2, 6, 2, 4, 5, 8
    t = make(rng, B, Hq, Hkv, S, P, d)
    n_rep = Hq // Hkv
    t2 = dict(q=t["q"], pk=np.repeat(t["pk"], n_rep, axis=0), pv=np.repeat(t["pv"], n_rep, axis=0),
              sk=np.repeat(t["sk"], n_rep, axis=1), sv=np.repeat(t["sv"], n_rep, axis=1))
    out0, lse0 = fwd(t, 0.35)
    out1, lse1 = fwd(t2, 0.35)
    assert np.max(np.abs(out0 - out1)) < 1e-13 and np.max(np.abs(lse0 - lse1)) < 1e-13
    do = rnd(rng, B, Hq, S, d)
    dq0, dk0, dv0 = bwd(t, do, 0.35)
    dq1, dk1, dv1 = bwd(t2, do, 0.35)
    assert np.max(np.abs(dq0 - dq1)) < 1e-13
    # a shared KV head receives the sum of its query heads' gradients
    assert np.max(np.abs(dk0 - dk1.reshape(B, Hkv, n_rep, S, d).sum(axis=2))) < 1e-13
    assert np.max(np.abs(dv0 - dv1.reshape(B, Hkv, n_rep, S, d).sum(axis=2))) < 1e-13


def test_lse_merge_identity():
    """Attention over the prefix alone and over the causal suffix alone, merged by
    lse = logaddexp(lse_p, lse_s), out = O_p e^{lse_p-lse} + O_s e^{lse_s-lse}, equals the joint result."""
    rng = np.random.default_rng(10)
    B, Hq, Hkv, S, P, d = 2, 4, 2, 5, 6, 8
    t = make(rng, B, Hq, Hkv, S, P, d)
    scale = 0.3
    out, lse = fwd(t, scale)
    empty = np.zeros((Hkv, 0, d))
    o_s, lse_s = oracle.attn_fwd(t["q"], empty, empty, t["sk"], t["sv"], scale)
    # prefix-only part: every row sees all P keys; taken from the library softmax
    o_p = np.empty_like(out)
    lse_p = np.empty_like(lse)
    for i in range(S):
        for b in range(B):
            for h in range(Hq):
                g = h // (Hq // Hkv)
                s = torch.from_numpy(scale * t["pk"][g] @ t["q"][b, h, i])
                lse_p[b, h, i] = torch.logsumexp(s, 0).item()
                o_p[b, h, i] = (torch.softmax(s, 0).numpy()[:, None] * t["pv"][g]).sum(axis=0)
    merged_lse = np.logaddexp(lse_p, lse_s)
    merged = o_p * np.exp(lse_p - merged_lse)[..., None] + o_s * np.exp(lse_s - merged_lse)[..., None]
    assert np.max(np.abs(merged - out)) < 1e-12
    assert np.max(np.abs(merged_lse - lse)) < 1e-12


def _loss(t, do, scale):
    out, _ = fwd(t, scale)
    return float(np.sum(out * do))


@pytest.mark.parametrize("shape", [(2, 4, 2, 3, 4, 4), (1, 2, 2, 4, 0, 4), (2, 3, 1, 2, 3, 4)])
def test_backward_matches_central_finite_differences(shape):
    rng = np.random.default_rng(11)
    t = make(rng, *shape)
    do = rnd(rng, *t["q"].shape)
    scale = 0.6
    dq, dk, dv = bwd(t, do, scale)
    eps = 1e-6
    for name, grad in (("q", dq), ("sk", dk), ("sv", dv)):
        fd = np.empty_like(grad)
        base = t[name]
        it = np.nditer(base, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            tp = dict(t)
            x = base.copy(); x[idx] += eps; tp[name] = x
            up = _loss(tp, do, scale)
            x = base.copy(); x[idx] -= eps; tp[name] = x
            dn = _loss(tp, do, scale)
            fd[idx] = (up - dn) / (2 * eps)
        err = np.max(np.abs(fd - grad))
        assert err < 1e-7 * max(1.0, np.max(np.abs(grad))), (name, err)


def test_backward_matches_library_autograd_on_full_sequence():
    """Gradients equal the suffix rows/keys of the no-cache full-sequence backward (torch fp64 autograd
    through the library attention), with the prefix keys' gradients discarded."""
    rng = np.random.default_rng(12)
    B, Hq, Hkv, S, P, d = 3, 4, 2, 5, 6, 8
    n_rep = Hq // Hkv
    t = make(rng, B, Hq, Hkv, S, P, d)
    do = rnd(rng, B, Hq, S, d)
    scale = 0.45
    dq, dk, dv = bwd(t, do, scale)
    q = torch.from_numpy(t["q"]).requires_grad_(True)
    sk = torch.from_numpy(t["sk"]).requires_grad_(True)
    sv = torch.from_numpy(t["sv"]).requires_grad_(True)
    pk = torch.from_numpy(t["pk"]); pv = torch.from_numpy(t["pv"])
    kfull = torch.cat([pk.expand(B, Hkv, P, d), sk], dim=2).repeat_interleave(n_rep, dim=1)
    vfull = torch.cat([pv.expand(B, Hkv, P, d), sv], dim=2).repeat_interleave(n_rep, dim=1)
    qfull = torch.cat([torch.zeros(B, Hq, P, d, dtype=torch.float64), q], dim=2)
    o = torch.nn.functional.scaled_dot_product_attention(qfull, kfull, vfull, is_causal=True, scale=scale)
    (o[:, :, P:] * torch.from_numpy(do)).sum().backward()
    assert np.max(np.abs(dq - q.grad.numpy())) < 1e-12
    assert np.max(np.abs(dk - sk.grad.numpy())) < 1e-12
    assert np.max(np.abs(dv - sv.grad.numpy())) < 1e-12


def test_backward_structure():
    rng = np.random.default_rng(13)
    t = make(rng, 2, 4, 2, 4, 5, 8)
    do = rnd(rng, *t["q"].shape)
    g1 = bwd(t, do, 0.3)
    for g in bwd(t, np.zeros_like(do), 0.3):
        assert np.all(g == 0.0)
    g2 = bwd(t, 2.5 * do, 0.3)
    for a, b_ in zip(g1, g2):
        assert np.max(np.abs(2.5 * a - b_)) < 1e-12
    # a constant added to every value row moves out by the same constant but changes no dq/dk
    t2 = dict(t, pv=t["pv"] + 3.0, sv=t["sv"] + 3.0)
    g3 = bwd(t2, do, 0.3)
    assert np.max(np.abs(g3[0] - g1[0])) < 1e-11
    assert np.max(np.abs(g3[1] - g1[1])) < 1e-11
    # sum_j ds_j = 0 per row, so adding one vector u to every key leaves dq unchanged
    u = rnd(rng, 8)
    t3 = dict(t, pk=t["pk"] + u, sk=t["sk"] + u)
    g4 = bwd(t3, do, 0.3)
    assert np.max(np.abs(g4[0] - g1[0])) < 1e-11


def test_bad_arguments_are_rejected():
    rng = np.random.default_rng(14)
    t = make(rng, 1, 3, 2, 2, 2, 4)  # Hq not a multiple of Hkv
    with pytest.raises(RuntimeError):
        fwd(t, 1.0)
