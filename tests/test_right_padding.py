"""Ragged candidate lengths in the full-suffix operator need no mask: suffixes are left-aligned and
right-padded (Sec. 4.3, suffix-centric alignment), padded positions come after every real token, and
the causal rule of Eq. 2 hides them from the real rows.  Real rows therefore equal the candidate
evaluated alone at its true length; pad rows hold finite values the loss mask ignores, and with a zero
upstream gradient on them they add nothing to any gradient.  Checked on the oracle (CPU) and through
the C ABI (GPU)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity


def _batch(seed, B, Hq, Hkv, S, P, d, lens):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    draw = lambda *s: torch.randn(s, generator=gen, dtype=torch.float32).to(torch.bfloat16)
    t = dict(q=draw(B, Hq, S, d), prefix_k=draw(Hkv, P, d), prefix_v=draw(Hkv, P, d), suffix_k=draw(B, Hkv, S, d),
             suffix_v=draw(B, Hkv, S, d), dout=draw(B, Hq, S, d))
    for b, n in enumerate(lens):          # pad positions: arbitrary finite contents, zero upstream gradient
        t["suffix_k"][b, :, n:] = 7.0
        t["suffix_v"][b, :, n:] = -5.0
        t["q"][b, :, n:] = 3.0
        t["dout"][b, :, n:] = 0.0
    return t


def test_oracle_right_padded_batch_equals_candidates_at_their_true_lengths():
    B, Hq, Hkv, S, P, d = 3, 4, 2, 6, 5, 8
    lens = (6, 2, 4)
    t = {k: parity.to_f64(v) for k, v in _batch(1, B, Hq, Hkv, S, P, d, lens).items()}
    out, lse = oracle.attn_fwd(t["q"], t["prefix_k"], t["prefix_v"], t["suffix_k"], t["suffix_v"], 0.4)
    dq, dk, dv = oracle.attn_bwd(t["dout"], t["q"], t["prefix_k"], t["prefix_v"], t["suffix_k"], t["suffix_v"], 0.4)
    for b, n in enumerate(lens):
        one = {k: (v if k.startswith("prefix") else v[b:b + 1, :, :n]) for k, v in t.items()}
        o1, l1 = oracle.attn_fwd(one["q"], one["prefix_k"], one["prefix_v"], one["suffix_k"], one["suffix_v"], 0.4)
        q1, k1, v1 = oracle.attn_bwd(one["dout"], one["q"], one["prefix_k"], one["prefix_v"], one["suffix_k"],
                                     one["suffix_v"], 0.4)
        assert np.array_equal(out[b:b + 1, :, :n], o1) and np.array_equal(lse[b:b + 1, :, :n], l1)
        assert np.max(np.abs(dq[b:b + 1, :, :n] - q1)) < 1e-13
        assert np.max(np.abs(dk[b:b + 1, :, :n] - k1)) < 1e-13 and np.max(np.abs(dv[b:b + 1, :, :n] - v1)) < 1e-13
        assert not dq[b, :, n:].any() and not dk[b, :, n:].any() and not dv[b, :, n:].any()


@pytest.mark.gpu
def test_right_padded_batch_on_the_gpu_matches_candidates_at_their_true_lengths():
    B, Hq, Hkv, S, P, d = 6, 8, 2, 48, 200, 128
    lens = (48, 20, 33, 1, 40, 27)
    t = _batch(2, B, Hq, Hkv, S, P, d, lens)
    dev = {k: v.cuda() for k, v in t.items()}
    scale = d ** -0.5
    out, lse = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"], scale)
    dq, dk, dv = pskv.pskv_attn_bwd(dev["dout"], dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"],
                                    dev["suffix_v"], out, lse, scale)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    f = {k: parity.to_f64(v) for k, v in t.items()}
    for b, n in enumerate(lens):
        one = {k: (v if k.startswith("prefix") else v[b:b + 1, :, :n]) for k, v in f.items()}
        ro, rl = oracle.attn_fwd(one["q"], one["prefix_k"], one["prefix_v"], one["suffix_k"], one["suffix_v"], scale)
        rq, rk, rv = oracle.attn_bwd(one["dout"], one["q"], one["prefix_k"], one["prefix_v"], one["suffix_k"],
                                     one["suffix_v"], scale)
        parity.check_tensor("out", parity.to_f64(out[b:b + 1, :, :n]), ro)
        parity.check_lse(parity.to_f64(lse[b:b + 1, :, :n]), rl)
        parity.check_tensor("dq", parity.to_f64(dq[b:b + 1, :, :n]), rq)
        parity.check_tensor("dk", parity.to_f64(dk[b:b + 1, :, :n]), rk)
        parity.check_tensor("dv", parity.to_f64(dv[b:b + 1, :, :n]), rv)
        assert torch.isfinite(out[b].float()).all()                       # pad rows: finite, to be ignored
        assert not dq[b, :, n:].any() and not dk[b, :, n:].any() and not dv[b, :, n:].any()
