"""Decode-shaped variant: only the last Sq of each candidate's suffix_len[b] cached suffix tokens are
queries (token-by-token suffix growth).  GPU parity against the fp64 oracle on seeded inputs whose
unused cache rows hold large finite garbage, plus host-side argument checks."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity

SEED = 260313420 + 99


def make(B, Hq, Hkv, Sq, Skv, P, d, ragged, seed=SEED):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + B + 7 * Sq + 13 * Skv + P)

    def draw(*shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16)

    t = dict(q=draw(B, Hq, Sq, d), prefix_k=draw(Hkv, P, d), prefix_v=draw(Hkv, P, d),
             suffix_k=draw(B, Hkv, Skv, d), suffix_v=draw(B, Hkv, Skv, d), dout=draw(B, Hq, Sq, d))
    lens = None
    if ragged:
        lens = torch.randint(Sq, Skv + 1, (B,), generator=gen, dtype=torch.int32)
        lens[0] = Sq           # the shortest legal cache: the queries are all there is
        lens[B - 1] = Skv      # and a full one
        for b in range(B):     # rows past the cached tokens must not matter
            t["suffix_k"][b, :, int(lens[b]):] = 3.0e4
            t["suffix_v"][b, :, int(lens[b]):] = -3.0e4
    return t, lens


CASES = [
    # B, Hq, Hkv, Sq, Skv, P, d, ragged
    (64, 32, 8, 1, 48, 256, 128, False),    # one new token per candidate, the GQA layer shape
    (130, 32, 8, 1, 48, 256, 128, True),    # ragged lengths; candidate count leaves a partial last tile
    (32, 8, 2, 8, 40, 300, 128, True),      # a few new tokens, prefix with a ragged last block
    (16, 4, 4, 4, 20, 160, 128, True),      # MHA
    (12, 4, 2, 3, 7, 33, 64, True),         # head dim 64, odd sizes
    (6, 4, 2, 2, 150, 64, 128, True),       # suffix cache longer than one key block
    (9, 8, 2, 2, 24, 0, 128, True),         # no prefix
    (20, 16, 4, 16, 64, 700, 128, False),   # prefix streamed in several blocks
    (4, 8, 2, 16, 300, 64, 128, True),      # long suffix cache: several 128-key blocks per candidate
    (6, 32, 8, 48, 64, 256, 128, True),     # more than 128 query rows per candidate and KV head
    (3, 8, 8, 24, 200, 0, 64, True),        # head dim 64, long cache, no prefix
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
def test_decode_forward_and_backward_match_the_oracle(case):
    B, Hq, Hkv, Sq, Skv, P, d, ragged = case
    t, lens = make(*case)
    scale = 1.0 / np.sqrt(d)
    dev = {k: v.cuda() for k, v in t.items()}
    dlens = None if lens is None else lens.cuda()
    pk = dev["prefix_k"] if P > 0 else None
    pv = dev["prefix_v"] if P > 0 else None
    out = parity.Guarded((B, Hq, Sq, d), torch.bfloat16, "cuda")
    lse = parity.Guarded((B, Hq, Sq), torch.float32, "cuda")
    pskv.pskv_attn_fwd_decode(dev["q"], pk, pv, dev["suffix_k"], dev["suffix_v"], dlens, scale,
                              out=out.view, lse=lse.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    out.check("out"); lse.check("lse")
    f = {k: parity.to_f64(v) for k, v in t.items()}
    nl = None if lens is None else lens.numpy()
    ref_out, ref_lse = oracle.attn_fwd_decode(f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"],
                                              scale, nl)
    parity.check_tensor("out", parity.to_f64(out.view), ref_out, strict_abs=(P + 1 >= 128))
    parity.check_lse(parity.to_f64(lse.view), ref_lse)

    dq = parity.Guarded((B, Hq, Sq, d), torch.bfloat16, "cuda")
    dk = parity.Guarded((B, Hkv, Skv, d), torch.bfloat16, "cuda")
    dv = parity.Guarded((B, Hkv, Skv, d), torch.bfloat16, "cuda")
    pskv.pskv_attn_bwd_decode(dev["dout"], dev["q"], pk, pv, dev["suffix_k"], dev["suffix_v"], dlens, out.view,
                              lse.view, scale, dq=dq.view, dk_suffix=dk.view, dv_suffix=dv.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dq.check("dq"); dk.check("dk_suffix"); dv.check("dv_suffix")
    rq, rk, rv = oracle.attn_bwd_decode(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"],
                                        f["suffix_v"], scale, nl)
    parity.check_tensor("dq", parity.to_f64(dq.view), rq)
    parity.check_tensor("dk_suffix", parity.to_f64(dk.view), rk)
    parity.check_tensor("dv_suffix", parity.to_f64(dv.view), rv)
    if lens is not None:   # gradients of rows that are not cached tokens are exactly zero
        for b in range(B):
            assert not dk.view[b, :, int(lens[b]):].any() and not dv.view[b, :, int(lens[b]):].any()


@pytest.mark.gpu
def test_all_tokens_as_queries_equals_the_full_suffix_call_bit_for_bit():
    B, Hq, Hkv, S, P, d = 16, 8, 2, 16, 200, 128
    t, _ = make(B, Hq, Hkv, S, S, P, d, False)
    dev = {k: v.cuda() for k, v in t.items()}
    scale = 1.0 / np.sqrt(d)
    o1, l1 = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"], scale)
    o2, l2 = pskv.pskv_attn_fwd_decode(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"],
                                       None, scale)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)


@pytest.mark.gpu
def test_growing_the_suffix_token_by_token_reproduces_the_full_evaluation():
    """Three decode steps of one token each give the last three rows of a full-suffix call."""
    B, Hq, Hkv, S, P, d = 24, 8, 2, 16, 256, 128
    t, _ = make(B, Hq, Hkv, S, S, P, d, False)
    dev = {k: v.cuda() for k, v in t.items()}
    scale = 1.0 / np.sqrt(d)
    o_full, l_full = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"],
                                        scale)
    for step, L in enumerate((S - 2, S - 1, S)):
        lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
        q1 = dev["q"][:, :, L - 1:L].contiguous()
        o1, l1 = pskv.pskv_attn_fwd_decode(q1, dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"],
                                           lens, scale)
        assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
        err = (o1.float() - o_full[:, :, L - 1:L].float()).abs().max().item()
        assert err <= 2e-2, (step, err)
        assert (l1 - l_full[:, :, L - 1:L]).abs().max().item() <= 1e-3 * max(1.0, l_full.abs().max().item())


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(40, 8, 2, 1, 24, 200, 128), (3, 8, 2, 256, 256, 100, 128)])
def test_rows_outside_the_safe_exponent_range_are_redone_in_every_tiling(shape):
    """Scores of several hundred nats in a few rows: the tensor-core kernel marks those rows and recomputes
    them with a running maximum, also when its tiles are whole candidates (decode) or lie inside one
    candidate (long suffix)."""
    B, Hq, Hkv, Sq, Skv, P, d = shape
    t, _ = make(B, Hq, Hkv, Sq, Skv, P, d, False)
    q = t["q"].float()
    q[1, 2, 0] *= 60.0
    q[B - 1, 0, Sq - 1] *= 45.0
    q[0, Hq - 1, Sq // 2] *= -50.0
    t["q"] = q.to(torch.bfloat16)
    scale = 1.0 / np.sqrt(d)
    out, lse = pskv.pskv_attn_fwd_decode(t["q"].cuda(), t["prefix_k"].cuda(), t["prefix_v"].cuda(), t["suffix_k"].cuda(),
                                         t["suffix_v"].cuda(), None, scale)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    f = {k: parity.to_f64(v) for k, v in t.items()}
    ro, rl = oracle.attn_fwd_decode(f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], scale)
    assert np.abs(rl).max() > 100.0
    parity.check_tensor("out", parity.to_f64(out), ro)
    parity.check_lse(parity.to_f64(lse), rl)


def test_decode_arguments_are_checked_on_the_host():
    L = pskv.binding.lib()
    fake = ctypes.c_void_p(4096)
    call = lambda Sq, Skv, lens=None, ws=256: L.pskv_attn_fwd_decode(
        fake, fake, fake, fake, fake, lens, ctypes.c_float(0.1), fake, fake, 8, 4, 4, Sq, Skv, 16, 128, fake, ws, None)
    assert call(9, 8) == pskv.PSKV_ERR_INVALID_ARG                       # more queries than cache rows
    assert call(0, 8) == pskv.PSKV_ERR_INVALID_ARG
    assert call(1, 8, ctypes.c_void_p(4098)) == pskv.PSKV_ERR_INVALID_ARG  # misaligned length array
    assert call(1, 8, None, 16) == pskv.PSKV_ERR_WORKSPACE
    assert pskv.pskv_attn_fwd_decode_workspace_bytes(8, 4, 4, 1, 8, 16, 128) == 256
    assert pskv.pskv_attn_fwd_decode_workspace_bytes(8, 4, 4, 9, 8, 16, 128) == 0
    assert pskv.pskv_attn_bwd_decode_workspace_bytes(8, 4, 4, 2, 8, 16, 128) >= 8 * 4 * 2 * 4


@pytest.mark.gpu
def test_single_key_rows_are_exact_up_to_one_rounding_of_the_probability():
    """One cached token and no prefix: the softmax has a single term, so out is that token's value row
    and dQ is zero.  The tensor-core forward feeds bf16 probabilities to the value contraction and
    divides by the fp32 sum of the unrounded ones, so `out` may differ from the value row by one bf16
    rounding (2^-8 relative), and the backward, which takes that `out`, sees D = <dout, out> off by the
    same amount: |dQ| stays below scale * 2^-7 * sum_c |dout_c v_c| * |k| instead of being exactly zero."""
    B, Hq, Hkv, d = 18, 14, 2, 128
    t, _ = make(B, Hq, Hkv, 1, 1, 0, d, False)
    scale = 1.0 / np.sqrt(d)
    dev = {k: v.cuda() for k, v in t.items()}
    out, lse = pskv.pskv_attn_fwd_decode(dev["q"], None, None, dev["suffix_k"], dev["suffix_v"], None, scale)
    n_rep = Hq // Hkv
    v = t["suffix_v"][:, :, 0].float().repeat_interleave(n_rep, dim=1)          # [B, Hq, d]
    k = t["suffix_k"][:, :, 0].float().repeat_interleave(n_rep, dim=1)
    o = out.cpu().float()[:, :, 0]
    assert torch.all((o - v).abs() <= 2.0 ** -7 * v.abs() + 1e-6)
    s = (t["q"].float()[:, :, 0] * k).sum(-1) * scale
    assert torch.all((lse.cpu()[:, :, 0] - s).abs() <= 1e-3 * torch.clamp(s.abs(), min=1.0))
    dq, dk, dv = pskv.pskv_attn_bwd_decode(dev["dout"], dev["q"], None, None, dev["suffix_k"], dev["suffix_v"], None,
                                           out, lse, scale)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dp = (t["dout"].float()[:, :, 0] * v).abs().sum(-1)                           # sum |dout_c v_c|, [B, Hq]
    bound = scale * 2.0 ** -7 * dp[..., None] * k.abs() + 1e-5
    assert torch.all(dq.cpu().float()[:, :, 0].abs() <= bound)
    # dV of the one key is the sum of dout over its query heads (p = 1)
    ref_dv = t["dout"].float()[:, :, 0].reshape(B, Hkv, n_rep, d).sum(2)
    assert torch.all((dv.cpu().float()[:, :, 0] - ref_dv).abs() <= 2.0 ** -7 * ref_dv.abs() + 2e-2)
