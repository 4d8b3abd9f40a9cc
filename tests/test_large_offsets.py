"""More than 2^31 elements per tensor: element offsets no longer fit 32 bits.  GPU parity on the first
and last candidates (the ones whose offsets are smallest and largest) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity

pytestmark = pytest.mark.gpu


def _device_randn(shape, seed):
    """bf16 normal values generated on the device in slices (a 4 GB tensor never exists in fp32)."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    x = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    step = max(1, shape[0] // 16)
    for b0 in range(0, shape[0], step):
        n = min(step, shape[0] - b0)
        x[b0:b0 + n] = torch.randn((n,) + tuple(shape[1:]), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    return x


@pytest.mark.parametrize("S,B", [(48, 11000),     # tensor-core kernels
                                  (47, 11200)])    # general kernels (S not a multiple of 8)
def test_forward_and_backward_with_more_than_2_to_31_elements(S, B):
    Hq, Hkv, P, d = 32, 8, 256, 128            # q, out, dout, dq: more than 2^31 elements each
    first_past = 2 ** 31 // (Hq * S * d) + 1   # first candidate that lies wholly past element 2^31
    assert first_past < B - 2
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2 ** 30:
        pytest.skip("needs about 24 GB of device memory")
    scale = 1.0 / np.sqrt(d)
    q = _device_randn((B, Hq, S, d), 1)
    dout = _device_randn((B, Hq, S, d), 2)
    sk = _device_randn((B, Hkv, S, d), 3)
    sv = _device_randn((B, Hkv, S, d), 4)
    pk = _device_randn((Hkv, P, d), 5)
    pv = _device_randn((Hkv, P, d), 6)
    out, lse = pskv.pskv_attn_fwd(q, pk, pv, sk, sv, scale)
    dq, dk, dv = pskv.pskv_attn_bwd(dout, q, pk, pv, sk, sv, out, lse, scale)
    torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    cand = [0, 1, B // 2, first_past - 1, first_past, B - 2, B - 1]   # around the first candidate past 2^31 elements
    idx = torch.tensor(cand, device="cuda")
    f = lambda x: parity.to_f64(x.index_select(0, idx).cpu())
    fp = lambda x: parity.to_f64(x.cpu())
    ref_out, ref_lse = oracle.attn_fwd(f(q), fp(pk), fp(pv), f(sk), f(sv), scale)
    parity.check_tensor("out", f(out), ref_out, strict_abs=True)
    parity.check_lse(f(lse), ref_lse)
    rq, rk, rv = oracle.attn_bwd(f(dout), f(q), fp(pk), fp(pv), f(sk), f(sv), scale)
    parity.check_tensor("dq", f(dq), rq)
    parity.check_tensor("dk_suffix", f(dk), rk)
    parity.check_tensor("dv_suffix", f(dv), rv)
    # nothing between the sampled candidates was left unwritten
    assert torch.isfinite(lse).all()
    assert bool((out[B - 64:].float().abs().amax(dim=(1, 2, 3)) > 0).all())
    assert bool((dq[B - 64:].float().abs().amax(dim=(1, 2, 3)) > 0).all())


def test_decode_shaped_call_with_a_suffix_cache_of_more_than_2_to_31_elements():
    Hq, Hkv, Sq, Skv, P, d = 32, 8, 1, 48, 256, 128
    B = 44000                                  # suffix K, V, dK, dV: 2.16e9 elements each
    assert B * Hkv * Skv * d > 2 ** 31
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2 ** 30:
        pytest.skip("needs about 20 GB of device memory")
    scale = 1.0 / np.sqrt(d)
    q = _device_randn((B, Hq, Sq, d), 11)
    dout = _device_randn((B, Hq, Sq, d), 12)
    sk = _device_randn((B, Hkv, Skv, d), 13)
    sv = _device_randn((B, Hkv, Skv, d), 14)
    pk = _device_randn((Hkv, P, d), 15)
    pv = _device_randn((Hkv, P, d), 16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(17)
    lens = torch.randint(Sq, Skv + 1, (B,), generator=gen, dtype=torch.int32)
    dlens = lens.cuda()
    out, lse = pskv.pskv_attn_fwd_decode(q, pk, pv, sk, sv, dlens, scale)
    dq, dk, dv = pskv.pskv_attn_bwd_decode(dout, q, pk, pv, sk, sv, dlens, out, lse, scale)
    torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    first_past = 2 ** 31 // (Hkv * Skv * d) + 1
    cand = [0, B // 3, first_past - 1, first_past, B - 2, B - 1]
    idx = torch.tensor(cand, device="cuda")
    f = lambda x: parity.to_f64(x.index_select(0, idx).cpu())
    fp = lambda x: parity.to_f64(x.cpu())
    nl = lens[cand].numpy()
    ref_out, ref_lse = oracle.attn_fwd_decode(f(q), fp(pk), fp(pv), f(sk), f(sv), scale, nl)
    parity.check_tensor("out", f(out), ref_out, strict_abs=True)
    parity.check_lse(f(lse), ref_lse)
    rq, rk, rv = oracle.attn_bwd_decode(f(dout), f(q), fp(pk), fp(pv), f(sk), f(sv), scale, nl)
    parity.check_tensor("dq", f(dq), rq)
    parity.check_tensor("dk_suffix", f(dk), rk)
    parity.check_tensor("dv_suffix", f(dv), rv)


def test_target_cross_entropy_with_more_than_2_to_31_hidden_elements():
    N, Lr, Dm, V = 26300, 20, 4096, 2048       # hidden: 2.15e9 elements
    assert N * Lr * Dm > 2 ** 31
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * 2 ** 30:
        pytest.skip("needs about 6 GB of device memory")
    hidden = _device_randn((N, Lr, Dm), 21)
    weight = _device_randn((V, Dm), 22) * 0.05
    weight = weight.to(torch.bfloat16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(23)
    target = torch.randint(0, V, (N, Lr), generator=gen, dtype=torch.int32)
    mask = (torch.rand((N, Lr), generator=gen) < 0.6).to(torch.float32)
    nll, lse, loss = pskv.pskv_target_ce_fwd(hidden, weight, target.cuda(), mask.cuda())
    torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    first_past = 2 ** 31 // (Lr * Dm) + 1
    cand = [0, N // 2, first_past - 1, first_past, N - 1]
    idx = torch.tensor(cand, device="cuda")
    h = parity.to_f64(hidden.index_select(0, idx).cpu())
    r_nll, r_lse, r_loss = oracle.target_ce_fwd(h, parity.to_f64(weight.cpu()), target[cand].numpy(), mask[cand].numpy())
    g = lambda x: x.index_select(0, idx).cpu().double().numpy()
    rel = lambda a, b: np.max(np.abs(a - b) / np.maximum(np.abs(b), 1.0))
    assert rel(g(lse), r_lse) <= 1e-3
    assert rel(g(nll), r_nll) <= 1e-3
    assert rel(g(loss), r_loss) <= 1e-3
    assert torch.isfinite(loss).all() and torch.isfinite(lse).all()


def test_multi_instruction_calls_with_more_than_2_to_31_elements():
    Hq, Hkv, S, Pmax, d, Bp = 32, 8, 48, 256, 128, 4
    B = 11200
    lens = [256, 200, 130, 77]
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2 ** 30:
        pytest.skip("needs about 24 GB of device memory")
    scale = 1.0 / np.sqrt(d)
    q = _device_randn((B, Hq, S, d), 31)
    dout = _device_randn((B, Hq, S, d), 32)
    sk = _device_randn((B, Hkv, S, d), 33)
    sv = _device_randn((B, Hkv, S, d), 34)
    pk = _device_randn((Bp, Hkv, Pmax, d), 35)
    pv = _device_randn((Bp, Hkv, Pmax, d), 36)
    out, lse = pskv.pskv_attn_fwd_multi(q, pk, pv, lens, sk, sv, scale)
    dq, dk, dv = pskv.pskv_attn_bwd_multi(dout, q, pk, pv, lens, sk, sv, out, lse, scale)
    torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    Kq = B // Bp
    cand = [i * Kq + j for i in range(Bp) for j in (0, Kq - 1)]      # first and last candidate of every instruction
    assert cand[-1] * Hq * S * d > 2 ** 31
    idx = torch.tensor(cand, device="cuda")
    f = lambda x: parity.to_f64(x.index_select(0, idx).cpu())
    fp = lambda x: parity.to_f64(x.cpu())
    mask = np.zeros((Bp, Pmax))
    for i, n in enumerate(lens):
        mask[i, Pmax - n:] = 1.0                                      # left padding
    ref_out, ref_lse = oracle.attn_fwd_multi(f(q), fp(pk), fp(pv), mask, f(sk), f(sv), scale)
    parity.check_tensor("out", f(out), ref_out, strict_abs=True)
    parity.check_lse(f(lse), ref_lse)
    rq, rk, rv = oracle.attn_bwd_multi(f(dout), f(q), fp(pk), fp(pv), mask, f(sk), f(sv), scale)
    parity.check_tensor("dq", f(dq), rq)
    parity.check_tensor("dk_suffix", f(dk), rk)
    parity.check_tensor("dv_suffix", f(dv), rv)


def test_prefix_gradients_over_more_than_2_to_31_elements_equal_the_sum_over_two_halves():
    """The prefix-cache gradients are sums over candidates, so the call over all candidates must equal
    the sum of two calls over halves whose own element offsets stay below 2^31."""
    Hq, Hkv, S, P, d = 32, 8, 48, 256, 128
    B = 11000
    free, _ = torch.cuda.mem_get_info()
    if free < 30 * 2 ** 30:
        pytest.skip("needs about 20 GB of device memory")
    scale = 1.0 / np.sqrt(d)
    q = _device_randn((B, Hq, S, d), 41)
    dout = _device_randn((B, Hq, S, d), 42)
    sk = _device_randn((B, Hkv, S, d), 43)
    sv = _device_randn((B, Hkv, S, d), 44)
    pk = _device_randn((Hkv, P, d), 45)
    pv = _device_randn((Hkv, P, d), 46)
    out, lse = pskv.pskv_attn_fwd(q, pk, pv, sk, sv, scale)
    gk, gv = pskv.pskv_attn_bwd_prefix(dout, None, q, pk, pv, out, lse, scale)
    h = B // 2
    parts = [pskv.pskv_attn_bwd_prefix(dout[a:b], None, q[a:b], pk, pv, out[a:b], lse[a:b], scale)
             for a, b in ((0, h), (h, B))]
    torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    for full, p0, p1 in ((gk, parts[0][0], parts[1][0]), (gv, parts[0][1], parts[1][1])):
        ref = p0.float() + p1.float()
        err = (full.float() - ref).abs()
        # one bf16 rounding each of the full result and of the two halves (which may cancel), plus the
        # order of the fp32 additions
        tol = 2.0 ** -8 * (full.float().abs() + p0.float().abs() + p1.float().abs()) + 2e-3 * ref.abs().mean()
        assert bool((err <= tol).all()), float((err - tol).max())
