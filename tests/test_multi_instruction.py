"""Batched multi-instruction variant (Sec. 4.3): one left-padded prefix cache per instruction, reused
by that instruction's candidates.  GPU parity against the fp64 oracle (which gathers the unmasked
prefix rows per candidate and runs plain attention), plus host-side argument checks."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity

SEED = 260313420 + 77


def make(B, Bp, Hq, Hkv, S, Pmax, d, lens, seed=SEED):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + B + 7 * Bp + 13 * S + Pmax)

    def draw(*shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16)

    t = dict(q=draw(B, Hq, S, d), prefix_k=draw(Bp, Hkv, Pmax, d), prefix_v=draw(Bp, Hkv, Pmax, d),
             suffix_k=draw(B, Hkv, S, d), suffix_v=draw(B, Hkv, S, d), dout=draw(B, Hq, S, d))
    # padding rows hold large finite garbage: it must not reach any result
    for i, n in enumerate(lens):
        t["prefix_k"][i, :, : Pmax - n] = 3.0e4
        t["prefix_v"][i, :, : Pmax - n] = -3.0e4
    return t


CASES = [
    # B, Bp, Hq, Hkv, S, Pmax, d, lens
    (12, 3, 8, 2, 16, 300, 128, (300, 129, 40)),   # tensor-core path, ragged prefixes, GQA
    (8, 2, 4, 4, 40, 160, 128, (160, 96)),         # MHA, 40-token suffix
    (6, 3, 4, 2, 8, 64, 64, (0, 64, 17)),          # head dim 64, an empty prefix, odd length
    (4, 4, 2, 1, 5, 33, 128, (33, 1, 20, 7)),      # general kernels (S not a multiple of 8)
    (64, 2, 32, 8, 48, 256, 128, (256, 200)),      # the GQA layer shape, two instructions
    (16, 4, 8, 2, 16, 600, 128, (600, 0, 130, 471)),  # one launch, prefix blocks streamed; an empty prefix and
                                                   # one whose padding covers three whole key blocks
    (8, 2, 4, 4, 32, 96, 64, (96, 50)),            # one launch, head dim 64
    (40, 5, 8, 2, 32, 200, 128, (200, 199, 73, 128, 1)),  # one launch, five instructions, odd lengths
]

# cases whose shape allows all instructions in one launch (every tile inside one instruction); the library takes
# that form by itself only while the padding is a small share of the keys, so the tests name the form
ONE_LAUNCH_SHAPES = {0, 4, 5, 6, 7}


@pytest.fixture(params=["one", "passes"])
def form(request, monkeypatch):
    pskv.pskv_set_multi_form(request.param)
    return request.param


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
def test_forward_and_backward_match_the_oracle(case, form):
    B, Bp, Hq, Hkv, S, Pmax, d, lens = case
    one = form == "one" and CASES.index(case) in ONE_LAUNCH_SHAPES
    t = make(*case)
    scale = 1.0 / np.sqrt(d)
    dev = {k: v.cuda() for k, v in t.items()}
    out = parity.Guarded((B, Hq, S, d), torch.bfloat16, "cuda")
    lse = parity.Guarded((B, Hq, S), torch.float32, "cuda")
    n0 = pskv.pskv_kernel_launches()
    pskv.pskv_attn_fwd_multi(dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"], dev["suffix_v"],
                             scale, out=out.view, lse=lse.view)
    assert pskv.pskv_kernel_launches() - n0 == (1 if one else Bp)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    out.check("out"); lse.check("lse")
    f = {k: parity.to_f64(v) for k, v in t.items()}
    mask = oracle.left_padding_mask(lens, Pmax)
    ref_out, ref_lse = oracle.attn_fwd_multi(f["q"], f["prefix_k"], f["prefix_v"], mask, f["suffix_k"], f["suffix_v"], scale)
    parity.check_tensor("out", parity.to_f64(out.view), ref_out, strict_abs=(min(lens) + S >= 128))
    parity.check_lse(parity.to_f64(lse.view), ref_lse)

    dq = parity.Guarded((B, Hq, S, d), torch.bfloat16, "cuda")
    dk = parity.Guarded((B, Hkv, S, d), torch.bfloat16, "cuda")
    dv = parity.Guarded((B, Hkv, S, d), torch.bfloat16, "cuda")
    n0 = pskv.pskv_kernel_launches()
    pskv.pskv_attn_bwd_multi(dev["dout"], dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"],
                             dev["suffix_v"], out.view, lse.view, scale, dq=dq.view, dk_suffix=dk.view,
                             dv_suffix=dv.view)
    if one:   # suffix gradients together with the row statistic (a pre-pass of its own for suffixes beyond 48
        # keys), then one dQ launch for all instructions
        assert pskv.pskv_kernel_launches() - n0 == (2 if S <= 48 and (Hq // Hkv) * S >= 128 else 3)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dq.check("dq"); dk.check("dk_suffix"); dv.check("dv_suffix")
    rq, rk, rv = oracle.attn_bwd_multi(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], mask, f["suffix_k"],
                                       f["suffix_v"], scale)
    parity.check_tensor("dq", parity.to_f64(dq.view), rq)
    parity.check_tensor("dk_suffix", parity.to_f64(dk.view), rk)
    parity.check_tensor("dv_suffix", parity.to_f64(dv.view), rv)


@pytest.mark.gpu
def test_one_launch_redoes_rows_outside_the_safe_exponent_range_with_their_own_prefix(monkeypatch):
    """Scores of several hundred nats in rows of different instructions: the one-launch forward marks them
    and recomputes each with a running maximum against its own instruction's unpadded prefix."""
    pskv.pskv_set_multi_form("one")
    case = (16, 4, 8, 2, 16, 300, 128, (300, 40, 170, 1))
    B, Bp, Hq, Hkv, S, Pmax, d, lens = case
    t = make(*case)
    q = t["q"].float()
    q[1, 2, 3] *= 60.0      # instruction 0
    q[5, 0, 15] *= -50.0    # instruction 1
    q[15, 7, 0] *= 45.0     # instruction 3
    t["q"] = q.to(torch.bfloat16)
    scale = 1.0 / np.sqrt(d)
    dev = {k: v.cuda() for k, v in t.items()}
    n0 = pskv.pskv_kernel_launches()
    out, lse = pskv.pskv_attn_fwd_multi(dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"],
                                        dev["suffix_v"], scale)
    assert pskv.pskv_kernel_launches() - n0 == 1
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    f = {k: parity.to_f64(v) for k, v in t.items()}
    mask = oracle.left_padding_mask(lens, Pmax)
    ref_out, ref_lse = oracle.attn_fwd_multi(f["q"], f["prefix_k"], f["prefix_v"], mask, f["suffix_k"], f["suffix_v"], scale)
    assert np.abs(ref_lse).max() > 100.0
    parity.check_tensor("out", parity.to_f64(out), ref_out)
    parity.check_lse(parity.to_f64(lse), ref_lse)


@pytest.mark.gpu
def test_one_unpadded_instruction_equals_the_single_prefix_call_bit_for_bit():
    B, Hq, Hkv, S, P, d = 16, 8, 2, 16, 200, 128
    t = make(B, 1, Hq, Hkv, S, P, d, (P,))
    dev = {k: v.cuda() for k, v in t.items()}
    scale = 1.0 / np.sqrt(d)
    o1, l1 = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"][0], dev["prefix_v"][0], dev["suffix_k"], dev["suffix_v"], scale)
    o2, l2 = pskv.pskv_attn_fwd_multi(dev["q"], dev["prefix_k"], dev["prefix_v"], (P,), dev["suffix_k"],
                                      dev["suffix_v"], scale)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)


def test_multi_arguments_are_checked_on_the_host():
    L = pskv.binding.lib()
    lens = (ctypes.c_int * 2)(4, 9)
    fake = ctypes.c_void_p(4096)
    args = lambda B, Bp, Pmax, ln: L.pskv_attn_fwd_multi(fake, fake, fake, ctypes.cast(ln, ctypes.c_void_p), fake, fake,
                                                          ctypes.c_float(0.1), fake, fake, B, Bp, 4, 4, 8, Pmax, 128, fake, 256, None)
    assert args(7, 2, 16, lens) == pskv.PSKV_ERR_INVALID_ARG          # B not a multiple of Bp
    assert args(8, 2, 8, lens) == pskv.PSKV_ERR_INVALID_ARG           # a length beyond Pmax
    assert args(8, 2, 16, None) == pskv.PSKV_ERR_INVALID_ARG          # no length array
    assert pskv.pskv_attn_bwd_multi_workspace_bytes(8, 2, 4, 4, 8, 16, 128) >= 8 * 4 * 8 * 4
    assert pskv.pskv_attn_fwd_multi_workspace_bytes(7, 2, 4, 4, 8, 16, 128) == 0


@pytest.mark.gpu
def test_the_library_takes_one_launch_by_itself_whenever_the_shape_allows_it(monkeypatch):
    pskv.pskv_set_multi_form("auto")
    for lens in ((256, 200), (256, 16)):
        case = (64, 2, 32, 8, 48, 256, 128, lens)
        t = make(*case)
        dev = {k: v.cuda() for k, v in t.items()}
        n0 = pskv.pskv_kernel_launches()
        out, lse = pskv.pskv_attn_fwd_multi(dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"],
                                            dev["suffix_v"], 0.088)
        assert pskv.pskv_kernel_launches() - n0 == 1
        n0 = pskv.pskv_kernel_launches()
        pskv.pskv_attn_bwd_multi(dev["dout"], dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"],
                                 dev["suffix_v"], out, lse, 0.088)
        assert pskv.pskv_kernel_launches() - n0 == 2   # suffix gradients with the row statistic, then dQ


@pytest.mark.gpu
def test_back_to_back_one_launch_calls_with_prefixes_that_are_padding_only(monkeypatch):
    """Instructions whose prefix is empty skip every prefix block, yet the resident copy of their run is
    still loaded: those loads have to land before the CTA exits or arms the buffers again.  Many calls in a
    row without a synchronisation in between, each checked against the first."""
    pskv.pskv_set_multi_form("one")
    case = (64, 4, 32, 8, 48, 256, 128, (256, 0, 0, 130))
    B, Bp, Hq, Hkv, S, Pmax, d, lens = case
    t = make(*case)
    dev = {k: v.cuda() for k, v in t.items()}
    scale = 1.0 / np.sqrt(d)
    ref_out, ref_lse = pskv.pskv_attn_fwd_multi(dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"],
                                                dev["suffix_v"], scale)
    torch.cuda.synchronize()
    outs = []
    for _ in range(40):
        outs.append(pskv.pskv_attn_fwd_multi(dev["q"], dev["prefix_k"], dev["prefix_v"], lens, dev["suffix_k"],
                                             dev["suffix_v"], scale))
    torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    for o, l in outs:
        assert torch.equal(o, ref_out) and torch.equal(l, ref_lse)
