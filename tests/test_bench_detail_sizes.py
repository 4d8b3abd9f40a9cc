"""The secondary lines of the benchmark at the sizes and in the launch configuration it times them: the
decode-shaped forward at B = 512 and B = 2048 (one new token on a ragged 48-token suffix cache, C2 layer
shape) and the multi-instruction forward + backward with 8 instructions x 64 candidates (both prefix-length
lists of the benchmark), the prefix-cache gradients over all 512 candidates and the 2048-token prefill.  The GPU runs the whole
batch; the fp64 oracle runs the sampled candidates one by one (candidates never meet in this operator, so a
candidate evaluated alone is its row of the batch), except for the prefix gradients, which sum over all."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity
from paper_2603_13420_b200.inputs import WORKLOADS

pytestmark = pytest.mark.gpu

SEED = 260313420 + 4242
MULTI_LENS = [256, 240, 224, 208, 192, 176, 160, 144]
MULTI_LENS_UNEQUAL = [256, 32, 32, 32, 200, 100, 16, 64]


def _draw(gen, *shape):
    return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16)


def _sample(B, rng, extra=()):
    return sorted(set([0, 1, B - 1] + list(extra) + rng.integers(0, B, size=5).tolist()))


@pytest.mark.parametrize("B", [512, 2048])
def test_decode_forward_at_benchmark_size_sampled(B):
    w = WORKLOADS["C2"]
    Sq, Skv = 1, 48
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED + B)
    q, sk, sv = _draw(gen, B, w.Hq, Sq, w.d), _draw(gen, B, w.Hkv, Skv, w.d), _draw(gen, B, w.Hkv, Skv, w.d)
    pk, pv = _draw(gen, w.Hkv, w.P, w.d), _draw(gen, w.Hkv, w.P, w.d)
    lens = torch.randint(Sq, Skv + 1, (B,), generator=gen, dtype=torch.int32)
    lens[0], lens[B - 1] = Sq, Skv
    for b in range(B):  # rows past the cached tokens must not matter
        sk[b, :, int(lens[b]):] = 3.0e4
        sv[b, :, int(lens[b]):] = -3.0e4
    out = parity.Guarded((B, w.Hq, Sq, w.d), torch.bfloat16, "cuda")
    lse = parity.Guarded((B, w.Hq, Sq), torch.float32, "cuda")
    pskv.pskv_attn_fwd_decode(q.cuda(), pk.cuda(), pv.cuda(), sk.cuda(), sv.cuda(), lens.cuda(), w.scale,
                              out=out.view, lse=lse.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    out.check("out"); lse.check("lse")
    got_out, got_lse = parity.to_f64(out.view), parity.to_f64(lse.view)
    rng = np.random.default_rng(SEED + B)
    # (candidates 29..32 sit around the first tile boundary of the 30- and 32-candidate tilings)
    for c in _sample(B, rng, extra=(29, 30, 31, 32)):
        ref_out, ref_lse = oracle.attn_fwd_decode(parity.to_f64(q[c:c + 1]), parity.to_f64(pk), parity.to_f64(pv),
                                                  parity.to_f64(sk[c:c + 1]), parity.to_f64(sv[c:c + 1]), w.scale,
                                                  lens[c:c + 1].numpy())
        parity.check_tensor("out[%d]" % c, got_out[c:c + 1], ref_out)
        parity.check_lse(got_lse[c:c + 1], ref_lse)


@pytest.mark.parametrize("lens", [MULTI_LENS, MULTI_LENS_UNEQUAL], ids=["staggered", "unequal"])
def test_multi_instruction_step_at_benchmark_size_sampled(lens):
    w = WORKLOADS["C2"]
    Bp, Pmax, B = len(lens), w.P, w.B
    kq = B // Bp
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED + sum(lens))
    q, sk, sv, do = (_draw(gen, B, w.Hq, w.S, w.d), _draw(gen, B, w.Hkv, w.S, w.d), _draw(gen, B, w.Hkv, w.S, w.d),
                     _draw(gen, B, w.Hq, w.S, w.d))
    pk, pv = _draw(gen, Bp, w.Hkv, Pmax, w.d), _draw(gen, Bp, w.Hkv, Pmax, w.d)
    for i, n in enumerate(lens):  # the padding must not matter
        pk[i, :, :Pmax - n] = 3.0e4
        pv[i, :, :Pmax - n] = -3.0e4
    dev = [x.cuda() for x in (q, pk, pv, sk, sv, do)]
    out = parity.Guarded((B, w.Hq, w.S, w.d), torch.bfloat16, "cuda")
    lse = parity.Guarded((B, w.Hq, w.S), torch.float32, "cuda")
    n0 = pskv.pskv_kernel_launches()
    pskv.pskv_attn_fwd_multi(dev[0], dev[1], dev[2], lens, dev[3], dev[4], w.scale, out=out.view, lse=lse.view)
    assert pskv.pskv_kernel_launches() - n0 == 1   # the one-launch form, as timed
    dq = parity.Guarded((B, w.Hq, w.S, w.d), torch.bfloat16, "cuda")
    dk = parity.Guarded((B, w.Hkv, w.S, w.d), torch.bfloat16, "cuda")
    dv = parity.Guarded((B, w.Hkv, w.S, w.d), torch.bfloat16, "cuda")
    pskv.pskv_attn_bwd_multi(dev[5], dev[0], dev[1], dev[2], lens, dev[3], dev[4], out.view, lse.view, w.scale,
                             dq=dq.view, dk_suffix=dk.view, dv_suffix=dv.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    for g, name in ((out, "out"), (lse, "lse"), (dq, "dq"), (dk, "dk_suffix"), (dv, "dv_suffix")):
        g.check(name)
    got = {k: parity.to_f64(v.view) for k, v in (("out", out), ("lse", lse), ("dq", dq), ("dk", dk), ("dv", dv))}
    mask = oracle.left_padding_mask(lens, Pmax)
    rng = np.random.default_rng(SEED + sum(lens))
    # every instruction once, plus the candidates on both sides of each instruction boundary of a KV head's tiles
    cands = sorted(set(_sample(B, rng) + [i * kq for i in range(Bp)] + [i * kq - 1 for i in range(1, Bp)]))
    for c in cands:
        i = c // kq
        f = [parity.to_f64(x) for x in (q[c:c + 1], pk[i:i + 1], pv[i:i + 1], sk[c:c + 1], sv[c:c + 1], do[c:c + 1])]
        ref_out, ref_lse = oracle.attn_fwd_multi(f[0], f[1], f[2], mask[i:i + 1], f[3], f[4], w.scale)
        parity.check_tensor("out[%d]" % c, got["out"][c:c + 1], ref_out, strict_abs=(lens[i] + w.S >= 128))
        parity.check_lse(got["lse"][c:c + 1], ref_lse)
        rq, rk, rv = oracle.attn_bwd_multi(f[5], f[0], f[1], f[2], mask[i:i + 1], f[3], f[4], w.scale)
        parity.check_tensor("dq[%d]" % c, got["dq"][c:c + 1], rq)
        parity.check_tensor("dk_suffix[%d]" % c, got["dk"][c:c + 1], rk)
        parity.check_tensor("dv_suffix[%d]" % c, got["dv"][c:c + 1], rv)


def test_prefix_gradients_at_benchmark_size():
    """dK_p / dV_p at the C2 shape with all 512 candidates (every key's gradient is a sum over 98 304 query
    rows of its KV head, so nothing can be sampled): the whole result against the oracle."""
    from paper_2603_13420_b200.inputs import make_inputs
    w = WORKLOADS["C2"]
    t = make_inputs(w, with_dout=True)
    dev = {k: v.cuda() for k, v in t.items()}
    out, lse = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"], w.scale)
    dk = parity.Guarded((w.Hkv, w.P, w.d), torch.bfloat16, "cuda")
    dv = parity.Guarded((w.Hkv, w.P, w.d), torch.bfloat16, "cuda")
    pskv.pskv_attn_bwd_prefix(dev["dout"], None, dev["q"], dev["prefix_k"], dev["prefix_v"], out, lse, w.scale,
                              dk_prefix=dk.view, dv_prefix=dv.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dk.check("dk_prefix"); dv.check("dv_prefix")
    f = {k: parity.to_f64(v) for k, v in t.items()}
    rk, rv = oracle.attn_bwd_prefix(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"],
                                    w.scale, None)
    parity.check_tensor("dk_prefix", parity.to_f64(dk.view), rk)
    parity.check_tensor("dv_prefix", parity.to_f64(dv.view), rv)


def test_prefill_of_a_2048_token_sequence_sampled_heads():
    """The prefill line: causal self-attention of one 2048-token sequence in the C3 head layout (B = 1, P = 0,
    the sequence's K/V passed as the suffix), launched whole; two KV heads with their query heads go through
    the oracle (heads never meet either)."""
    w = WORKLOADS["C3"]
    S = w.P
    n_rep = w.Hq // w.Hkv
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED + S)
    q, k, v = _draw(gen, 1, w.Hq, S, w.d), _draw(gen, 1, w.Hkv, S, w.d), _draw(gen, 1, w.Hkv, S, w.d)
    out = parity.Guarded((1, w.Hq, S, w.d), torch.bfloat16, "cuda")
    lse = parity.Guarded((1, w.Hq, S), torch.float32, "cuda")
    pskv.pskv_attn_fwd(q.cuda(), None, None, k.cuda(), v.cuda(), w.scale, out=out.view, lse=lse.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    out.check("out"); lse.check("lse")
    got_out, got_lse = parity.to_f64(out.view), parity.to_f64(lse.view)
    empty = np.zeros((1, 0, w.d))
    for g in (0, w.Hkv - 1):
        hs = slice(g * n_rep, (g + 1) * n_rep)
        ref_out, ref_lse = oracle.attn_fwd(parity.to_f64(q[:, hs]), empty, empty, parity.to_f64(k[:, g:g + 1]),
                                           parity.to_f64(v[:, g:g + 1]), w.scale)
        # (the first rows see one or two keys: relative bounds, as everywhere a row has fewer than 128 keys)
        parity.check_tensor("out[head group %d]" % g, got_out[:, hs], ref_out)
        parity.check_lse(got_lse[:, hs], ref_lse)
