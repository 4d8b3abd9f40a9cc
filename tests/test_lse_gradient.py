"""pskv_attn_bwd_lse: the backward with a gradient arriving on the log-sum-exp output, against the fp64
oracle (L = sum(out * dout) + sum(lse * dlse)), on the tensor-core and the general kernel families."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity
from paper_2603_13420_b200.inputs import Workload, make_inputs

SHAPES = [
    # B, Hq, Hkv, S, P, d
    (24, 32, 8, 48, 256, 128),   # the GQA layer shape (tensor-core dQ and suffix-gradient kernels)
    (16, 4, 4, 40, 160, 128),    # MHA
    (6, 8, 2, 16, 300, 64),      # head dim 64
    (4, 4, 2, 5, 33, 128),       # general kernels (odd S)
]


@pytest.mark.gpu
@pytest.mark.parametrize("shape", SHAPES)
def test_backward_with_lse_gradient_matches_the_oracle(shape):
    B, Hq, Hkv, S, P, d = shape
    w = Workload("lse", 700 + sum(shape), B=B, Hq=Hq, Hkv=Hkv, d=d, P=P, S=S, backward=True)
    t = make_inputs(w, with_dout=True)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed)
    dlse = torch.randn((B, Hq, S), generator=gen, dtype=torch.float32)
    dev = {k: v.cuda() for k, v in t.items()}
    out, lse = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"], w.scale)
    dq = parity.Guarded((B, Hq, S, d), torch.bfloat16, "cuda")
    dk = parity.Guarded((B, Hkv, S, d), torch.bfloat16, "cuda")
    dv = parity.Guarded((B, Hkv, S, d), torch.bfloat16, "cuda")
    pskv.pskv_attn_bwd_lse(dev["dout"], dlse.cuda(), dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"],
                           dev["suffix_v"], out, lse, w.scale, dq=dq.view, dk_suffix=dk.view, dv_suffix=dv.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dq.check("dq"); dk.check("dk_suffix"); dv.check("dv_suffix")
    f = {k: parity.to_f64(v) for k, v in t.items()}
    rq, rk, rv = oracle.attn_bwd_lse(f["dout"], dlse.numpy().astype(np.float64), f["q"], f["prefix_k"], f["prefix_v"],
                                     f["suffix_k"], f["suffix_v"], w.scale)
    parity.check_tensor("dq", parity.to_f64(dq.view), rq)
    parity.check_tensor("dk_suffix", parity.to_f64(dk.view), rk)
    parity.check_tensor("dv_suffix", parity.to_f64(dv.view), rv)
    # and the lse term really is there: the plain backward differs
    pq, _, _ = oracle.attn_bwd(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], w.scale)
    assert np.max(np.abs(pq - rq)) > 10 * np.max(np.abs(parity.to_f64(dq.view) - rq))


def test_lse_gradient_arguments_are_checked_on_the_host():
    L = pskv.binding.lib()
    fake = ctypes.c_void_p(4096)
    call = lambda dlse: L.pskv_attn_bwd_lse(fake, dlse, fake, fake, fake, fake, fake, fake, fake, ctypes.c_float(0.1),
                                            fake, fake, fake, 8, 4, 4, 8, 16, 128, fake, 1 << 20, None)
    assert call(None) == pskv.PSKV_ERR_INVALID_ARG
    assert call(ctypes.c_void_p(4100)) == pskv.PSKV_ERR_INVALID_ARG
