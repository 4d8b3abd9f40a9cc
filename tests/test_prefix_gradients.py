"""pskv_attn_bwd_prefix: gradients of the shared prefix cache (summed over all candidates) against the
fp64 oracle, on the tensor-core kernel (head dim 128) and the general one, with and without a gradient
on the log-sum-exp."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity
from paper_2603_13420_b200.inputs import Workload, make_inputs

SHAPES = [
    # B, Hq, Hkv, S, P, d, with_dlse
    (24, 32, 8, 48, 256, 128, False),   # the GQA layer shape: four key blocks, row groups of 192
    (40, 4, 4, 40, 160, 128, True),     # MHA, a partial last key block, lse gradient
    (7, 8, 2, 16, 33, 128, False),      # one key block, odd candidate count
    (3, 14, 2, 5, 70, 128, True),       # n_rep = 7, S = 5
    (6, 8, 2, 16, 100, 64, False),      # head dim 64: general kernel
    (130, 8, 2, 8, 64, 128, False),     # more candidates than one chunk holds
]


@pytest.mark.gpu
@pytest.mark.parametrize("shape", SHAPES)
def test_prefix_gradients_match_the_oracle(shape):
    B, Hq, Hkv, S, P, d, with_dlse = shape
    w = Workload("pre", 900 + sum(shape[:6]), B=B, Hq=Hq, Hkv=Hkv, d=d, P=P, S=S, backward=True)
    t = make_inputs(w, with_dout=True)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed)
    dlse = torch.randn((B, Hq, S), generator=gen, dtype=torch.float32) if with_dlse else None
    dev = {k: v.cuda() for k, v in t.items()}
    out, lse = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"], w.scale)
    dk = parity.Guarded((Hkv, P, d), torch.bfloat16, "cuda")
    dv = parity.Guarded((Hkv, P, d), torch.bfloat16, "cuda")
    pskv.pskv_attn_bwd_prefix(dev["dout"], None if dlse is None else dlse.cuda(), dev["q"], dev["prefix_k"],
                              dev["prefix_v"], out, lse, w.scale, dk_prefix=dk.view, dv_prefix=dv.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dk.check("dk_prefix"); dv.check("dv_prefix")
    f = {k: parity.to_f64(v) for k, v in t.items()}
    rk, rv = oracle.attn_bwd_prefix(f["dout"], f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"],
                                    w.scale, None if dlse is None else dlse.numpy().astype(np.float64))
    parity.check_tensor("dk_prefix", parity.to_f64(dk.view), rk)
    parity.check_tensor("dv_prefix", parity.to_f64(dv.view), rv)


def test_prefix_gradient_arguments_are_checked_on_the_host():
    L = pskv.binding.lib()
    fake = ctypes.c_void_p(4096)
    call = lambda P, ws=1 << 30, dk=fake: L.pskv_attn_bwd_prefix(fake, None, fake, fake, fake, fake, fake, ctypes.c_float(0.1),
                                                                  dk, fake, 8, 4, 4, 8, P, 128, fake, ws, None)
    assert call(0) == pskv.PSKV_ERR_INVALID_ARG          # no prefix, nothing to differentiate
    assert call(16, dk=None) == pskv.PSKV_ERR_INVALID_ARG
    assert call(16, ws=64) == pskv.PSKV_ERR_WORKSPACE
    assert pskv.pskv_attn_bwd_prefix_workspace_bytes(8, 4, 4, 8, 16, 128) >= 8 * 4 * 8 * 4 + 2 * 4 * 16 * 128 * 4
    assert pskv.pskv_attn_bwd_prefix_workspace_bytes(8, 4, 4, 8, 0, 128) == 0
