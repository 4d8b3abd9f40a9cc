"""HostStep: a layer step whose inputs and results are pinned host tensors, run as candidate chunks
through an upload, a compute and a download stream.  Candidates never interact, so the chunked step must
reproduce the unchunked library calls bit for bit; one oracle comparison guards against both being wrong
together."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity
from paper_2603_13420_b200.host_step import HostStep


@pytest.mark.gpu
@pytest.mark.parametrize("B,chunks", [(40, 8), (37, 5), (6, 8), (64, 16)])
def test_chunked_host_step_equals_the_unchunked_calls(B, chunks):
    Hq, Hkv, S, P, d = 8, 2, 16, 200, 128
    gen = torch.Generator(device="cpu")
    gen.manual_seed(260313420 + B)
    draw = lambda *s: torch.randn(s, generator=gen, dtype=torch.float32).to(torch.bfloat16).pin_memory()
    hin = dict(q=draw(B, Hq, S, d), dout=draw(B, Hq, S, d), suffix_k=draw(B, Hkv, S, d), suffix_v=draw(B, Hkv, S, d),
               prefix_k=draw(Hkv, P, d), prefix_v=draw(Hkv, P, d))
    hout = dict(out=torch.empty_like(hin["q"]).pin_memory(), dq=torch.empty_like(hin["q"]).pin_memory(),
                lse=torch.empty((B, Hq, S), dtype=torch.float32).pin_memory(),
                dk=torch.empty_like(hin["suffix_k"]).pin_memory(), dv=torch.empty_like(hin["suffix_v"]).pin_memory())
    scale = d ** -0.5
    step = HostStep(B, Hq, Hkv, S, P, d, scale, "cuda", chunks=chunks)
    for _ in range(2):   # the second run reuses streams and buffers
        for v in hout.values():
            v.fill_(float("nan"))
        step.run(hin, hout)
        torch.cuda.synchronize()
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    dev = {k: v.cuda() for k, v in hin.items()}
    out, lse = pskv.pskv_attn_fwd(dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"], dev["suffix_v"], scale)
    dq, dk, dv = pskv.pskv_attn_bwd(dev["dout"], dev["q"], dev["prefix_k"], dev["prefix_v"], dev["suffix_k"],
                                    dev["suffix_v"], out, lse, scale)
    for name, ref in (("out", out), ("lse", lse), ("dq", dq), ("dk", dk), ("dv", dv)):
        assert torch.equal(hout[name], ref.cpu()), name
    f = {k: parity.to_f64(v) for k, v in hin.items()}
    ref_out, _ = oracle.attn_fwd(f["q"], f["prefix_k"], f["prefix_v"], f["suffix_k"], f["suffix_v"], scale)
    parity.check_tensor("out", parity.to_f64(hout["out"]), ref_out)
