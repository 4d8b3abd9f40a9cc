"""The calls enqueue work and nothing else (no allocation, no synchronisation), so a layer step can be
captured into a CUDA graph and replayed on new contents of the same buffers.  Also covers the
multi-instruction call, whose passes fork onto an internal stream and join again inside the capture."""
import numpy as np
import pytest
import torch

import paper_2603_13420_b200 as pskv


def _draw(gen, *shape):
    return torch.randn(shape, generator=gen, dtype=torch.float32).to(torch.bfloat16).cuda()


@pytest.mark.gpu
def test_forward_and_backward_replay_from_a_cuda_graph():
    B, Hq, Hkv, S, P, d = 24, 8, 2, 16, 200, 128
    gen = torch.Generator(device="cpu")
    gen.manual_seed(5)
    t = {k: _draw(gen, *s) for k, s in dict(q=(B, Hq, S, d), pk=(Hkv, P, d), pv=(Hkv, P, d), sk=(B, Hkv, S, d),
                                             sv=(B, Hkv, S, d), do=(B, Hq, S, d)).items()}
    scale = d ** -0.5
    out, lse = torch.empty_like(t["q"]), torch.empty((B, Hq, S), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(t["q"]), torch.empty_like(t["sk"]), torch.empty_like(t["sv"])
    ws_f = torch.empty(256, dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(max(pskv.pskv_attn_bwd_workspace_bytes(B, Hq, Hkv, S, P, d), 256), dtype=torch.uint8, device="cuda")

    def step():
        pskv.pskv_attn_fwd(t["q"], t["pk"], t["pv"], t["sk"], t["sv"], scale, out=out, lse=lse, workspace=ws_f)
        pskv.pskv_attn_bwd(t["do"], t["q"], t["pk"], t["pv"], t["sk"], t["sv"], out, lse, scale, dq=dq, dk_suffix=dk,
                           dv_suffix=dv, workspace=ws_b)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):       # warm-up outside the capture (first-launch attribute calls)
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for trial in range(2):
        for k in ("q", "sk", "sv", "do"):   # new contents, same buffers
            t[k].copy_(_draw(gen, *t[k].shape))
        graph.replay()
        torch.cuda.synchronize()
        got = [x.clone() for x in (out, lse, dq, dk, dv)]
        step()
        torch.cuda.synchronize()
        for a, b in zip(got, (out, lse, dq, dk, dv)):
            assert torch.equal(a, b)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK


@pytest.mark.gpu
@pytest.mark.parametrize("form", ["passes", "one"])
def test_multi_instruction_forward_replays_from_a_cuda_graph(form, monkeypatch):
    pskv.pskv_set_multi_form(form)   # per-instruction passes on two streams / one launch
    B, Bp, Hq, Hkv, S, Pmax, d = 32, 4, 8, 2, 16, 160, 128
    lens = (160, 120, 64, 33)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(6)
    q, sk, sv = _draw(gen, B, Hq, S, d), _draw(gen, B, Hkv, S, d), _draw(gen, B, Hkv, S, d)
    pk, pv = _draw(gen, Bp, Hkv, Pmax, d), _draw(gen, Bp, Hkv, Pmax, d)
    out, lse = torch.empty_like(q), torch.empty((B, Hq, S), dtype=torch.float32, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    scale = d ** -0.5

    def step():
        pskv.pskv_attn_fwd_multi(q, pk, pv, lens, sk, sv, scale, out=out, lse=lse, workspace=ws)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    q.copy_(_draw(gen, B, Hq, S, d))
    graph.replay()
    torch.cuda.synchronize()
    got_out, got_lse = out.clone(), lse.clone()
    step()
    torch.cuda.synchronize()
    assert torch.equal(got_out, out) and torch.equal(got_lse, lse)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
