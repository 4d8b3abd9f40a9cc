"""pskv_target_ce_fwd: masked target cross-entropy fused with the vocabulary projection, against the fp64
oracle on seeded bf16 inputs (hidden states N(0,1), output head N(0, 1/Dm), so logits are O(1) with a few
large ones), plus host-side argument checks."""
import ctypes
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_13420_b200 as pskv
import parity


def make(N, Lr, Dm, V, seed, gain=1.0):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(260313420 + seed)
    h = (gain * torch.randn((N, Lr, Dm), generator=gen)).to(torch.bfloat16)
    w = (torch.randn((V, Dm), generator=gen) / math.sqrt(Dm)).to(torch.bfloat16)
    t = torch.randint(0, V, (N, Lr), generator=gen, dtype=torch.int32)
    m = (torch.rand((N, Lr), generator=gen) < 0.7).to(torch.float32)
    m[0] = 0.0           # a candidate without any weighted position
    t[0, 0] = -1         # an illegal id is fine where the mask is zero
    if N > 1:
        t[1, 0] = V - 1  # last vocabulary entry (inside a partial block when V % 256 != 0)
        t[1, Lr - 1] = 0
        m[1] = 1.0
    return h, w, t, m


CASES = [
    # N, Lr, Dm, V
    (5, 7, 64, 300),        # single partial row tile, partial second vocabulary block
    (40, 8, 256, 2500),     # several row tiles, two panels (the second partial)
    (16, 20, 4096, 1000),   # the real hidden size: 64 k-steps per block
    (3, 50, 136, 4097),     # hidden size not a multiple of 64, vocabulary one past a block
    (300, 1, 128, 512),     # one scored position per candidate
    (24, 16, 512, 32000),   # a Llama-2 sized vocabulary: 16 panels
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
def test_fused_cross_entropy_matches_the_oracle(case):
    N, Lr, Dm, V = case
    h, w, t, m = make(N, Lr, Dm, V, seed=sum(case))
    nll = parity.Guarded((N, Lr), torch.float32, "cuda")
    lse = parity.Guarded((N, Lr), torch.float32, "cuda")
    loss = parity.Guarded((N,), torch.float32, "cuda")
    pskv.pskv_target_ce_fwd(h.cuda(), w.cuda(), t.cuda(), m.cuda(), nll=nll.view, lse=lse.view, loss=loss.view)
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    nll.check("nll"); lse.check("lse"); loss.check("loss")
    rn, rl, rs = oracle.target_ce_fwd(parity.to_f64(h), parity.to_f64(w), t.numpy(), m.numpy().astype(np.float64))
    # fp32 accumulation of exact bf16 products over Dm terms, ex2.approx in the sum: 1e-3 relative is ample
    assert np.max(np.abs(parity.to_f64(lse.view) - rl) / np.maximum(np.abs(rl), 1.0)) <= 1e-3
    assert np.max(np.abs(parity.to_f64(nll.view) - rn) / np.maximum(np.abs(rn), 1.0)) <= 1e-3
    assert np.max(np.abs(parity.to_f64(loss.view) - rs) / np.maximum(np.abs(rs), 1.0)) <= 1e-3
    assert not nll.view[m.cuda() == 0].any()
    assert float(loss.view[0]) == 0.0


@pytest.mark.gpu
def test_full_size_head_on_sampled_candidates():
    """512 candidates x 20 positions against a 4096 x 32000 head (the launch shape of the bench line, with the
    smaller of the two vocabularies so that the fp64 copy of the head fits the host): four candidates, the
    first and last among them, are checked against the oracle; every lse must also be finite and at least
    the largest logit bound ln(V) - |min| cannot beat, i.e. >= the target logit (nll >= 0)."""
    N, Lr, Dm, V = 512, 20, 4096, 32000
    h, w, t, m = make(N, Lr, Dm, V, seed=1234)
    nll, lse, loss = pskv.pskv_target_ce_fwd(h.cuda(), w.cuda(), t.cuda(), m.cuda())
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    assert torch.isfinite(lse).all() and torch.isfinite(nll).all() and (nll >= 0).all()
    cand = [0, 1, 255, 511]
    rn, rl, rs = oracle.target_ce_fwd(parity.to_f64(h[cand]), parity.to_f64(w), t[cand].numpy(),
                                      m[cand].numpy().astype(np.float64))
    assert np.max(np.abs(parity.to_f64(lse[cand]) - rl) / np.maximum(np.abs(rl), 1.0)) <= 1e-3
    assert np.max(np.abs(parity.to_f64(nll[cand]) - rn) / np.maximum(np.abs(rn), 1.0)) <= 1e-3
    assert np.max(np.abs(parity.to_f64(loss[cand]) - rs) / np.maximum(np.abs(rs), 1.0)) <= 1e-3


@pytest.mark.gpu
def test_large_logits_need_the_running_maximum():
    """Hidden states x12: logits of +-40 and more, far outside what exp() without a max can take in the sum."""
    N, Lr, Dm, V = 8, 6, 256, 3000
    h, w, t, m = make(N, Lr, Dm, V, seed=99, gain=12.0)
    nll, lse, loss = pskv.pskv_target_ce_fwd(h.cuda(), w.cuda(), t.cuda(), m.cuda())
    assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
    rn, rl, rs = oracle.target_ce_fwd(parity.to_f64(h), parity.to_f64(w), t.numpy(), m.numpy().astype(np.float64))
    assert np.max(np.abs(rl)) > 30.0
    assert np.max(np.abs(parity.to_f64(lse) - rl) / np.maximum(np.abs(rl), 1.0)) <= 1e-3
    assert np.max(np.abs(parity.to_f64(nll) - rn) / np.maximum(np.abs(rn), 1.0)) <= 1e-3


@pytest.mark.gpu
def test_weighted_bad_token_id_shows_as_nan():
    N, Lr, Dm, V = 2, 4, 64, 100
    h, w, t, m = make(N, Lr, Dm, V, seed=7)
    t[1, 2] = V
    nll, _, loss = pskv.pskv_target_ce_fwd(h.cuda(), w.cuda(), t.cuda(), m.cuda())
    assert torch.isnan(nll[1, 2]) and torch.isnan(loss[1])


def test_target_ce_arguments_are_checked_on_the_host():
    L = pskv.binding.lib()
    fake = ctypes.c_void_p(4096)
    call = lambda N, Lr, Dm, V, ws=1 << 30, hid=fake: L.pskv_target_ce_fwd(hid, fake, fake, fake, fake, fake, fake,
                                                                            N, Lr, Dm, V, fake, ws, None)
    assert call(0, 4, 64, 100) == pskv.PSKV_ERR_INVALID_ARG
    assert call(4, 4, 60, 100) == pskv.PSKV_ERR_UNSUPPORTED_SHAPE      # row pitch not a multiple of 16 bytes
    assert call(4, 4, 64, 100, hid=None) == pskv.PSKV_ERR_INVALID_ARG
    assert call(4, 4, 64, 100, ws=16) == pskv.PSKV_ERR_WORKSPACE
    need = pskv.pskv_target_ce_fwd_workspace_bytes(512, 20, 4096, 128256)
    assert need % 256 == 0 and need >= 2 * 63 * 10240 * 4
    assert pskv.pskv_target_ce_fwd_workspace_bytes(4, 4, 60, 100) == 0
