"""pskv_attn_bwd_static: the backward entry point for callers that cannot allocate device memory
(for instance because a framework's allocator owns the whole card, or because a cudaMalloc would
stall every stream of a latency-bound loop).  Its scratch is a fixed array inside the library, so
it takes no workspace.  Called through the C ABI twice in a row, it must give what pskv_attn_bwd
gives with a caller-provided workspace.  This file sorts last on purpose: a run that stops at the
first failure has then already run every other test."""
import dataclasses

import pytest
import torch

import paper_2603_13420_b200 as pskv
from paper_2603_13420_b200.inputs import WORKLOADS, make_inputs

import parity

pytestmark = pytest.mark.gpu


def _gradients(w):
    t = make_inputs(w, with_dout=True)
    d = {k: v.cuda() for k, v in t.items()}
    out, lse = pskv.pskv_attn_fwd(d["q"], d["prefix_k"], d["prefix_v"], d["suffix_k"], d["suffix_v"], w.scale)
    args = (d["dout"], d["q"], d["prefix_k"], d["prefix_v"], d["suffix_k"], d["suffix_v"], out, lse, w.scale)
    ref = pskv.pskv_attn_bwd(*args)
    return args, ref


@pytest.mark.parametrize("name,B", [("C4", 6), ("C2", 3), ("C0", 8)])
def test_static_scratch_backward_matches_workspace_backward_twice(name, B):
    w = dataclasses.replace(WORKLOADS[name], B=B, backward=True)
    assert w.B * w.Hq * w.S <= pskv.pskv_attn_bwd_static_max_rows()
    args, ref = _gradients(w)
    for call in range(2):  # the second call finds the first call's values in the shared array
        # outputs pre-filled with NaN: every element must be written by the call
        outs = [torch.full_like(r, float("nan")) for r in ref]
        got = pskv.pskv_attn_bwd_static(*args, dq=outs[0], dk_suffix=outs[1], dv_suffix=outs[2])
        assert pskv.pskv_poll_device_status() == pskv.PSKV_OK
        for label, g, r in zip(("dq", "dk_suffix", "dv_suffix"), got, ref):
            parity.check_tensor("%s (call %d)" % (label, call), parity.to_f64(g), parity.to_f64(r))
            assert torch.equal(g, r), label  # same kernels, same inputs: bit-identical in fact


def test_sizes_beyond_the_built_in_scratch_are_refused():
    rows_max = pskv.pskv_attn_bwd_static_max_rows()
    w = dataclasses.replace(WORKLOADS["C0"], B=8)
    args, ref = _gradients(w)
    # pretend the batch is larger than the scratch can serve: only the sizes are inspected
    lib = pskv.binding.lib()
    import ctypes
    vp = ctypes.c_void_p
    ptrs = [vp(a.data_ptr()) for a in args[:8]]
    outs = [vp(r.data_ptr()) for r in ref]
    big_B = rows_max // (w.Hq * w.S) + 1
    rc = lib.pskv_attn_bwd_static(*ptrs, w.scale, *outs, big_B, w.Hq, w.Hkv, w.S, w.P, w.d, None)
    assert rc == pskv.PSKV_ERR_WORKSPACE
