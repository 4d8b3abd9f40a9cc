"""Forward + backward of one layer for data that lives in pinned HOST memory.

The operator is independent across candidates (only the prefix K/V is shared), so a step whose inputs
and results are host tensors is cut into candidate chunks that flow through a three-stage pipeline: an
upload stream copies chunk c+1 in while a compute stream runs the two library calls of chunk c and a
download stream copies the results of chunk c-1 out, over a small ring of device buffer sets.  Both copy
engines then stay busy for the whole step instead of one long copy in, the kernels, and one long copy
out.  Nothing is computed here: every chunk goes through ``pskv_attn_fwd`` / ``pskv_attn_bwd`` exactly as
a whole batch would, and since rows of different candidates never meet in those kernels, the results
are those of the unchunked calls.
"""
from __future__ import annotations

import torch

from . import binding

_SETS = 4  # device buffer sets in the ring: chunks that can be in flight at once


class HostStep:
    """Reusable plan (streams, events, device buffer sets) for host-resident steps of one shape."""

    def __init__(self, B, Hq, Hkv, S, P, d, scale, device, chunks=8):
        if B < 1 or chunks < 1:
            raise ValueError("B and chunks must be positive")
        self.dims = (B, Hq, Hkv, S, P, d)
        self.scale = float(scale)
        self.device = torch.device(device)
        self.cb = (B + min(chunks, B) - 1) // min(chunks, B)   # candidates per chunk
        cb = self.cb
        self.s_in, self.s_comp, self.s_out = (torch.cuda.Stream(device=self.device) for _ in range(3))
        bf, f32, u8 = torch.bfloat16, torch.float32, torch.uint8
        mk = lambda shape, dt: torch.empty(shape, dtype=dt, device=self.device)
        self.prefix_k = mk((Hkv, P, d), bf) if P > 0 else None
        self.prefix_v = mk((Hkv, P, d), bf) if P > 0 else None
        self.sets = []
        for _ in range(_SETS):
            self.sets.append(dict(
                q=mk((cb, Hq, S, d), bf), dout=mk((cb, Hq, S, d), bf), suffix_k=mk((cb, Hkv, S, d), bf),
                suffix_v=mk((cb, Hkv, S, d), bf), out=mk((cb, Hq, S, d), bf), lse=mk((cb, Hq, S), f32),
                dq=mk((cb, Hq, S, d), bf), dk=mk((cb, Hkv, S, d), bf), dv=mk((cb, Hkv, S, d), bf),
                ws_f=mk((max(binding.pskv_attn_fwd_workspace_bytes(cb, Hq, Hkv, S, P, d), 256),), u8),
                ws_b=mk((max(binding.pskv_attn_bwd_workspace_bytes(cb, Hq, Hkv, S, P, d), 256),), u8),
                in_done=torch.cuda.Event(), comp_done=torch.cuda.Event(), out_done=torch.cuda.Event()))
        self.start = torch.cuda.Event()
        self.done = torch.cuda.Event()

    def run(self, host_in, host_out):
        """host_in: pinned q, dout [B,Hq,S,d], suffix_k, suffix_v [B,Hkv,S,d], prefix_k, prefix_v
        [Hkv,P,d]; host_out: pinned out, dq [B,Hq,S,d], lse [B,Hq,S], dk, dv [B,Hkv,S,d].  Enqueues the
        whole step; the caller's current stream waits for it, the host does not."""
        B, P = self.dims[0], self.dims[4]
        cur = torch.cuda.current_stream(self.device)
        self.start.record(cur)             # orders this step behind earlier work of the caller
        for st in (self.s_in, self.s_comp, self.s_out):
            st.wait_event(self.start)
        with torch.cuda.stream(self.s_in):
            if P > 0:
                self.prefix_k.copy_(host_in["prefix_k"], non_blocking=True)
                self.prefix_v.copy_(host_in["prefix_v"], non_blocking=True)
        c = 0
        for b0 in range(0, B, self.cb):
            n = min(self.cb, B - b0)
            bufs = self.sets[c % _SETS]
            sl = slice(b0, b0 + n)
            d = {k: bufs[k][:n] for k in ("q", "dout", "suffix_k", "suffix_v", "out", "lse", "dq", "dk", "dv")}
            with torch.cuda.stream(self.s_in):
                if c >= _SETS:
                    self.s_in.wait_event(bufs["comp_done"])   # the set's previous chunk has been computed
                for k in ("q", "suffix_k", "suffix_v", "dout"):
                    d[k].copy_(host_in[k][sl], non_blocking=True)
                bufs["in_done"].record(self.s_in)
            with torch.cuda.stream(self.s_comp):
                self.s_comp.wait_event(bufs["in_done"])
                if c >= _SETS:
                    self.s_comp.wait_event(bufs["out_done"])  # ... and its results have been copied out
                binding.pskv_attn_fwd(d["q"], self.prefix_k, self.prefix_v, d["suffix_k"], d["suffix_v"], self.scale,
                                      out=d["out"], lse=d["lse"], workspace=bufs["ws_f"])
                binding.pskv_attn_bwd(d["dout"], d["q"], self.prefix_k, self.prefix_v, d["suffix_k"], d["suffix_v"],
                                      d["out"], d["lse"], self.scale, dq=d["dq"], dk_suffix=d["dk"],
                                      dv_suffix=d["dv"], workspace=bufs["ws_b"])
                bufs["comp_done"].record(self.s_comp)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(bufs["comp_done"])
                for k in ("out", "lse", "dq", "dk", "dv"):
                    host_out[k][sl].copy_(d[k], non_blocking=True)
                bufs["out_done"].record(self.s_out)
            c += 1
        self.done.record(self.s_out)       # the download stream finishes last: it waits for every chunk
        cur.wait_event(self.done)
