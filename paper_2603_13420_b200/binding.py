"""ctypes binding of libpskv.so: argument marshalling only.

Each function has the name and argument order of its C entry point in
``include/pskv.h``; tensors are torch CUDA tensors whose ``data_ptr()`` is
handed through, sizes are read from the tensors' shapes, and the work is
enqueued on torch's current stream.  Nothing is computed here and there is no
fallback: if the shared library has not been built, loading fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
# PSKV_LIBRARY_PATH selects another build of the same library (e.g. one compiled with tracing).
LIB_PATH = os.environ.get("PSKV_LIBRARY_PATH") or os.path.join(_PKG_DIR, "libpskv.so")

PSKV_OK = 0
PSKV_ERR_INVALID_ARG = 1
PSKV_ERR_UNSUPPORTED_SHAPE = 2
PSKV_ERR_UNSUPPORTED_ARCH = 3
PSKV_ERR_WORKSPACE = 4
PSKV_ERR_CUDA = 5
PSKV_ERR_DEVICE_TIMEOUT = 6

_lib = None


class PskvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        name = lib().pskv_status_string(self.status).decode()
        extra = ""
        if self.status == PSKV_ERR_CUDA:
            extra = " (cudaError %d)" % lib().pskv_last_cuda_error()
        super().__init__("%s: %s%s" % (where, name, extra))


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libpskv.so is missing at %s: build it with `python -m paper_2603_13420_b200.build` "
                "(there is no CPU or PyTorch fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, ci, cf = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_float
        six = [ci] * 6
        L.pskv_attn_fwd_workspace_bytes.argtypes = six
        L.pskv_attn_fwd_workspace_bytes.restype = sz
        L.pskv_attn_bwd_workspace_bytes.argtypes = six
        L.pskv_attn_bwd_workspace_bytes.restype = sz
        L.pskv_attn_fwd.argtypes = [vp] * 5 + [cf] + [vp] * 2 + six + [vp, sz, vp]
        L.pskv_attn_fwd.restype = ci
        L.pskv_attn_bwd.argtypes = [vp] * 8 + [cf] + [vp] * 3 + six + [vp, sz, vp]
        L.pskv_attn_bwd.restype = ci
        L.pskv_attn_bwd_lse.argtypes = [vp] * 9 + [cf] + [vp] * 3 + six + [vp, sz, vp]
        L.pskv_attn_bwd_lse.restype = ci
        L.pskv_attn_bwd_prefix_workspace_bytes.argtypes = six
        L.pskv_attn_bwd_prefix_workspace_bytes.restype = sz
        L.pskv_attn_bwd_prefix.argtypes = [vp] * 7 + [cf] + [vp] * 2 + six + [vp, sz, vp]
        L.pskv_attn_bwd_prefix.restype = ci
        seven = [ci] * 7
        L.pskv_attn_fwd_multi_workspace_bytes.argtypes = seven
        L.pskv_attn_fwd_multi_workspace_bytes.restype = sz
        L.pskv_attn_bwd_multi_workspace_bytes.argtypes = seven
        L.pskv_attn_bwd_multi_workspace_bytes.restype = sz
        L.pskv_attn_fwd_multi.argtypes = [vp] * 6 + [cf] + [vp] * 2 + seven + [vp, sz, vp]
        L.pskv_attn_fwd_multi.restype = ci
        L.pskv_attn_bwd_multi.argtypes = [vp] * 9 + [cf] + [vp] * 3 + seven + [vp, sz, vp]
        L.pskv_attn_bwd_multi.restype = ci
        L.pskv_attn_fwd_decode_workspace_bytes.argtypes = seven
        L.pskv_attn_fwd_decode_workspace_bytes.restype = sz
        L.pskv_attn_bwd_decode_workspace_bytes.argtypes = seven
        L.pskv_attn_bwd_decode_workspace_bytes.restype = sz
        L.pskv_attn_fwd_decode.argtypes = [vp] * 6 + [cf] + [vp] * 2 + seven + [vp, sz, vp]
        L.pskv_attn_fwd_decode.restype = ci
        L.pskv_attn_bwd_decode.argtypes = [vp] * 9 + [cf] + [vp] * 3 + seven + [vp, sz, vp]
        L.pskv_attn_bwd_decode.restype = ci
        L.pskv_target_ce_fwd_workspace_bytes.argtypes = [ci] * 4
        L.pskv_target_ce_fwd_workspace_bytes.restype = sz
        L.pskv_target_ce_fwd.argtypes = [vp] * 7 + [ci] * 4 + [vp, sz, vp]
        L.pskv_target_ce_fwd.restype = ci
        L.pskv_attn_bwd_static.argtypes = [vp] * 8 + [cf] + [vp] * 3 + six + [vp]
        L.pskv_attn_bwd_static.restype = ci
        L.pskv_attn_bwd_static_max_rows.argtypes = []
        L.pskv_attn_bwd_static_max_rows.restype = ctypes.c_longlong
        L.pskv_poll_device_status.argtypes = [vp]
        L.pskv_poll_device_status.restype = ci
        L.pskv_status_string.argtypes = [ci]
        L.pskv_status_string.restype = ctypes.c_char_p
        L.pskv_last_cuda_error.argtypes = []
        L.pskv_last_cuda_error.restype = ci
        L.pskv_version.argtypes = []
        L.pskv_version.restype = ci
        L.pskv_kernel_timing_enable.argtypes = [ci]
        L.pskv_kernel_timing_enable.restype = None
        L.pskv_kernel_timing_count.argtypes = []
        L.pskv_kernel_timing_count.restype = ci
        L.pskv_kernel_timing_name.argtypes = [ci]
        L.pskv_kernel_timing_name.restype = ctypes.c_char_p
        L.pskv_kernel_timing_read.argtypes = [ci, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong)]
        L.pskv_kernel_timing_read.restype = ci
        L.pskv_kernel_launches.argtypes = []
        L.pskv_kernel_launches.restype = ctypes.c_longlong
        L.pskv_kernel_family.argtypes = [ci] + six
        L.pskv_kernel_family.restype = ci
        L.pskv_selftest_wait_timeout.argtypes = [ctypes.c_longlong, vp]
        L.pskv_selftest_wait_timeout.restype = ci
        L.pskv_selftest_per_device_once.argtypes = []
        L.pskv_selftest_per_device_once.restype = ci
        L.pskv_set_multi_form.argtypes = [ci]
        L.pskv_set_multi_form.restype = ci
        L.pskv_enable_cta_pairs.argtypes = [ci]
        L.pskv_enable_cta_pairs.restype = None
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensors must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dims(q, prefix_k, suffix_k):
    B, Hq, S, d = q.shape
    Hkv = suffix_k.shape[1]
    P = 0 if prefix_k is None else prefix_k.shape[1]
    return [int(B), int(Hq), int(Hkv), int(S), int(P), int(d)]


def pskv_version() -> int:
    return int(lib().pskv_version())


def pskv_kernel_timing_enable(on) -> None:
    lib().pskv_kernel_timing_enable(int(bool(on)))


def pskv_kernel_timing_count() -> int:
    return int(lib().pskv_kernel_timing_count())


def pskv_kernel_timing_name(kernel_id) -> str:
    return lib().pskv_kernel_timing_name(int(kernel_id)).decode()


def pskv_kernel_timing_read(kernel_id):
    """(total device milliseconds, launches) of one kernel id since the last read."""
    ms, n = ctypes.c_double(0.0), ctypes.c_longlong(0)
    st = lib().pskv_kernel_timing_read(int(kernel_id), ctypes.byref(ms), ctypes.byref(n))
    if st != PSKV_OK:
        raise PskvError(st, "pskv_kernel_timing_read")
    return ms.value, int(n.value)


def pskv_kernel_launches() -> int:
    return int(lib().pskv_kernel_launches())


def pskv_last_cuda_error() -> int:
    return int(lib().pskv_last_cuda_error())


def pskv_status_string(status: int) -> str:
    return lib().pskv_status_string(int(status)).decode()


def pskv_selftest_wait_timeout(budget_cycles: int = 100000) -> None:
    """Enqueue the tiny kernel whose bounded wait runs out (see include/pskv.h)."""
    st = lib().pskv_selftest_wait_timeout(int(budget_cycles), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_selftest_wait_timeout")


def pskv_selftest_per_device_once() -> int:
    return int(lib().pskv_selftest_per_device_once())


def pskv_set_multi_form(form) -> None:
    """0 / "auto": the library chooses; 1 / "one": one launch for all instructions where the shapes allow
    it; 2 / "passes": one pass per instruction."""
    form = {"auto": 0, "one": 1, "passes": 2}.get(form, form)
    st = lib().pskv_set_multi_form(int(form))
    if st != PSKV_OK:
        raise PskvError(st, "pskv_set_multi_form")


def pskv_enable_cta_pairs(on: bool) -> None:
    lib().pskv_enable_cta_pairs(int(bool(on)))


def pskv_kernel_family(backward, B, Hq, Hkv, S, P, d) -> int:
    return int(lib().pskv_kernel_family(int(bool(backward)), B, Hq, Hkv, S, P, d))


def pskv_attn_fwd_workspace_bytes(B, Hq, Hkv, S, P, d) -> int:
    return int(lib().pskv_attn_fwd_workspace_bytes(B, Hq, Hkv, S, P, d))


def pskv_attn_bwd_workspace_bytes(B, Hq, Hkv, S, P, d) -> int:
    return int(lib().pskv_attn_bwd_workspace_bytes(B, Hq, Hkv, S, P, d))


def _workspace(nbytes, device, workspace):
    if workspace is not None:
        return workspace
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def pskv_attn_fwd(q, prefix_k, prefix_v, suffix_k, suffix_v, scale, out=None, lse=None,
                  workspace=None):
    """out [B,Hq,S,d] bf16 and lse [B,Hq,S] fp32; q/suffix_* are per candidate, prefix_* [Hkv,P,d] shared."""
    dims = _dims(q, prefix_k, suffix_k)
    B, Hq, Hkv, S, P, d = dims
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((B, Hq, S), dtype=torch.float32, device=q.device)
    ws = _workspace(pskv_attn_fwd_workspace_bytes(*dims), q.device, workspace)
    st = lib().pskv_attn_fwd(_ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(suffix_k), _ptr(suffix_v),
                             float(scale), _ptr(out), _ptr(lse), *dims,
                             _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_fwd")
    return out, lse


def pskv_attn_bwd(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, out, lse, scale,
                  dq=None, dk_suffix=None, dv_suffix=None, workspace=None):
    """dq, dk_suffix, dv_suffix (bf16) of L = sum(out * dout); the prefix cache gets no gradient."""
    dims = _dims(q, prefix_k, suffix_k)
    if dq is None:
        dq = torch.empty_like(q)
    if dk_suffix is None:
        dk_suffix = torch.empty_like(suffix_k)
    if dv_suffix is None:
        dv_suffix = torch.empty_like(suffix_v)
    ws = _workspace(pskv_attn_bwd_workspace_bytes(*dims), q.device, workspace)
    st = lib().pskv_attn_bwd(_ptr(dout), _ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(suffix_k),
                             _ptr(suffix_v), _ptr(out), _ptr(lse), float(scale),
                             _ptr(dq), _ptr(dk_suffix), _ptr(dv_suffix), *dims,
                             _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_bwd")
    return dq, dk_suffix, dv_suffix


def pskv_attn_bwd_lse(dout, dlse, q, prefix_k, prefix_v, suffix_k, suffix_v, out, lse, scale,
                      dq=None, dk_suffix=None, dv_suffix=None, workspace=None):
    """Backward of L = sum(out * dout) + sum(lse * dlse): pskv_attn_bwd with a gradient on lse (fp32 [B,Hq,S])."""
    dims = _dims(q, prefix_k, suffix_k)
    if dq is None:
        dq = torch.empty_like(q)
    if dk_suffix is None:
        dk_suffix = torch.empty_like(suffix_k)
    if dv_suffix is None:
        dv_suffix = torch.empty_like(suffix_v)
    if dlse is None or dlse.dtype != torch.float32 or tuple(dlse.shape) != tuple(q.shape[:3]):
        raise ValueError("dlse must be a float32 CUDA tensor of shape [B,Hq,S]")
    ws = _workspace(pskv_attn_bwd_workspace_bytes(*dims), q.device, workspace)
    st = lib().pskv_attn_bwd_lse(_ptr(dout), _ptr(dlse), _ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(suffix_k),
                                 _ptr(suffix_v), _ptr(out), _ptr(lse), float(scale),
                                 _ptr(dq), _ptr(dk_suffix), _ptr(dv_suffix), *dims,
                                 _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_bwd_lse")
    return dq, dk_suffix, dv_suffix


def pskv_attn_bwd_prefix_workspace_bytes(B, Hq, Hkv, S, P, d) -> int:
    return int(lib().pskv_attn_bwd_prefix_workspace_bytes(B, Hq, Hkv, S, P, d))


def pskv_attn_bwd_prefix(dout, dlse, q, prefix_k, prefix_v, out, lse, scale, dk_prefix=None, dv_prefix=None,
                         workspace=None):
    """Gradients of the shared prefix cache, dk_prefix / dv_prefix [Hkv,P,d] (bf16), summed over all
    candidates; dlse (fp32 [B,Hq,S]) may be None."""
    B, Hq, S, d = (int(x) for x in q.shape)
    Hkv, P = int(prefix_k.shape[0]), int(prefix_k.shape[1])
    if dk_prefix is None:
        dk_prefix = torch.empty_like(prefix_k)
    if dv_prefix is None:
        dv_prefix = torch.empty_like(prefix_v)
    ws = _workspace(pskv_attn_bwd_prefix_workspace_bytes(B, Hq, Hkv, S, P, d), q.device, workspace)
    st = lib().pskv_attn_bwd_prefix(_ptr(dout), _ptr(dlse), _ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(out),
                                    _ptr(lse), float(scale), _ptr(dk_prefix), _ptr(dv_prefix), B, Hq, Hkv, S, P, d,
                                    _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_bwd_prefix")
    return dk_prefix, dv_prefix


def _multi_dims(q, prefix_k, suffix_k, prefix_len):
    B, Hq, S, d = q.shape
    Hkv = suffix_k.shape[1]
    Bp = len(prefix_len)
    Pmax = 0 if prefix_k is None else prefix_k.shape[2]
    return [int(B), int(Bp), int(Hq), int(Hkv), int(S), int(Pmax), int(d)]


def _host_lens(prefix_len):
    arr = (ctypes.c_int * len(prefix_len))(*[int(x) for x in prefix_len])
    return arr


def pskv_attn_fwd_multi_workspace_bytes(B, Bp, Hq, Hkv, S, Pmax, d) -> int:
    return int(lib().pskv_attn_fwd_multi_workspace_bytes(B, Bp, Hq, Hkv, S, Pmax, d))


def pskv_attn_bwd_multi_workspace_bytes(B, Bp, Hq, Hkv, S, Pmax, d) -> int:
    return int(lib().pskv_attn_bwd_multi_workspace_bytes(B, Bp, Hq, Hkv, S, Pmax, d))


def pskv_attn_fwd_multi(q, prefix_k, prefix_v, prefix_len, suffix_k, suffix_v, scale, out=None, lse=None,
                        workspace=None):
    """Forward with one left-padded prefix cache per instruction: prefix_k / prefix_v are
    [Bp, Hkv, Pmax, d], prefix_len (host ints) the true lengths, candidate b uses instruction
    b // (B // Bp).  Padding rows may hold any finite values."""
    dims = _multi_dims(q, prefix_k, suffix_k, prefix_len)
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    ws = _workspace(max(256, pskv_attn_fwd_multi_workspace_bytes(*dims)), q.device, workspace)
    lens = _host_lens(prefix_len)
    st = lib().pskv_attn_fwd_multi(_ptr(q), _ptr(prefix_k), _ptr(prefix_v), ctypes.cast(lens, ctypes.c_void_p),
                                   _ptr(suffix_k), _ptr(suffix_v), float(scale), _ptr(out), _ptr(lse), *dims,
                                   _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_fwd_multi")
    return out, lse


def pskv_attn_bwd_multi(dout, q, prefix_k, prefix_v, prefix_len, suffix_k, suffix_v, out, lse, scale,
                        dq=None, dk_suffix=None, dv_suffix=None, workspace=None):
    """Backward of pskv_attn_fwd_multi: dq, dk_suffix, dv_suffix; the prefix caches get no gradient."""
    dims = _multi_dims(q, prefix_k, suffix_k, prefix_len)
    if dq is None:
        dq = torch.empty_like(q)
    if dk_suffix is None:
        dk_suffix = torch.empty_like(suffix_k)
    if dv_suffix is None:
        dv_suffix = torch.empty_like(suffix_v)
    ws = _workspace(pskv_attn_bwd_multi_workspace_bytes(*dims), q.device, workspace)
    lens = _host_lens(prefix_len)
    st = lib().pskv_attn_bwd_multi(_ptr(dout), _ptr(q), _ptr(prefix_k), _ptr(prefix_v),
                                   ctypes.cast(lens, ctypes.c_void_p), _ptr(suffix_k), _ptr(suffix_v), _ptr(out),
                                   _ptr(lse), float(scale), _ptr(dq), _ptr(dk_suffix), _ptr(dv_suffix), *dims,
                                   _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_bwd_multi")
    return dq, dk_suffix, dv_suffix


def _decode_dims(q, prefix_k, suffix_k):
    B, Hq, Sq, d = q.shape
    Hkv, Skv = suffix_k.shape[1], suffix_k.shape[2]
    P = 0 if prefix_k is None else prefix_k.shape[1]
    return [int(B), int(Hq), int(Hkv), int(Sq), int(Skv), int(P), int(d)]


def _len_ptr(suffix_len, B):
    if suffix_len is None:
        return None
    if suffix_len.dtype != torch.int32 or tuple(suffix_len.shape) != (B,):
        raise ValueError("suffix_len must be an int32 CUDA tensor of shape [B]")
    return _ptr(suffix_len)


def pskv_attn_fwd_decode_workspace_bytes(B, Hq, Hkv, Sq, Skv, P, d) -> int:
    return int(lib().pskv_attn_fwd_decode_workspace_bytes(B, Hq, Hkv, Sq, Skv, P, d))


def pskv_attn_bwd_decode_workspace_bytes(B, Hq, Hkv, Sq, Skv, P, d) -> int:
    return int(lib().pskv_attn_bwd_decode_workspace_bytes(B, Hq, Hkv, Sq, Skv, P, d))


def pskv_attn_fwd_decode(q, prefix_k, prefix_v, suffix_k, suffix_v, suffix_len, scale, out=None, lse=None,
                         workspace=None):
    """Decode-shaped forward: q [B,Hq,Sq,d] are the last Sq of each candidate's suffix_len[b] cached
    suffix tokens (suffix_k / suffix_v [B,Hkv,Skv,d]; suffix_len an int32 CUDA tensor [B] or None)."""
    dims = _decode_dims(q, prefix_k, suffix_k)
    if out is None:
        out = torch.empty_like(q)
    if lse is None:
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    ws = _workspace(pskv_attn_fwd_decode_workspace_bytes(*dims), q.device, workspace)
    st = lib().pskv_attn_fwd_decode(_ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(suffix_k), _ptr(suffix_v),
                                    _len_ptr(suffix_len, dims[0]), float(scale), _ptr(out), _ptr(lse), *dims,
                                    _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_fwd_decode")
    return out, lse


def pskv_attn_bwd_decode(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, suffix_len, out, lse, scale,
                         dq=None, dk_suffix=None, dv_suffix=None, workspace=None):
    """Backward of pskv_attn_fwd_decode: dq [B,Hq,Sq,d], dk_suffix / dv_suffix [B,Hkv,Skv,d]."""
    dims = _decode_dims(q, prefix_k, suffix_k)
    if dq is None:
        dq = torch.empty_like(q)
    if dk_suffix is None:
        dk_suffix = torch.empty_like(suffix_k)
    if dv_suffix is None:
        dv_suffix = torch.empty_like(suffix_v)
    ws = _workspace(pskv_attn_bwd_decode_workspace_bytes(*dims), q.device, workspace)
    st = lib().pskv_attn_bwd_decode(_ptr(dout), _ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(suffix_k),
                                    _ptr(suffix_v), _len_ptr(suffix_len, dims[0]), _ptr(out), _ptr(lse),
                                    float(scale), _ptr(dq), _ptr(dk_suffix), _ptr(dv_suffix), *dims,
                                    _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_bwd_decode")
    return dq, dk_suffix, dv_suffix


def pskv_target_ce_fwd_workspace_bytes(N, Lr, Dm, V) -> int:
    return int(lib().pskv_target_ce_fwd_workspace_bytes(N, Lr, Dm, V))


def pskv_target_ce_fwd(hidden, weight, target, mask, nll=None, lse=None, loss=None, workspace=None):
    """Masked target cross-entropy fused with the vocabulary projection: hidden bf16 [N,Lr,Dm], weight
    bf16 [V,Dm], target int32 [N,Lr], mask fp32 [N,Lr].  Returns nll [N,Lr], lse [N,Lr], loss [N] (fp32)."""
    N, Lr, Dm = (int(x) for x in hidden.shape)
    V = int(weight.shape[0])
    if target.dtype != torch.int32 or mask.dtype != torch.float32:
        raise ValueError("target must be int32 and mask float32")
    if tuple(target.shape) != (N, Lr) or tuple(mask.shape) != (N, Lr) or int(weight.shape[1]) != Dm:
        raise ValueError("shape mismatch")
    f32 = dict(dtype=torch.float32, device=hidden.device)
    nll = torch.empty((N, Lr), **f32) if nll is None else nll
    lse = torch.empty((N, Lr), **f32) if lse is None else lse
    loss = torch.empty((N,), **f32) if loss is None else loss
    ws = _workspace(pskv_target_ce_fwd_workspace_bytes(N, Lr, Dm, V), hidden.device, workspace)
    st = lib().pskv_target_ce_fwd(_ptr(hidden), _ptr(weight), _ptr(target), _ptr(mask), _ptr(nll), _ptr(lse),
                                  _ptr(loss), N, Lr, Dm, V, _ptr(ws), ws.numel() * ws.element_size(), _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_target_ce_fwd")
    return nll, lse, loss


def pskv_attn_bwd_static_max_rows() -> int:
    return int(lib().pskv_attn_bwd_static_max_rows())


def pskv_attn_bwd_static(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, out, lse, scale,
                         dq=None, dk_suffix=None, dv_suffix=None):
    """pskv_attn_bwd for callers that cannot allocate device memory (a framework owns the card, or
    a cudaMalloc would stall the device): the scratch is a fixed array inside the library, so no
    workspace is passed.  Serves up to pskv_attn_bwd_static_max_rows() query rows (B*Hq*S); calls
    that overlap on the GPU race on that array, so keep them on one stream.  The gradient tensors
    are still the caller's (pass dq / dk_suffix / dv_suffix to avoid even those allocations)."""
    dims = _dims(q, prefix_k, suffix_k)
    if dq is None:
        dq = torch.empty_like(q)
    if dk_suffix is None:
        dk_suffix = torch.empty_like(suffix_k)
    if dv_suffix is None:
        dv_suffix = torch.empty_like(suffix_v)
    st = lib().pskv_attn_bwd_static(_ptr(dout), _ptr(q), _ptr(prefix_k), _ptr(prefix_v), _ptr(suffix_k),
                                    _ptr(suffix_v), _ptr(out), _ptr(lse), float(scale),
                                    _ptr(dq), _ptr(dk_suffix), _ptr(dv_suffix), *dims, _stream())
    if st != PSKV_OK:
        raise PskvError(st, "pskv_attn_bwd_static")
    return dq, dk_suffix, dv_suffix


def pskv_poll_device_status() -> int:
    """Synchronise the current stream and return the device status (PSKV_OK or an error code)."""
    return int(lib().pskv_poll_device_status(_stream()))
