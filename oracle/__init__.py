"""fp64 CPU oracle for shared-prefix batched causal attention (ctypes wrapper).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the CPU-baseline leg of
the benchmark may import this package; the product path never does, and this
package imports nothing from the CUDA package.

``attn_fwd`` / ``attn_bwd`` take numpy arrays of any float dtype, widen them
to fp64 and call the plain-C program in ``pskv_oracle.c`` (paper Eq. 2 over
the per-candidate duplicated prefix cache of Eq. 3).  Inputs that are meant
to be bf16 must already hold bf16-representable values; the oracle does not
round anything.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pskv_oracle.c")
_LIB = os.path.join(_HERE, "libpskv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile pskv_oracle.c with gcc (OpenMP) into libpskv_oracle.so."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        ints = [ctypes.c_int] * 6
        lib.pskv_oracle_attn_fwd.argtypes = [dp] * 5 + [ctypes.c_double] + [dp] * 2 + ints
        lib.pskv_oracle_attn_fwd.restype = ctypes.c_int
        lib.pskv_oracle_attn_bwd.argtypes = [dp] * 6 + [ctypes.c_double] + [dp] * 3 + ints
        lib.pskv_oracle_attn_bwd.restype = ctypes.c_int
        lib.pskv_oracle_attn_bwd_lse.argtypes = [dp] * 7 + [ctypes.c_double] + [dp] * 3 + ints
        lib.pskv_oracle_attn_bwd_lse.restype = ctypes.c_int
        lib.pskv_oracle_attn_bwd_prefix.argtypes = [dp] * 7 + [ctypes.c_double] + [dp] * 2 + ints
        lib.pskv_oracle_attn_bwd_prefix.restype = ctypes.c_int
        ip = ctypes.POINTER(ctypes.c_int)
        ints7 = [ctypes.c_int] * 7
        lib.pskv_oracle_attn_fwd_multi.argtypes = [dp] * 3 + [ip] + [dp] * 2 + [ctypes.c_double] + [dp] * 2 + ints7
        lib.pskv_oracle_attn_fwd_multi.restype = ctypes.c_int
        lib.pskv_oracle_attn_bwd_multi.argtypes = [dp] * 4 + [ip] + [dp] * 2 + [ctypes.c_double] + [dp] * 3 + ints7
        lib.pskv_oracle_attn_bwd_multi.restype = ctypes.c_int
        lib.pskv_oracle_attn_fwd_decode.argtypes = [dp] * 5 + [ip] + [ctypes.c_double] + [dp] * 2 + ints7
        lib.pskv_oracle_attn_fwd_decode.restype = ctypes.c_int
        lib.pskv_oracle_attn_bwd_decode.argtypes = [dp] * 6 + [ip] + [ctypes.c_double] + [dp] * 3 + ints7
        lib.pskv_oracle_attn_bwd_decode.restype = ctypes.c_int
        lib.pskv_oracle_target_ce_fwd.argtypes = [dp, dp, ip, dp, dp, dp, dp] + [ctypes.c_int] * 4
        lib.pskv_oracle_target_ce_fwd.restype = ctypes.c_int
        lib.pskv_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the C program uses (OpenMP max threads)."""
    return int(_load().pskv_oracle_num_threads())


def _f64(a, shape):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if a.shape != tuple(shape):
        raise ValueError("expected shape %s, got %s" % (tuple(shape), a.shape))
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _dims(q, prefix_k, suffix_k):
    q = np.asarray(q)
    B, Hq, S, d = q.shape
    Hkv, P = np.asarray(prefix_k).shape[:2]
    return B, Hq, Hkv, S, P, d


def attn_fwd(q, prefix_k, prefix_v, suffix_k, suffix_v, scale):
    """out [B,Hq,S,d] and lse [B,Hq,S] (fp64) per Eq. 2 with the duplicated cache of Eq. 3."""
    B, Hq, Hkv, S, P, d = _dims(q, prefix_k, suffix_k)
    q = _f64(q, (B, Hq, S, d))
    pk = _f64(prefix_k, (Hkv, P, d))
    pv = _f64(prefix_v, (Hkv, P, d))
    sk = _f64(suffix_k, (B, Hkv, S, d))
    sv = _f64(suffix_v, (B, Hkv, S, d))
    out = np.empty((B, Hq, S, d), dtype=np.float64)
    lse = np.empty((B, Hq, S), dtype=np.float64)
    rc = _load().pskv_oracle_attn_fwd(_ptr(q), _ptr(pk), _ptr(pv), _ptr(sk), _ptr(sv),
                                      float(scale), _ptr(out), _ptr(lse), B, Hq, Hkv, S, P, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_fwd failed with code %d" % rc)
    return out, lse


def attn_bwd(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, scale):
    """dq, dk_suffix, dv_suffix (fp64) of L = sum(out * dout); prefix K/V frozen."""
    B, Hq, Hkv, S, P, d = _dims(q, prefix_k, suffix_k)
    do = _f64(dout, (B, Hq, S, d))
    q = _f64(q, (B, Hq, S, d))
    pk = _f64(prefix_k, (Hkv, P, d))
    pv = _f64(prefix_v, (Hkv, P, d))
    sk = _f64(suffix_k, (B, Hkv, S, d))
    sv = _f64(suffix_v, (B, Hkv, S, d))
    dq = np.empty((B, Hq, S, d), dtype=np.float64)
    dk = np.empty((B, Hkv, S, d), dtype=np.float64)
    dv = np.empty((B, Hkv, S, d), dtype=np.float64)
    rc = _load().pskv_oracle_attn_bwd(_ptr(do), _ptr(q), _ptr(pk), _ptr(pv), _ptr(sk), _ptr(sv),
                                      float(scale), _ptr(dq), _ptr(dk), _ptr(dv),
                                      B, Hq, Hkv, S, P, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_bwd failed with code %d" % rc)
    return dq, dk, dv


def attn_bwd_lse(dout, dlse, q, prefix_k, prefix_v, suffix_k, suffix_v, scale):
    """dq, dk_suffix, dv_suffix (fp64) of L = sum(out * dout) + sum(lse * dlse); prefix K/V frozen."""
    B, Hq, Hkv, S, P, d = _dims(q, prefix_k, suffix_k)
    do = _f64(dout, (B, Hq, S, d))
    dl = _f64(dlse, (B, Hq, S))
    q = _f64(q, (B, Hq, S, d))
    pk = _f64(prefix_k, (Hkv, P, d))
    pv = _f64(prefix_v, (Hkv, P, d))
    sk = _f64(suffix_k, (B, Hkv, S, d))
    sv = _f64(suffix_v, (B, Hkv, S, d))
    dq = np.empty((B, Hq, S, d), dtype=np.float64)
    dk = np.empty((B, Hkv, S, d), dtype=np.float64)
    dv = np.empty((B, Hkv, S, d), dtype=np.float64)
    rc = _load().pskv_oracle_attn_bwd_lse(_ptr(do), _ptr(dl), _ptr(q), _ptr(pk), _ptr(pv), _ptr(sk), _ptr(sv),
                                          float(scale), _ptr(dq), _ptr(dk), _ptr(dv), B, Hq, Hkv, S, P, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_bwd_lse failed with code %d" % rc)
    return dq, dk, dv


def attn_bwd_prefix(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, scale, dlse=None):
    """dk_prefix, dv_prefix [Hkv,P,d] (fp64) of L = sum(out * dout) (+ sum(lse * dlse)): the gradients of the
    shared prefix cache, summed over all candidates."""
    B, Hq, Hkv, S, P, d = _dims(q, prefix_k, suffix_k)
    do = _f64(dout, (B, Hq, S, d))
    q = _f64(q, (B, Hq, S, d))
    pk = _f64(prefix_k, (Hkv, P, d))
    pv = _f64(prefix_v, (Hkv, P, d))
    sk = _f64(suffix_k, (B, Hkv, S, d))
    sv = _f64(suffix_v, (B, Hkv, S, d))
    dl = None if dlse is None else _f64(dlse, (B, Hq, S))
    dk = np.empty((Hkv, P, d), dtype=np.float64)
    dv = np.empty((Hkv, P, d), dtype=np.float64)
    rc = _load().pskv_oracle_attn_bwd_prefix(_ptr(do), None if dl is None else _ptr(dl), _ptr(q), _ptr(pk), _ptr(pv),
                                             _ptr(sk), _ptr(sv), float(scale), _ptr(dk), _ptr(dv), B, Hq, Hkv, S, P, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_bwd_prefix failed with code %d" % rc)
    return dk, dv


def _mask_i32(mask, Bp, Pmax):
    m = np.ascontiguousarray(np.asarray(mask, dtype=np.int32))
    if m.shape != (Bp, Pmax):
        raise ValueError("expected mask shape %s, got %s" % ((Bp, Pmax), m.shape))
    return m


def left_padding_mask(prefix_len, Pmax):
    """Prefix attention mask of left-padded prefixes: 1 on the last prefix_len[i] positions."""
    lens = np.asarray(prefix_len, dtype=np.int64)
    return (np.arange(Pmax)[None, :] >= (Pmax - lens)[:, None]).astype(np.int32)


def attn_fwd_multi(q, prefix_k, prefix_v, mask, suffix_k, suffix_v, scale):
    """Batched multi-instruction forward (Sec. 4.3): prefix_k / prefix_v [Bp,Hkv,Pmax,d], mask
    [Bp,Pmax] (1 = real prefix token), candidate b uses instruction b // (B // Bp)."""
    q = np.asarray(q)
    B, Hq, S, d = q.shape
    Bp, Hkv, Pmax = np.asarray(prefix_k).shape[:3]
    q = _f64(q, (B, Hq, S, d))
    pk = _f64(prefix_k, (Bp, Hkv, Pmax, d))
    pv = _f64(prefix_v, (Bp, Hkv, Pmax, d))
    sk = _f64(suffix_k, (B, Hkv, S, d))
    sv = _f64(suffix_v, (B, Hkv, S, d))
    m = _mask_i32(mask, Bp, Pmax)
    out = np.empty((B, Hq, S, d), dtype=np.float64)
    lse = np.empty((B, Hq, S), dtype=np.float64)
    rc = _load().pskv_oracle_attn_fwd_multi(_ptr(q), _ptr(pk), _ptr(pv), m.ctypes.data_as(ctypes.POINTER(ctypes.c_int)),
                                            _ptr(sk), _ptr(sv), float(scale), _ptr(out), _ptr(lse),
                                            B, Bp, Hq, Hkv, S, Pmax, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_fwd_multi failed with code %d" % rc)
    return out, lse


def attn_bwd_multi(dout, q, prefix_k, prefix_v, mask, suffix_k, suffix_v, scale):
    """dq, dk_suffix, dv_suffix (fp64) of the multi-instruction forward; prefix caches frozen."""
    q = np.asarray(q)
    B, Hq, S, d = q.shape
    Bp, Hkv, Pmax = np.asarray(prefix_k).shape[:3]
    do = _f64(dout, (B, Hq, S, d))
    q = _f64(q, (B, Hq, S, d))
    pk = _f64(prefix_k, (Bp, Hkv, Pmax, d))
    pv = _f64(prefix_v, (Bp, Hkv, Pmax, d))
    sk = _f64(suffix_k, (B, Hkv, S, d))
    sv = _f64(suffix_v, (B, Hkv, S, d))
    m = _mask_i32(mask, Bp, Pmax)
    dq = np.empty((B, Hq, S, d), dtype=np.float64)
    dk = np.empty((B, Hkv, S, d), dtype=np.float64)
    dv = np.empty((B, Hkv, S, d), dtype=np.float64)
    rc = _load().pskv_oracle_attn_bwd_multi(_ptr(do), _ptr(q), _ptr(pk), _ptr(pv),
                                            m.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), _ptr(sk), _ptr(sv),
                                            float(scale), _ptr(dq), _ptr(dk), _ptr(dv), B, Bp, Hq, Hkv, S, Pmax, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_bwd_multi failed with code %d" % rc)
    return dq, dk, dv


def _len_i32(suffix_len, B):
    if suffix_len is None:
        return None, None
    a = np.ascontiguousarray(np.asarray(suffix_len, dtype=np.int32))
    if a.shape != (B,):
        raise ValueError("expected suffix_len shape %s, got %s" % ((B,), a.shape))
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int))


def attn_fwd_decode(q, prefix_k, prefix_v, suffix_k, suffix_v, scale, suffix_len=None):
    """Decode-shaped forward: q [B,Hq,Sq,d] are the LAST Sq of each candidate's suffix_len[b]
    cached suffix tokens (suffix_k / suffix_v [B,Hkv,Skv,d], rows past suffix_len[b] ignored;
    None = all Skv rows real).  Returns out [B,Hq,Sq,d], lse [B,Hq,Sq]."""
    q = np.asarray(q)
    B, Hq, Sq, d = q.shape
    Hkv, P = np.asarray(prefix_k).shape[:2]
    Skv = np.asarray(suffix_k).shape[2]
    q = _f64(q, (B, Hq, Sq, d))
    pk = _f64(prefix_k, (Hkv, P, d))
    pv = _f64(prefix_v, (Hkv, P, d))
    sk = _f64(suffix_k, (B, Hkv, Skv, d))
    sv = _f64(suffix_v, (B, Hkv, Skv, d))
    keep, lp = _len_i32(suffix_len, B)
    out = np.empty((B, Hq, Sq, d), dtype=np.float64)
    lse = np.empty((B, Hq, Sq), dtype=np.float64)
    rc = _load().pskv_oracle_attn_fwd_decode(_ptr(q), _ptr(pk), _ptr(pv), _ptr(sk), _ptr(sv), lp, float(scale),
                                             _ptr(out), _ptr(lse), B, Hq, Hkv, Sq, Skv, P, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_fwd_decode failed with code %d" % rc)
    return out, lse


def attn_bwd_decode(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, scale, suffix_len=None):
    """dq [B,Hq,Sq,d], dk_suffix, dv_suffix [B,Hkv,Skv,d] (fp64) of the decode-shaped forward;
    rows past suffix_len[b] of the key-side gradients are zero; prefix K/V frozen."""
    q = np.asarray(q)
    B, Hq, Sq, d = q.shape
    Hkv, P = np.asarray(prefix_k).shape[:2]
    Skv = np.asarray(suffix_k).shape[2]
    do = _f64(dout, (B, Hq, Sq, d))
    q = _f64(q, (B, Hq, Sq, d))
    pk = _f64(prefix_k, (Hkv, P, d))
    pv = _f64(prefix_v, (Hkv, P, d))
    sk = _f64(suffix_k, (B, Hkv, Skv, d))
    sv = _f64(suffix_v, (B, Hkv, Skv, d))
    keep, lp = _len_i32(suffix_len, B)
    dq = np.empty((B, Hq, Sq, d), dtype=np.float64)
    dk = np.empty((B, Hkv, Skv, d), dtype=np.float64)
    dv = np.empty((B, Hkv, Skv, d), dtype=np.float64)
    rc = _load().pskv_oracle_attn_bwd_decode(_ptr(do), _ptr(q), _ptr(pk), _ptr(pv), _ptr(sk), _ptr(sv), lp,
                                             float(scale), _ptr(dq), _ptr(dk), _ptr(dv), B, Hq, Hkv, Sq, Skv, P, d)
    if rc != 0:
        raise RuntimeError("pskv_oracle_attn_bwd_decode failed with code %d" % rc)
    return dq, dk, dv


def target_ce_fwd(hidden, weight, target, mask):
    """Masked target cross-entropy on top of the vocabulary projection: hidden [N,Lr,Dm], weight [V,Dm],
    target [N,Lr] ints, mask [N,Lr] loss weights.  Returns nll [N,Lr], lse [N,Lr], loss [N] (fp64)."""
    hidden = np.asarray(hidden)
    N, Lr, Dm = hidden.shape
    V = np.asarray(weight).shape[0]
    h = _f64(hidden, (N, Lr, Dm))
    w = _f64(weight, (V, Dm))
    t = np.ascontiguousarray(np.asarray(target, dtype=np.int32))
    if t.shape != (N, Lr):
        raise ValueError("expected target shape %s, got %s" % ((N, Lr), t.shape))
    m = _f64(mask, (N, Lr))
    nll = np.empty((N, Lr), dtype=np.float64)
    lse = np.empty((N, Lr), dtype=np.float64)
    loss = np.empty((N,), dtype=np.float64)
    rc = _load().pskv_oracle_target_ce_fwd(_ptr(h), _ptr(w), t.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), _ptr(m),
                                           _ptr(nll), _ptr(lse), _ptr(loss), N, Lr, Dm, V)
    if rc != 0:
        raise RuntimeError("pskv_oracle_target_ce_fwd failed with code %d" % rc)
    return nll, lse, loss
