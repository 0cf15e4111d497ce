"""ctypes front end of the fp64 CPU oracle (``hg_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg may import this module; the
product package never does, and this module never imports the product.  Arrays are numpy;
16-bit inputs are passed as raw ``uint16`` bit patterns which the C code decodes itself.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hg_oracle.c")
_SO = os.path.join(_HERE, "libhg_oracle.so")
_lock = threading.Lock()
_lib = None

F16, BF16 = 0, 1
DTYPES = {"f16": F16, "bf16": BF16}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no optimisation flags that change fp semantics)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


_p = C.c_void_p
_i64 = C.c_int64
_int = C.c_int
_dbl = C.c_double


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            L.hgo_decode_f16.restype = _dbl
            L.hgo_decode_f16.argtypes = [C.c_uint16]
            L.hgo_decode_bf16.restype = _dbl
            L.hgo_decode_bf16.argtypes = [C.c_uint16]
            L.hgo_decode.argtypes = [_p, _i64, _int, _p]
            L.hgo_logits.argtypes = [_p, _p, _i64, _int, _int, _dbl, _p, _i64, _i64, _p]
            L.hgo_partial.argtypes = [_p, _p, _p, _i64, _int, _int, _dbl, _p, _i64, _i64, _p, _p, _p]
            L.hgo_partial_from_logits.argtypes = [_p, _p, _i64, _int, _int, _i64, _p, _p, _p]
            L.hgo_partial_from_logits.restype = None
            L.hgo_full.argtypes = [_p, _p, _p, _i64, _int, _int, _dbl, _p, _i64, _i64, _p, _p]
            L.hgo_merge.argtypes = [_i64, _p, _p, _p, _int, _p, _p]
            L.hgo_literal.argtypes = [_p, _p, _p, _i64, _int, _int, _dbl, _p, _i64, _p, _i64, _p, _p]
            L.hgo_chunked_partials.argtypes = [_p, _p, _p, _int, _int, _int, _int, _int, _i64, _dbl, _p, _p,
                                               _i64, _i64, _p, _p, _p, _int]
            L.hgo_full_batch.argtypes = [_p, _p, _p, _int, _int, _int, _int, _int, _i64, _dbl, _p, _p, _p, _p, _int]
            for f in ("hgo_decode", "hgo_logits", "hgo_partial", "hgo_full", "hgo_merge", "hgo_literal",
                      "hgo_chunked_partials", "hgo_full_batch"):
                getattr(L, f).restype = None
            _lib = L
    return _lib


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _idx(idx):
    if idx is None:
        return None, None
    a = np.ascontiguousarray(idx, dtype=np.int64)
    return a, a.ctypes.data


def _ptr(a):
    return a.ctypes.data


def host_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def decode(bits, dtype: str) -> np.ndarray:
    b = _u16(bits)
    out = np.empty(b.shape, dtype=np.float64)
    lib().hgo_decode(_ptr(b), b.size, DTYPES[dtype], _ptr(out))
    return out


def _rows(K):
    """K given as [n_tokens][D] (or any row-major array whose rows are tokens) -> (array, tok_stride)."""
    K = _u16(K)
    assert K.ndim == 2
    return K, K.shape[1]


def logits(q, K, dtype: str, scale: float = 0.0, idx=None, t0: int = 0, n: int | None = None) -> np.ndarray:
    q = _u16(q); K, ts = _rows(K)
    ia, ip = _idx(idx)
    n = (len(ia) if ia is not None else (K.shape[0] - t0 if n is None else n))
    s = np.empty(n, dtype=np.float64)
    lib().hgo_logits(_ptr(q), _ptr(K), ts, q.shape[-1], DTYPES[dtype], scale, ip, t0, n, _ptr(s))
    return s


def partial(q, K, V, dtype: str, scale: float = 0.0, idx=None, t0: int = 0, n: int | None = None):
    """PARTIAL over tokens idx (or [t0, t0+n)) of row arrays K, V [tokens][D] -> (m, l, o[D])."""
    q = _u16(q); K, ts = _rows(K); V, _ = _rows(V)
    ia, ip = _idx(idx)
    n = (len(ia) if ia is not None else (K.shape[0] - t0 if n is None else n))
    D = q.shape[-1]
    m, l, o = _dbl(), _dbl(), np.empty(D, dtype=np.float64)
    lib().hgo_partial(_ptr(q), _ptr(K), _ptr(V), ts, D, DTYPES[dtype], scale, ip, t0, n, C.byref(m), C.byref(l), _ptr(o))
    return m.value, l.value, o


def partial_from_logits(s, Vsel, dtype: str):
    """PARTIAL from n given logits s[n] (fp64) and the matching V rows Vsel [n][D] -> (m, l, o[D])."""
    s = np.ascontiguousarray(s, dtype=np.float64)
    Vsel, rs = _rows(Vsel)
    D = Vsel.shape[1]
    m, l, o = _dbl(), _dbl(), np.empty(D, dtype=np.float64)
    lib().hgo_partial_from_logits(_ptr(s), _ptr(Vsel), rs, D, DTYPES[dtype], len(s), C.byref(m), C.byref(l), _ptr(o))
    return m.value, l.value, o


def full(q, K, V, dtype: str, scale: float = 0.0, idx=None, t0: int = 0, n: int | None = None):
    """FULL over tokens idx (or [t0, t0+n)) -> (out[D], lse)."""
    q = _u16(q); K, ts = _rows(K); V, _ = _rows(V)
    ia, ip = _idx(idx)
    n = (len(ia) if ia is not None else (K.shape[0] - t0 if n is None else n))
    D = q.shape[-1]
    out, lse = np.empty(D, dtype=np.float64), _dbl()
    lib().hgo_full(_ptr(q), _ptr(K), _ptr(V), ts, D, DTYPES[dtype], scale, ip, t0, n, _ptr(out), C.byref(lse))
    return out, lse.value


def merge(m, l, o):
    """MERGE of n sources: m[n], l[n], o[n][D] -> (out[D], lse)."""
    m = np.ascontiguousarray(m, dtype=np.float64); l = np.ascontiguousarray(l, dtype=np.float64)
    o = np.ascontiguousarray(o, dtype=np.float64)
    n, D = o.shape
    out, lse = np.empty(D, dtype=np.float64), _dbl()
    lib().hgo_merge(n, _ptr(m), _ptr(l), _ptr(o), D, _ptr(out), C.byref(lse))
    return out, lse.value


def literal(q, K, V, dtype: str, idx_a, idx_b, scale: float = 0.0):
    """The paper's hand-off: logits from two devices concatenated in token order, one softmax."""
    q = _u16(q); K, ts = _rows(K); V, _ = _rows(V)
    a, ap = _idx(np.asarray(idx_a, dtype=np.int64)); b, bp = _idx(np.asarray(idx_b, dtype=np.int64))
    D = q.shape[-1]
    out, lse = np.empty(D, dtype=np.float64), _dbl()
    lib().hgo_literal(_ptr(q), _ptr(K), _ptr(V), ts, D, DTYPES[dtype], scale, ap, len(a), bp, len(b), _ptr(out), C.byref(lse))
    return out, lse.value


def chunked_partials(q, K, V, dtype: str, lo, hi, chunk: int, NC: int, scale: float = 0.0, threads: int = 0):
    """PARTIAL per (b, h, chunk) over a logical cache K, V [B][Lmax][Hkv][D]; q [B][Hq][D].

    Chunk c of sequence b is [(lo_b // chunk + c) * chunk, +chunk) clipped to [lo_b, hi_b); chunk = 0
    means one piece per sequence.  Returns m, l [B][Hq][NC] and o [B][Hq][NC][D].
    """
    q = _u16(q); K = _u16(K); V = _u16(V)
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = K.shape
    lo = np.ascontiguousarray(lo, dtype=np.int64); hi = np.ascontiguousarray(hi, dtype=np.int64)
    m = np.empty((B, Hq, NC)); l = np.empty((B, Hq, NC)); o = np.empty((B, Hq, NC, D))
    lib().hgo_chunked_partials(_ptr(q), _ptr(K), _ptr(V), B, Hq, Hkv, D, DTYPES[dtype], Lmax, scale,
                               _ptr(lo), _ptr(hi), chunk, NC, _ptr(m), _ptr(l), _ptr(o), threads or host_threads())
    return m, l, o


def full_batch(q, K, V, dtype: str, lo, hi, scale: float = 0.0, threads: int = 0):
    """FULL over [lo_b, hi_b) for every (b, h) -> out [B][Hq][D], lse [B][Hq]."""
    q = _u16(q); K = _u16(K); V = _u16(V)
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = K.shape
    lo = np.ascontiguousarray(lo, dtype=np.int64); hi = np.ascontiguousarray(hi, dtype=np.int64)
    out = np.empty((B, Hq, D)); lse = np.empty((B, Hq))
    lib().hgo_full_batch(_ptr(q), _ptr(K), _ptr(V), B, Hq, Hkv, D, DTYPES[dtype], Lmax, scale,
                         _ptr(lo), _ptr(hi), _ptr(out), _ptr(lse), threads or host_threads())
    return out, lse


def merge_batch(m, l, o):
    """MERGE along the source axis: m, l [..., n], o [..., n, D] -> out [..., D], lse [...]."""
    m = np.asarray(m, dtype=np.float64); l = np.asarray(l, dtype=np.float64); o = np.asarray(o, dtype=np.float64)
    lead = m.shape[:-1]
    n, D = o.shape[-2:]
    m2 = m.reshape(-1, n); l2 = l.reshape(-1, n); o2 = o.reshape(-1, n, D)
    out = np.empty((m2.shape[0], D)); lse = np.empty(m2.shape[0])
    for i in range(m2.shape[0]):
        out[i], lse[i] = merge(m2[i], l2[i], o2[i])
    return out.reshape(*lead, D), lse.reshape(lead)
