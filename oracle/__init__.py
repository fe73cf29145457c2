"""ctypes front end of the CPU oracle.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.
It wraps ``packcache_oracle.c`` (plain C, fp64, explicit loops) and does no
arithmetic of its own: arrays are passed through and results handed back as
numpy arrays.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "packcache_oracle.c")
_LIB = os.path.join(_HERE, "libpackcache_oracle.so")

GEOMETRIC, CLOSED_HALF, LINEAR, HALFLIFE = 0, 1, 2, 3
OK, ERR_ARG, ERR_BUDGET, ERR_NAN = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=gnu11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.po_max_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray], t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle error {code}")
        self.code = code


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


def max_threads() -> int:
    return lib().po_max_threads()


def set_threads(n: int) -> None:
    lib().po_set_threads(C.c_int(n))


def rope(x: np.ndarray, pos: Sequence[int], base: float = 10000.0) -> np.ndarray:
    x = _f32(x)
    p = _i32(list(pos)[:3] + [0])
    out = np.empty(x.shape[-1], dtype=np.float64)
    lib().po_rope(_p(x, C.c_float), _p(p, C.c_int32), C.c_int(x.shape[-1]), C.c_double(base), _p(out, C.c_double))
    return out


def plan_budget(kind: int, param: float, total: int, keep_full: int, avail: Sequence[int], min_quota: int = 0) -> np.ndarray:
    avail = _i32(avail)
    out = np.zeros(len(avail), dtype=np.int32)
    _check(lib().po_plan_budget_min(C.c_int(kind), C.c_double(param), C.c_int64(total), C.c_int(keep_full),
                                    C.c_int(min_quota), C.c_int(len(avail)), _p(avail, C.c_int32), _p(out, C.c_int32)))
    return out


def score(k, k_pos, q, q_pos, base=10000.0, valid=None, idx=None) -> np.ndarray:
    k, q, k_pos, q_pos = _f32(k), _f32(q), _i32(k_pos), _i32(q_pos)
    n_src, hkv, d = k.shape
    n_q, hq, _ = q.shape
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.int64)
    n_idx = n_src if idx is None else len(idx)
    if valid is not None:
        valid = np.ascontiguousarray(valid, dtype=np.uint8)
    out = np.empty(n_idx, dtype=np.float64)
    _check(lib().po_score(_p(k, C.c_float), _p(k_pos, C.c_int32), C.c_int64(n_src), _p(q, C.c_float),
                          _p(q_pos, C.c_int32), C.c_int(n_q), C.c_int(hq), C.c_int(hkv), C.c_int(d),
                          C.c_double(base), _p(valid, C.c_uint8), _p(idx, C.c_int64), C.c_int64(n_idx),
                          _p(out, C.c_double)))
    return out


def score_pooled(k, k_pos, q, q_pos, base=10000.0, valid=None) -> np.ndarray:
    k, q, k_pos, q_pos = _f32(k), _f32(q), _i32(k_pos), _i32(q_pos)
    n_src, hkv, d = k.shape
    n_q, hq, _ = q.shape
    if valid is not None:
        valid = np.ascontiguousarray(valid, dtype=np.uint8)
    out = np.empty(n_src, dtype=np.float64)
    _check(lib().po_score_pooled(_p(k, C.c_float), _p(k_pos, C.c_int32), C.c_int64(n_src), _p(q, C.c_float),
                                 _p(q_pos, C.c_int32), C.c_int(n_q), C.c_int(hq), C.c_int(hkv), C.c_int(d),
                                 C.c_double(base), _p(valid, C.c_uint8), _p(out, C.c_double)))
    return out


def select(scores_f32, frame_count, budget) -> np.ndarray:
    s = _f32(scores_f32)
    fc, b = _i32(frame_count), _i32(budget)
    out = np.empty(int(b.sum()), dtype=np.int32)
    _check(lib().po_select(_p(s, C.c_float), C.c_int(len(fc)), _p(fc, C.c_int32), _p(b, C.c_int32),
                           _p(out, C.c_int32)))
    return out


def pack(src_k, src_v, src_pos, sel_idx, delta_t=0):
    src_k, src_v, src_pos, sel = _f32(src_k), _f32(src_v), _i32(src_pos), _i32(sel_idx)
    row = int(np.prod(src_k.shape[1:]))
    n = len(sel)
    dk = np.empty((n,) + src_k.shape[1:], dtype=np.float32)
    dv = np.empty_like(dk)
    dp = np.empty((n, 4), dtype=np.int32)
    lib().po_pack(_p(src_k, C.c_float), _p(src_v, C.c_float), _p(src_pos, C.c_int32), C.c_int(row),
                  _p(sel, C.c_int32), C.c_int64(n), C.c_int32(delta_t), _p(dk, C.c_float), _p(dv, C.c_float),
                  _p(dp, C.c_int32))
    return dk, dv, dp


def attend(q, q_pos, segments, base=10000.0, rows=None, want_lse=False):
    """segments: list of (k, v, pos) in key order (anchors, packed history, current)."""
    q, q_pos = _f32(q), _i32(q_pos)
    n_q, hq, d = q.shape
    segs = [(_f32(k), _f32(v), _i32(p)) for (k, v, p) in segments if len(k)]
    hkv = segs[0][0].shape[1]
    ns = len(segs)
    ka = (C.POINTER(C.c_float) * ns)(*[_p(s[0], C.c_float) for s in segs])
    va = (C.POINTER(C.c_float) * ns)(*[_p(s[1], C.c_float) for s in segs])
    pa = (C.POINTER(C.c_int32) * ns)(*[_p(s[2], C.c_int32) for s in segs])
    na = (C.c_int64 * ns)(*[len(s[0]) for s in segs])
    if rows is not None:
        rows = _i32(rows).reshape(-1, 2)
        n_rows = len(rows)
        out = np.empty((n_rows, d), dtype=np.float64)
    else:
        n_rows = n_q * hq
        out = np.empty((n_q, hq, d), dtype=np.float64)
    lse = np.empty(n_rows, dtype=np.float64)
    _check(lib().po_attend(_p(q, C.c_float), _p(q_pos, C.c_int32), C.c_int(n_q), C.c_int(hq), C.c_int(hkv),
                           C.c_int(d), C.c_double(base), C.c_int(ns), ka, va, pa, na,
                           _p(rows, C.c_int32), C.c_int64(n_rows), _p(out, C.c_double), _p(lse, C.c_double)))
    if rows is None:
        lse = lse.reshape(n_q, hq)
    return (out, lse) if want_lse else out


def attend_mass(q, q_pos, segments, base=10000.0) -> np.ndarray:
    """Mean attention probability every key receives (Sec. 3.4); segments: list of (k, pos) or (k, v, pos)."""
    q, q_pos = _f32(q), _i32(q_pos)
    n_q, hq, d = q.shape
    segs = [(_f32(s[0]), _i32(s[-1])) for s in segments if len(s[0])]
    hkv = segs[0][0].shape[1]
    ns = len(segs)
    ka = (C.POINTER(C.c_float) * ns)(*[_p(s[0], C.c_float) for s in segs])
    pa = (C.POINTER(C.c_int32) * ns)(*[_p(s[1], C.c_int32) for s in segs])
    na = (C.c_int64 * ns)(*[len(s[0]) for s in segs])
    out = np.empty(sum(len(s[0]) for s in segs), dtype=np.float64)
    _check(lib().po_attend_mass(_p(q, C.c_float), _p(q_pos, C.c_int32), C.c_int(n_q), C.c_int(hq), C.c_int(hkv),
                                C.c_int(d), C.c_double(base), C.c_int(ns), ka, pa, na, _p(out, C.c_double)))
    return out


def full_block_causal_attention(q, k, v, pos, block, base=10000.0) -> np.ndarray:
    q, k, v, pos, block = _f32(q), _f32(k), _f32(v), _i32(pos), _i32(block)
    n, hq, d = q.shape
    hkv = k.shape[1]
    out = np.empty((n, hq, d), dtype=np.float64)
    _check(lib().po_full_block_causal_attention(_p(q, C.c_float), _p(k, C.c_float), _p(v, C.c_float),
                                                _p(pos, C.c_int32), _p(block, C.c_int32), C.c_int64(n),
                                                C.c_int(hq), C.c_int(hkv), C.c_int(d), C.c_double(base),
                                                _p(out, C.c_double)))
    return out
