"""ctypes binding of ``libpackcache.so`` — same names as the C ABI, argument marshalling only.

Every step of the path (scoring, selection, packing, rotary embedding, attention) runs in the library's CUDA
kernels; PyTorch is used here for device memory and streams.  There is no CPU fallback: if the library cannot be
loaded, importing callers get an error.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

PC_OK, PC_ERR_INVALID_ARG, PC_ERR_BUDGET, PC_ERR_CAPACITY, PC_ERR_UNSUPPORTED, PC_ERR_CUDA, PC_ERR_TIMEOUT = range(7)
PC_F32, PC_BF16 = 0, 1
PC_GEOMETRIC, PC_CLOSED_HALF, PC_LINEAR, PC_HALFLIFE = 0, 1, 2, 3
PC_MAX_FRAMES = 256

EXPORTS = ["pc_create", "pc_destroy", "pc_plan_budget", "pc_score", "pc_compact", "pc_attend_frame",
           "pc_poll_status", "pc_set_attend_impl", "pc_set_kv_splits", "pc_set_timing", "pc_get_timing",
           "pc_frame_step_host", "pc_status_string", "pc_score_tokens_static", "pc_set_cluster_merge",
           "pc_window_create", "pc_window_destroy", "pc_window_append", "pc_window_append_masked", "pc_window_update", "pc_window_cache",
           "pc_window_state", "pc_attend_prepare", "pc_attend_prepared", "pc_attend_mass", "pc_frame_step",
           "pc_forget_anchors", "pc_set_wait_limit_us", "pc_test_expect_extra_bytes", "pc_window_step", "pc_window_step_host", "pc_set_timing_skip",
           "pc_get_span", "pc_probe_stream_read", "pc_probe_mma_rate"]


class pc_layer_desc(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32),
                ("rope_base", C.c_double), ("max_pos", C.c_int32 * 3), ("max_q", C.c_int32), ("max_keys", C.c_int32)]


class pc_segment(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("pos", C.c_void_p), ("n_tokens", C.c_int32),
                ("capacity", C.c_int32)]


class pc_cache(C.Structure):
    _fields_ = [("anchors", pc_segment), ("history", pc_segment), ("n_frames", C.c_int32),
                ("frame_count", C.POINTER(C.c_int32))]


class pc_budget_params(C.Structure):
    _fields_ = [("kind", C.c_int32), ("param", C.c_double), ("total", C.c_int64), ("keep_full", C.c_int32),
                ("min_quota", C.c_int32)]


class pc_window_params(C.Structure):
    _fields_ = [("window", C.c_int32), ("budget", pc_budget_params), ("rebase", C.c_int32), ("t_step", C.c_int32)]


class pc_host_frame(C.Structure):
    _fields_ = [("q", C.c_void_p), ("q_pos", C.c_void_p), ("n_q", C.c_int32), ("anchor_k", C.c_void_p),
                ("anchor_v", C.c_void_p), ("anchor_pos", C.c_void_p), ("n_anchor", C.c_int32), ("hist_k", C.c_void_p),
                ("hist_v", C.c_void_p), ("hist_pos", C.c_void_p), ("n_frames", C.c_int32),
                ("frame_count", C.POINTER(C.c_int32)), ("out", C.c_void_p)]


class pc_host_window_step(C.Structure):
    _fields_ = [("frame_k", C.c_void_p), ("frame_v", C.c_void_p), ("frame_pos", C.c_void_p), ("n_frame", C.c_int32),
                ("q", C.c_void_p), ("q_pos", C.c_void_p), ("n_q", C.c_int32), ("out", C.c_void_p)]


class pc_window_step_workspace(C.Structure):
    _fields_ = [("q", C.c_void_p), ("q_pos", C.c_void_p), ("out", C.c_void_p)]


class pc_device_workspace(C.Structure):
    _fields_ = [("src", pc_cache), ("dst", pc_cache), ("q", C.c_void_p), ("q_pos", C.c_void_p), ("scores", C.c_void_p),
                ("sel_idx", C.c_void_p), ("out", C.c_void_p)]


STAGES = ["qpool", "score", "select", "pack", "rope", "attend", "combine", "mass"]


class PackCacheError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = _lib.pc_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{what}: {msg} (pc_status {status})")


_lib = None


def load() -> C.CDLL:
    """Load the CUDA library (building it with nvcc if the .so is absent).  Raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()
    lib = C.CDLL(path)
    lib.pc_status_string.restype = C.c_char_p
    lib.pc_status_string.argtypes = [C.c_int]
    lib.pc_create.argtypes = [C.POINTER(pc_layer_desc), C.POINTER(C.c_void_p)]
    lib.pc_destroy.argtypes = [C.c_void_p]
    lib.pc_plan_budget.argtypes = [C.POINTER(pc_budget_params), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.pc_score.argtypes = [C.c_void_p, C.POINTER(pc_cache), C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int32),
                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.pc_compact.argtypes = [C.c_void_p, C.POINTER(pc_cache), C.c_void_p, C.POINTER(C.c_int32), C.c_int32,
                               C.POINTER(pc_cache), C.c_void_p]
    lib.pc_attend_frame.argtypes = [C.c_void_p, C.POINTER(pc_cache), C.POINTER(pc_segment), C.c_void_p, C.c_void_p,
                                    C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.pc_poll_status.argtypes = [C.c_void_p, C.c_void_p]
    lib.pc_set_attend_impl.argtypes = [C.c_void_p, C.c_int32]
    lib.pc_set_kv_splits.argtypes = [C.c_void_p, C.c_int32]
    lib.pc_set_cluster_merge.argtypes = [C.c_void_p, C.c_int32]
    lib.pc_set_timing.argtypes = [C.c_void_p, C.c_int32]
    lib.pc_get_timing.argtypes = [C.c_void_p, C.POINTER(C.c_float)]
    lib.pc_set_timing_skip.argtypes = [C.c_void_p, C.c_uint32]
    lib.pc_get_span.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_float)]
    lib.pc_probe_stream_read.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.pc_probe_mma_rate.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.pc_frame_step_host.argtypes = [C.c_void_p, C.POINTER(pc_host_frame), C.POINTER(pc_device_workspace),
                                       C.POINTER(pc_budget_params), C.c_int32, C.c_void_p]
    lib.pc_score_tokens_static.argtypes = [C.POINTER(pc_layer_desc), C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                           C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.pc_attend_prepare.argtypes = [C.c_void_p, C.POINTER(pc_cache), C.POINTER(pc_segment), C.c_void_p]
    lib.pc_attend_prepared.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.pc_attend_mass.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
    lib.pc_frame_step.argtypes = [C.c_void_p, C.POINTER(pc_cache), C.POINTER(C.c_int32), C.c_int32, C.POINTER(pc_cache),
                                  C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.pc_forget_anchors.argtypes = [C.c_void_p]
    lib.pc_set_wait_limit_us.argtypes = [C.c_void_p, C.c_uint32]
    lib.pc_test_expect_extra_bytes.argtypes = [C.c_void_p, C.c_uint32]
    lib.pc_window_create.argtypes = [C.c_void_p, C.POINTER(pc_window_params), C.POINTER(pc_segment), C.POINTER(pc_segment),
                                     C.POINTER(pc_segment), C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p)]
    lib.pc_window_destroy.argtypes = [C.c_void_p]
    lib.pc_window_append.argtypes = [C.c_void_p, C.POINTER(pc_segment), C.c_void_p]
    lib.pc_window_append_masked.argtypes = [C.c_void_p, C.POINTER(pc_segment), C.c_void_p, C.c_int32, C.c_void_p]
    lib.pc_window_update.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(C.c_int32), C.c_void_p]
    lib.pc_window_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_int32),
                                   C.c_void_p]
    lib.pc_window_step_host.argtypes = [C.c_void_p, C.POINTER(pc_host_window_step), C.POINTER(pc_window_step_workspace),
                                        C.POINTER(C.c_int32), C.c_void_p]
    lib.pc_window_cache.argtypes = [C.c_void_p, C.POINTER(pc_cache)]
    lib.pc_window_state.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int64),
                                    C.POINTER(C.c_int32)]
    _lib = lib
    return lib


def _check(status: int, what: str) -> None:
    if status != PC_OK:
        raise PackCacheError(status, what)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _i32p(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


@dataclass
class Segment:
    """A run of tokens on the device: K/V [capacity][Hkv][d], pos [capacity][4] int32."""
    k: Optional[torch.Tensor]
    v: Optional[torch.Tensor]
    pos: Optional[torch.Tensor]
    n_tokens: int

    @staticmethod
    def empty() -> "Segment":
        return Segment(None, None, None, 0)

    @property
    def capacity(self) -> int:
        return 0 if self.k is None else self.k.shape[0]

    def c(self) -> pc_segment:
        return pc_segment(_ptr(self.k), _ptr(self.v), _ptr(self.pos), self.n_tokens, self.capacity)


@dataclass
class Cache:
    """Anchors held apart from the history frames (oldest -> newest); frame_count lives on the host."""
    anchors: Segment
    history: Segment
    frame_count: np.ndarray

    def c(self) -> pc_cache:
        self._fc = _i32(self.frame_count)            # keep alive for the duration of the call
        return pc_cache(self.anchors.c(), self.history.c(), len(self._fc), _i32p(self._fc))


class Context:
    """Owns a pc_ctx (rotary tables, status word, scratch) on the current CUDA device."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int, rope_base: float,
                 max_pos: Sequence[int], max_q: int, max_keys: int):
        lib = load()
        self.desc = pc_layer_desc(n_q_heads, n_kv_heads, head_dim, dtype, rope_base, (C.c_int32 * 3)(*max_pos),
                                  max_q, max_keys)
        self.torch_dtype = torch.bfloat16 if dtype == PC_BF16 else torch.float32
        h = C.c_void_p()
        _check(lib.pc_create(C.byref(self.desc), C.byref(h)), "pc_create")
        self.handle = h

    def close(self) -> None:
        if getattr(self, "handle", None):
            load().pc_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pc_plan_budget(kind: int, param: float, total: int, keep_full: int, avail: Sequence[int],
                   min_quota: int = 0) -> np.ndarray:
    avail = _i32(avail)
    out = np.zeros(len(avail), dtype=np.int32)
    p = pc_budget_params(kind, param, total, keep_full, min_quota)
    _check(load().pc_plan_budget(C.byref(p), len(avail), _i32p(avail), _i32p(out)), "pc_plan_budget")
    return out


def pc_score(ctx: Context, src: Cache, q: Optional[torch.Tensor], q_pos: Optional[torch.Tensor], budget,
             valid: Optional[torch.Tensor] = None, scores_override: Optional[torch.Tensor] = None,
             scores: Optional[torch.Tensor] = None, sel_idx: Optional[torch.Tensor] = None, stream=None):
    """Returns (scores [n_src] fp32, sel_idx [sum(budget)] int32), both on the device."""
    budget = _i32(budget)
    dev = src.history.k.device if src.history.k is not None else torch.device("cuda")
    if scores is None and scores_override is None:
        scores = torch.empty(max(src.history.n_tokens, 1), dtype=torch.float32, device=dev)
    if sel_idx is None:
        sel_idx = torch.empty(max(int(budget.sum()), 1), dtype=torch.int32, device=dev)
    n_q = 0 if q is None else q.shape[0]
    c = src.c()
    _check(load().pc_score(ctx.handle, C.byref(c), _ptr(q), _ptr(q_pos), n_q, _i32p(budget), _ptr(valid),
                           _ptr(scores_override), _ptr(scores), _ptr(sel_idx), _stream(stream)), "pc_score")
    return scores, sel_idx


def pc_compact(ctx: Context, src: Cache, sel_idx: torch.Tensor, budget, delta_t: int, dst: Cache, stream=None) -> None:
    budget = _i32(budget)
    cs, cd = src.c(), dst.c()
    _check(load().pc_compact(ctx.handle, C.byref(cs), _ptr(sel_idx), _i32p(budget), delta_t, C.byref(cd),
                             _stream(stream)), "pc_compact")
    dst.history.n_tokens = int(budget.sum())
    dst.frame_count = budget.copy()


def pc_attend_frame(ctx: Context, cache: Cache, current: Optional[Segment], q: torch.Tensor, q_pos: torch.Tensor,
                    out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None, want_lse: bool = False,
                    stream=None):
    if out is None:
        out = torch.empty_like(q)
    if lse is None and want_lse:
        lse = torch.empty(q.shape[0], q.shape[1], dtype=torch.float32, device=q.device)
    c = cache.c()
    cur = current.c() if current is not None else None
    _check(load().pc_attend_frame(ctx.handle, C.byref(c), C.byref(cur) if cur is not None else None, _ptr(q),
                                  _ptr(q_pos), q.shape[0], _ptr(out), _ptr(lse), _stream(stream)), "pc_attend_frame")
    return (out, lse) if want_lse else out


def pc_frame_step(ctx: Context, src: Cache, budget, delta_t: int, dst: Cache, q: torch.Tensor, q_pos: torch.Tensor,
                  scores: Optional[torch.Tensor] = None, sel_idx: Optional[torch.Tensor] = None,
                  out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None, want_lse: bool = False, stream=None):
    """score -> select -> pack -> attend in one call; returns (out, scores, sel_idx[, lse]); dst receives the packed rows."""
    budget = _i32(budget)
    if scores is None:
        scores = torch.empty(max(src.history.n_tokens, 1), dtype=torch.float32, device=q.device)
    if sel_idx is None:
        sel_idx = torch.empty(max(int(budget.sum()), 1), dtype=torch.int32, device=q.device)
    if out is None:
        out = torch.empty_like(q)
    if lse is None and want_lse:
        lse = torch.empty(q.shape[0], q.shape[1], dtype=torch.float32, device=q.device)
    cs, cd = src.c(), dst.c()
    _check(load().pc_frame_step(ctx.handle, C.byref(cs), _i32p(budget), delta_t, C.byref(cd), _ptr(q), _ptr(q_pos), q.shape[0],
                                _ptr(scores), _ptr(sel_idx), _ptr(out), _ptr(lse), _stream(stream)), "pc_frame_step")
    dst.history.n_tokens = int(budget.sum())
    dst.frame_count = budget.copy()
    return (out, scores, sel_idx, lse) if want_lse else (out, scores, sel_idx)


def pc_forget_anchors(ctx: Context) -> None:
    _check(load().pc_forget_anchors(ctx.handle), "pc_forget_anchors")


def pc_set_wait_limit_us(ctx: Context, limit_us: int) -> None:
    _check(load().pc_set_wait_limit_us(ctx.handle, limit_us), "pc_set_wait_limit_us")


def pc_test_expect_extra_bytes(ctx: Context, n_bytes: int) -> None:
    _check(load().pc_test_expect_extra_bytes(ctx.handle, n_bytes), "pc_test_expect_extra_bytes")


def pc_attend_prepare(ctx: Context, cache: Cache, current: Optional[Segment] = None, stream=None) -> None:
    c = cache.c()
    cur = current.c() if current is not None else None
    _check(load().pc_attend_prepare(ctx.handle, C.byref(c), C.byref(cur) if cur is not None else None, _stream(stream)),
           "pc_attend_prepare")


def pc_attend_prepared(ctx: Context, q: torch.Tensor, q_pos: torch.Tensor, out: Optional[torch.Tensor] = None,
                       lse: Optional[torch.Tensor] = None, want_lse: bool = False, stream=None):
    if out is None:
        out = torch.empty_like(q)
    if lse is None and want_lse:
        lse = torch.empty(q.shape[0], q.shape[1], dtype=torch.float32, device=q.device)
    _check(load().pc_attend_prepared(ctx.handle, _ptr(q), _ptr(q_pos), q.shape[0], _ptr(out), _ptr(lse), _stream(stream)),
           "pc_attend_prepared")
    return (out, lse) if want_lse else out


def pc_attend_mass(ctx: Context, lse: torch.Tensor, n_keys: int, mass: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Attention mass of every key of the most recent attention call on ctx (lse = what that call wrote)."""
    if mass is None:
        mass = torch.empty(n_keys, dtype=torch.float32, device=lse.device)
    _check(load().pc_attend_mass(ctx.handle, _ptr(lse), _ptr(mass), n_keys, _stream(stream)), "pc_attend_mass")
    return mass


def pc_poll_status(ctx: Context, stream=None) -> int:
    return load().pc_poll_status(ctx.handle, _stream(stream))


def pc_set_attend_impl(ctx: Context, impl: int) -> None:
    _check(load().pc_set_attend_impl(ctx.handle, impl), "pc_set_attend_impl")


def pc_set_kv_splits(ctx: Context, n: int) -> None:
    _check(load().pc_set_kv_splits(ctx.handle, n), "pc_set_kv_splits")


def pc_set_cluster_merge(ctx: Context, on: bool) -> None:
    _check(load().pc_set_cluster_merge(ctx.handle, 1 if on else 0), "pc_set_cluster_merge")


def pc_set_timing(ctx: Context, on: bool) -> None:
    _check(load().pc_set_timing(ctx.handle, 1 if on else 0), "pc_set_timing")


def pc_get_timing(ctx: Context) -> dict:
    """Milliseconds of each kernel of the most recent calls (see STAGES); -1 for a kernel that did not run."""
    ms = (C.c_float * len(STAGES))()
    _check(load().pc_get_timing(ctx.handle, ms), "pc_get_timing")
    return {name: float(ms[i]) for i, name in enumerate(STAGES)}


MARKS = {"SCORE0": 0, "QPOOL": 1, "SCORE": 2, "SELECT": 3, "PACK0": 4, "PACK": 5, "ATT0": 6, "ROPE": 7, "ATTEND": 8,
         "COMBINE": 9, "MASS0": 10, "MASS": 11}


def pc_set_timing_skip(ctx: Context, marks: Sequence[str]) -> None:
    """Leave out the named event marks (see MARKS) from now on."""
    mask = 0
    for m in marks:
        mask |= 1 << MARKS[m]
    _check(load().pc_set_timing_skip(ctx.handle, mask), "pc_set_timing_skip")


def pc_get_span(ctx: Context, a: str, b: str) -> float:
    """Milliseconds between two recorded marks of the most recent calls, -1 if either is missing."""
    ms = C.c_float(-1.0)
    _check(load().pc_get_span(ctx.handle, MARKS[a], MARKS[b], C.byref(ms)), "pc_get_span")
    return float(ms.value)


def pc_probe_stream_read(rows: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """Stream the rows of a [n][...] tensor from device memory (one 32-bit word out per row): a bandwidth yardstick."""
    n = rows.shape[0]
    row_bytes = rows[0].numel() * rows.element_size()
    _check(load().pc_probe_stream_read(_ptr(rows), n, row_bytes, _ptr(out), _stream(stream)), "pc_probe_stream_read")


MMA_FORMS = {"qk": (0, 16), "pv": (1, 16), "mix": (2, 32)}   # form id, multiply-adds per round


def pc_probe_mma_rate(ctx: Context, form: str, rounds: int = 2000, n_cta: int | None = None, stream=None):
    """The attention kernel's tensor-core issue stream alone (form "qk", "pv" or "mix").  Returns (cycles per multiply-add,
    SM clock in GHz), each the median over the CTAs (one per SM unless n_cta says otherwise).  Synchronises."""
    fid, per_round = MMA_FORMS[form]
    if n_cta is None:
        n_cta = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    cycles = torch.zeros(n_cta, dtype=torch.int64, device="cuda")
    nanos = torch.zeros(n_cta, dtype=torch.int64, device="cuda")
    _check(load().pc_probe_mma_rate(ctx.handle, fid, rounds, n_cta, _ptr(cycles), _ptr(nanos), _stream(stream)), "pc_probe_mma_rate")
    torch.cuda.synchronize()
    c, n = cycles.double(), nanos.double().clamp(min=1.0)
    return float((c / (rounds * per_round)).median()), float((c / n).median())


def pc_frame_step_host(ctx: Context, host: dict, ws_src: Cache, ws_dst: Cache, ws: dict, kind: int, param: float,
                       total: int, keep_full: int, delta_t: int = 0, stream=None) -> None:
    """host: pinned CPU tensors q, q_pos, anchor_k, anchor_v, anchor_pos, hist_k, hist_v, hist_pos, out and the numpy
    frame_count; ws: device tensors q, q_pos, scores, sel_idx, out.  Blocks until the output is in host['out']."""
    fc = _i32(host["frame_count"])
    hf = pc_host_frame(_ptr(host["q"]), _ptr(host["q_pos"]), host["q"].shape[0], _ptr(host["anchor_k"]),
                       _ptr(host["anchor_v"]), _ptr(host["anchor_pos"]), host["anchor_k"].shape[0],
                       _ptr(host["hist_k"]), _ptr(host["hist_v"]), _ptr(host["hist_pos"]), len(fc), _i32p(fc),
                       _ptr(host["out"]))
    w = pc_device_workspace(ws_src.c(), ws_dst.c(), _ptr(ws["q"]), _ptr(ws["q_pos"]), _ptr(ws["scores"]),
                            _ptr(ws["sel_idx"]), _ptr(ws["out"]))
    p = pc_budget_params(kind, param, total, keep_full, 0)
    _check(load().pc_frame_step_host(ctx.handle, C.byref(hf), C.byref(w), C.byref(p), delta_t, _stream(stream)),
           "pc_frame_step_host")


def pc_score_tokens_static(desc: pc_layer_desc, hist_k: torch.Tensor, hist_pos: torch.Tensor, n_src: int,
                           q: torch.Tensor, q_pos: torch.Tensor, scores: torch.Tensor, status: torch.Tensor,
                           valid: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Context-free scoring that allocates nothing: every buffer, including the [n_src] fp32 ``scores`` output and the
    zeroed [2] int32 ``status`` word, is the caller's; the library's scratch is a fixed device array."""
    _check(load().pc_score_tokens_static(C.byref(desc), _ptr(hist_k), _ptr(hist_pos), n_src, _ptr(q), _ptr(q_pos),
                                         q.shape[0], _ptr(valid), _ptr(scores), _ptr(status), _stream(stream)),
           "pc_score_tokens_static")
    return scores


PC_WINDOW_FILL, PC_WINDOW_PACK, PC_WINDOW_SLIDE = 0, 1, 2


class Window:
    """The Fill / Pack / Slide cache window over two caller-owned history buffers (Segments with capacity; their n_tokens
    is managed by the library).  Argument marshalling only: plan, score, select, pack run in the library."""

    def __init__(self, ctx: Context, window: int, kind: int, param: float, total: int, keep_full: int, anchors: Segment,
                 hist_a: Segment, hist_b: Segment, rebase: bool = False, t_step: int = 4, min_quota: int = 0):
        self.ctx, self.anchors, self.bufs = ctx, anchors, (hist_a, hist_b)
        cap = min(hist_a.capacity, hist_b.capacity)
        dev = hist_a.k.device
        self.scores = torch.empty(cap, dtype=torch.float32, device=dev)
        self.sel_idx = torch.empty(cap, dtype=torch.int32, device=dev)
        self.window = window
        p = pc_window_params(window, pc_budget_params(kind, param, total, keep_full, min_quota), 1 if rebase else 0, t_step)
        a, ha, hb = anchors.c(), hist_a.c(), hist_b.c()
        h = C.c_void_p()
        _check(load().pc_window_create(ctx.handle, C.byref(p), C.byref(a), C.byref(ha), C.byref(hb), _ptr(self.scores),
                                       _ptr(self.sel_idx), C.byref(h)), "pc_window_create")
        self.handle = h

    def append(self, frame: Segment, stream=None) -> None:
        f = frame.c()
        _check(load().pc_window_append(self.handle, C.byref(f), _stream(stream)), "pc_window_append")

    def append_masked(self, frame: Segment, valid: torch.Tensor, n_valid: int, stream=None) -> None:
        f = frame.c()
        _check(load().pc_window_append_masked(self.handle, C.byref(f), _ptr(valid), n_valid, _stream(stream)),
               "pc_window_append_masked")

    def update(self, q: Optional[torch.Tensor], q_pos: Optional[torch.Tensor], scores_override: Optional[torch.Tensor] = None,
               stream=None) -> int:
        regime = C.c_int32(-1)
        _check(load().pc_window_update(self.handle, _ptr(q), _ptr(q_pos), 0 if q is None else q.shape[0],
                                       _ptr(scores_override), C.byref(regime), _stream(stream)), "pc_window_update")
        return regime.value

    def step(self, q: torch.Tensor, q_pos: torch.Tensor, out: Optional[torch.Tensor] = None,
             lse: Optional[torch.Tensor] = None, stream=None):
        """Update and attention in one call; returns (regime, out)."""
        if out is None:
            out = torch.empty_like(q)
        regime = C.c_int32(-1)
        _check(load().pc_window_step(self.handle, _ptr(q), _ptr(q_pos), q.shape[0], _ptr(out), _ptr(lse), C.byref(regime),
                                     _stream(stream)), "pc_window_step")
        return regime.value, out

    def step_host(self, frame: Optional[dict], q: torch.Tensor, q_pos: torch.Tensor, out: torch.Tensor, ws: dict,
                  stream=None) -> int:
        """frame: pinned CPU tensors k, v, pos of the frame to append (or None); q, q_pos, out: pinned CPU tensors;
        ws: device tensors q, q_pos, out.  Blocks until ``out`` holds the result; returns the regime."""
        n = 0 if frame is None else frame["k"].shape[0]
        h = pc_host_window_step(_ptr(frame["k"]) if n else None, _ptr(frame["v"]) if n else None,
                                _ptr(frame["pos"]) if n else None, n, _ptr(q), _ptr(q_pos), q.shape[0], _ptr(out))
        wsp = pc_window_step_workspace(_ptr(ws["q"]), _ptr(ws["q_pos"]), _ptr(ws["out"]))
        regime = C.c_int32(-1)
        _check(load().pc_window_step_host(self.handle, C.byref(h), C.byref(wsp), C.byref(regime), _stream(stream)),
               "pc_window_step_host")
        return regime.value

    def state(self):
        """(token counts oldest -> newest, accumulated temporal shift, index of the active buffer)"""
        n, shift, active = C.c_int32(), C.c_int64(), C.c_int32()
        counts = (C.c_int32 * (self.window + 1))()
        _check(load().pc_window_state(self.handle, C.byref(n), counts, C.byref(shift), C.byref(active)), "pc_window_state")
        return np.array(counts[:n.value], dtype=np.int32), int(shift.value), int(active.value)

    def cache(self) -> Cache:
        counts, _, active = self.state()
        b = self.bufs[active]
        return Cache(self.anchors, Segment(b.k, b.v, b.pos, int(counts.sum())), counts)

    def close(self) -> None:
        if getattr(self, "handle", None):
            load().pc_window_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
