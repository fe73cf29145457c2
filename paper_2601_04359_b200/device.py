"""Device-side plumbing shared by the tests, the smoke check and the benchmark: move a seeded workload into GPU
memory (PyTorch tensors) and wrap it in the binding's Segment / Cache records.  No arithmetic of the method here."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as pc
from . import workload as wl


def dev(x: np.ndarray, dtype: str) -> torch.Tensor:
    """float32 host array (already rounded to the storage type) -> device tensor of that type."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16).contiguous() if dtype == wl.BF16 else t.contiguous()


def idev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def make_ctx(cfg: wl.Config, max_keys: int = 0, max_q: int = 0, max_pos=None) -> pc.Context:
    n_keys = cfg.n_anchor + cfg.n_src + cfg.n_q
    return pc.Context(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                      pc.PC_BF16 if cfg.dtype == wl.BF16 else pc.PC_F32, cfg.rope_base,
                      max_pos or cfg.max_pos, max_q or cfg.n_q, max_keys or n_keys)


def segment(k: np.ndarray, v: np.ndarray, pos: np.ndarray, dtype: str, capacity: int = 0) -> pc.Segment:
    n = len(k)
    if capacity > n:
        pad = lambda a: np.concatenate([a, np.zeros((capacity - n,) + a.shape[1:], a.dtype)])
        k, v, pos = pad(k), pad(v), pad(pos)
    return pc.Segment(dev(k, dtype), dev(v, dtype), idev(pos), n)


class DeviceLayer:
    """A workload layer resident on the GPU."""

    def __init__(self, L: wl.Layer):
        cfg = L.cfg
        self.L, self.cfg = L, cfg
        self.q, self.q_pos = dev(L.q, cfg.dtype), idev(L.q_pos)
        self.cache = pc.Cache(segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype),
                              segment(L.hist_k, L.hist_v, L.hist_pos, cfg.dtype), L.frame_count.copy())
        self.current = segment(L.cur_k, L.cur_v, L.q_pos, cfg.dtype) if L.cur_k is not None else None

    def empty_packed(self, capacity: int, poison: float = 0.0) -> pc.Cache:
        cfg = self.cfg
        td = torch.bfloat16 if cfg.dtype == wl.BF16 else torch.float32
        shape = (max(capacity, 1), cfg.n_kv_heads, cfg.head_dim)
        k = torch.full(shape, poison, dtype=td, device="cuda")
        v = torch.full(shape, poison, dtype=td, device="cuda")
        p = torch.full((max(capacity, 1), 4), -7, dtype=torch.int32, device="cuda")
        return pc.Cache(self.cache.anchors, pc.Segment(k, v, p, 0), np.zeros(cfg.n_frames, np.int32))


def score_tolerance(ref: np.ndarray, frame_count) -> np.ndarray:
    """Per-token bound 1e-4 * max(|s|, rms of the token's frame) for fp32 scores."""
    tol = np.empty_like(ref)
    base = 0
    for n in frame_count:
        fr = ref[base:base + n]
        finite = fr[np.isfinite(fr)]
        rms = np.sqrt(np.mean(finite ** 2)) if len(finite) else 0.0
        tol[base:base + n] = 1e-4 * np.maximum(np.abs(np.where(np.isfinite(fr), fr, 0.0)), rms)
        base += n
    return tol
