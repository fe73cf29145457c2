"""Reference state machine of the cache window.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

The Fill / Pack / Slide regimes of the paper's Sec. 3.4 (Fig. 6) and the temporal rebase of Eq. 9, written as plain
Python over the oracle's own primitives (plan_budget, score_pooled, select, pack); it imports nothing from the CUDA
package.  Reading taken where the paper is silent: frames are appended whole while they fit both the window W and the
token budget; otherwise frames beyond W leave first (first in, first out), the retained frames get quotas from the
decay kernel over their *current* token counts, each keeps its best-scoring tokens (re-selection from what the last
pack kept plus what was appended since), and with rebase the temporal coordinate of every retained token falls by
t_step per dropped frame while (h, w, tag) stay as they are.  Frames that the plan leaves with nothing at the old end of
the window (the minimum quota b_min starves the oldest frames first when the budget cannot serve every frame) leave the
window like frames beyond W: first in, first out, counted in the rebase.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np

import oracle

FILL, PACK, SLIDE = 0, 1, 2


class WindowRef:
    def __init__(self, window: int, kind: int, param: float, total: int, keep_full: int, rebase: bool = False,
                 t_step: int = 4, rope_base: float = 10000.0, min_quota: int = 0):
        self.window, self.kind, self.param, self.total, self.keep_full = window, kind, param, total, keep_full
        self.min_quota = min_quota
        self.rebase, self.t_step, self.rope_base = rebase, t_step, rope_base
        self.k: Optional[np.ndarray] = None        # [tokens][Hkv][d], frames oldest -> newest
        self.v: Optional[np.ndarray] = None
        self.pos: Optional[np.ndarray] = None      # [tokens][4]
        self.count: List[int] = []
        self.t_shift = 0

    def append(self, k: np.ndarray, v: np.ndarray, pos: np.ndarray, valid: Optional[np.ndarray] = None) -> None:
        if valid is not None:                      # cache mask (Eq. 1): masked positions are removed, not stored
            keep = np.asarray(valid) != 0
            k, v, pos = k[keep], v[keep], pos[keep]
        cat = lambda a, b: b.copy() if a is None else np.concatenate([a, b], axis=0)
        self.k, self.v, self.pos = cat(self.k, k), cat(self.v, v), cat(self.pos, pos)
        self.count.append(len(k))

    def source_after_drop(self):
        """(K, V, pos, counts, dropped frames) of what a pack would select from right now."""
        drop = max(0, len(self.count) - self.window)
        first = int(np.sum(self.count[:drop]))
        return self.k[first:], self.v[first:], self.pos[first:], list(self.count[drop:]), drop

    def update(self, q: np.ndarray, q_pos: np.ndarray, scores32: Optional[np.ndarray] = None) -> int:
        k, v, pos, counts, drop = self.source_after_drop()
        if drop == 0 and int(np.sum(counts)) <= self.total:
            return FILL
        budget = oracle.plan_budget(self.kind, self.param, self.total, self.keep_full, counts, self.min_quota)
        lead = 0                                   # frames at the old end that the plan leaves with nothing: they leave too
        while lead < len(budget) and budget[lead] == 0:
            lead += 1
        if lead:
            first = int(np.sum(counts[:lead]))
            k, v, pos, counts, budget, drop = k[first:], v[first:], pos[first:], counts[lead:], budget[lead:], drop + lead
            if scores32 is not None:
                scores32 = scores32[first:]
        if scores32 is None:
            scores32 = oracle.score_pooled(k, pos, q, q_pos, self.rope_base).astype(np.float32) if len(k) else np.zeros(0, np.float32)
        sel = oracle.select(scores32, counts, budget)
        delta = drop * self.t_step if self.rebase else 0
        self.k, self.v, self.pos = oracle.pack(k, v, pos, sel, delta)
        self.count = [int(b) for b in budget]
        self.t_shift += delta
        return SLIDE if drop else PACK
