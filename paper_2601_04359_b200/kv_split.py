"""One layer split over several GPUs by KV head (grouped-query attention shards by KV head without any exchange of K, V
or attention outputs; only the scores need one).

Each rank holds its slice of the KV heads — K / V ``[token][Hkv_local][d]`` — and the query heads that read them.
The score of a history token is a mean over all query heads, i.e. a weighted sum of per-rank scores, so one all-reduce
of the fp32 score vector (n_src x 4 bytes: 190 KB at 47 frames) per layer per frame lets every rank select on the same
numbers and therefore keep the same tokens; pack and attention are then rank-local, and the output heads are simply
the concatenation of the ranks' outputs.  This module is argument marshalling and one collective; scoring, selection,
packing and attention run in the library's kernels.

Not measured on several GPUs: the logic is covered by a world-size-2 ``gloo`` test on CPU and by a one-GPU test that
runs the ranks' slices one after the other and adds their scores.
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np
import torch

from . import binding as pc


def head_slice(rank: int, world: int, n_q_heads: int, n_kv_heads: int) -> Tuple[int, int, int, int]:
    """(first KV head, end KV head, first query head, end query head) of a rank; KV heads must divide evenly."""
    if n_kv_heads % world or n_q_heads % n_kv_heads:
        raise ValueError("KV heads must divide evenly over the ranks, and query heads over the KV heads")
    per = n_kv_heads // world
    group = n_q_heads // n_kv_heads
    return rank * per, (rank + 1) * per, rank * per * group, (rank + 1) * per * group


def reduce_scores(local_scores: torch.Tensor, local_q_heads: int, total_q_heads: int, dist=None) -> torch.Tensor:
    """Scores over all query heads from the ranks' scores over their own heads: a rank's score is a mean over its
    ``local_q_heads``, the global one a mean over ``total_q_heads``, so each rank contributes with weight
    local / total.  In place; every rank ends up with the same vector (the all-reduce adds in one order for all)."""
    local_scores.mul_(float(local_q_heads) / float(total_q_heads))
    if dist is not None:
        dist.all_reduce(local_scores, op=dist.ReduceOp.SUM)
    return local_scores


def frame_step(ctx: pc.Context, src: pc.Cache, budget, delta_t: int, dst: pc.Cache, q: torch.Tensor, q_pos: torch.Tensor,
               total_q_heads: int, dist=None, scores: Optional[torch.Tensor] = None, sel_idx: Optional[torch.Tensor] = None,
               out: Optional[torch.Tensor] = None, stream=None):
    """One frame on one rank's head slice: local scores, all-reduce, selection on the reduced scores (identical on every
    rank), local pack, local attention.  ``ctx`` is a context for the local head counts.  Returns (out, scores, sel_idx)."""
    zero = np.zeros(len(src.frame_count), np.int32)
    scores, _ = pc.pc_score(ctx, src, q, q_pos, zero, scores=scores, stream=stream)          # scores only: empty budget
    reduce_scores(scores[:src.history.n_tokens], q.shape[1], total_q_heads, dist)
    _, sel_idx = pc.pc_score(ctx, src, None, None, budget, scores_override=scores, sel_idx=sel_idx, stream=stream)
    pc.pc_compact(ctx, src, sel_idx, budget, delta_t, dst, stream=stream)
    out = pc.pc_attend_frame(ctx, dst, None, q, q_pos, out=out, stream=stream)
    return out, scores, sel_idx
