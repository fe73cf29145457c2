"""The KV-head split of one layer on one GPU: the ranks' head slices are processed one after the other by the library
(scores of each slice, then their weighted sum as every rank would hold it after the all-reduce, then selection, pack
and attention per slice) and compared with the unsplit layer and with the oracle."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import kv_split
from paper_2601_04359_b200 import workload as wl
from paper_2601_04359_b200.device import DeviceLayer, dev, host, idev, score_tolerance

from .test_gpu_parity import check_bf16_attention

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 4])
def test_kv_head_split_emulated_rank_by_rank(world):
    cfg = wl.small_bf16(n_frames=3, grid=(11, 13), n_text=130, total=260, seed=80)
    L = wl.make_layer(cfg)
    b = cfg.budget
    budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    n_sel = int(budget.sum())
    ref = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)

    ranks = []
    for r in range(world):
        kv0, kv1, q0, q1 = kv_split.head_slice(r, world, cfg.n_q_heads, cfg.n_kv_heads)
        ctx = pc.Context(q1 - q0, kv1 - kv0, cfg.head_dim, pc.PC_BF16, cfg.rope_base, cfg.max_pos, cfg.n_q,
                         cfg.n_anchor + cfg.n_src + cfg.n_q)
        seg = lambda k, v, p: pc.Segment(dev(k[:, kv0:kv1], cfg.dtype), dev(v[:, kv0:kv1], cfg.dtype), idev(p), len(k))
        cache = pc.Cache(seg(L.anchor_k, L.anchor_v, L.anchor_pos), seg(L.hist_k, L.hist_v, L.hist_pos), L.frame_count.copy())
        q = dev(L.q[:, q0:q1], cfg.dtype)
        scores, _ = pc.pc_score(ctx, cache, q, idev(L.q_pos), np.zeros(cfg.n_frames, np.int32))
        ranks.append(dict(ctx=ctx, cache=cache, q=q, heads=(kv0, kv1, q0, q1), scores=scores))
    # what the all-reduce leaves on every rank: the weighted sum of the ranks' scores
    reduced = torch.zeros(cfg.n_src, dtype=torch.float32, device="cuda")
    for R in ranks:
        reduced += kv_split.reduce_scores(R["scores"][:cfg.n_src].clone(), R["heads"][3] - R["heads"][2], cfg.n_q_heads)
    got = host(reduced).astype(np.float64)
    assert (np.abs(got - ref) <= score_tolerance(ref, L.frame_count)).all()

    want_sel = oracle.select(host(reduced), L.frame_count, budget)
    wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, want_sel, 0)
    want = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)], cfg.rope_base)
    for R in ranks:
        kv0, kv1, q0, q1 = R["heads"]
        _, sel = pc.pc_score(R["ctx"], R["cache"], None, None, budget, scores_override=reduced)
        assert sel.cpu().numpy()[:n_sel].tolist() == want_sel.tolist()              # every rank keeps the same tokens
        k = torch.zeros((n_sel, kv1 - kv0, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
        dst = pc.Cache(R["cache"].anchors, pc.Segment(k, torch.zeros_like(k), torch.zeros((n_sel, 4), dtype=torch.int32, device="cuda"), 0),
                       np.zeros(cfg.n_frames, np.int32))
        pc.pc_compact(R["ctx"], R["cache"], sel, budget, 0, dst)
        assert np.array_equal(host(dst.history.k), wk[:, kv0:kv1]) and np.array_equal(dst.history.pos.cpu().numpy(), wp)
        out = pc.pc_attend_frame(R["ctx"], dst, None, R["q"], idev(L.q_pos))
        assert pc.pc_poll_status(R["ctx"]) == pc.PC_OK
        check_bf16_attention(host(out).astype(np.float64), want[:, q0:q1])           # the rank's heads of the layer's output
        R["ctx"].close()
