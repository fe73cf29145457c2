"""Seeded random shapes through the whole path on the GPU, every stage against the oracle: head groupings from 2/2 to
32/8, frames of 1 to 550 tokens, 0 to 200 text tokens, all four decay kernels, budgets from nothing to everything, with
and without the current frame, 1-4 key ranges (or the automatic choice), both merge forms, the default and the CTA-pair
attention kernel, and the attention mass where the tensor-core path takes the shape."""
from __future__ import annotations

from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import workload as wl
from paper_2601_04359_b200.device import DeviceLayer, host, make_ctx, score_tolerance

pytestmark = pytest.mark.gpu

HEADS = [(24, 8), (8, 8), (16, 4), (32, 8), (6, 2), (4, 2), (12, 4), (2, 2)]
DECAY = {wl.HALFLIFE: 2.0, wl.LINEAR: 0.0, wl.GEOMETRIC: 0.6, wl.CLOSED_HALF: 0.5}


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4])
def test_random_shapes_against_the_oracle(seed):
    rng = np.random.default_rng(seed)
    for case in range(5):
        hq, hkv = HEADS[rng.integers(len(HEADS))]
        grid = (int(rng.integers(1, 20)), int(rng.integers(1, 30)))
        n_frames, n_text = int(rng.integers(1, 6)), int(rng.integers(0, 200))
        n = grid[0] * grid[1]
        total = int(rng.integers(0, n_frames * n + 1))
        keep_full = int(rng.integers(0, 2)) if total >= n else 0
        kind = list(DECAY)[rng.integers(4)]
        cfg = replace(wl.small_bf16(n_frames=n_frames, grid=grid, n_text=n_text, total=total, kind=kind, param=DECAY[kind],
                                    keep_full=keep_full, seed=2000 + 10 * seed + case), n_q_heads=hq, n_kv_heads=hkv)
        with_cur, splits, cluster = bool(rng.integers(2)), int(rng.integers(0, 5)), bool(rng.integers(2))
        impl = [0, 0, 2][rng.integers(3)]
        what = f"{cfg.name} heads {hq}/{hkv} text {n_text} budget {total}/{keep_full} decay {kind} current {with_cur} ranges {splits} " \
               f"cluster {cluster} impl {impl}"
        L = wl.make_layer(cfg, with_current=True)
        D = DeviceLayer(L)
        ctx = make_ctx(cfg)
        b = cfg.budget
        budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
        assert budget.tolist() == oracle.plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count).tolist(), what
        scores, _ = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
        ref = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)
        assert (np.abs(host(scores)[:cfg.n_src].astype(np.float64) - ref) <= score_tolerance(ref, L.frame_count)).all(), what
        ref32 = ref.astype(np.float32)
        _, sel = pc.pc_score(ctx, D.cache, None, None, budget, scores_override=torch.from_numpy(ref32).cuda())
        want_sel = oracle.select(ref32, L.frame_count, budget)
        m = len(want_sel)
        assert sel.cpu().numpy()[:m].tolist() == want_sel.tolist(), what
        dst = D.empty_packed(m + 3)
        pc.pc_compact(ctx, D.cache, sel, budget, 4, dst)
        wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, want_sel, 4)
        assert np.array_equal(host(dst.history.k)[:m], wk) and np.array_equal(host(dst.history.v)[:m], wv), what
        assert np.array_equal(dst.history.pos.cpu().numpy()[:m], wp), what
        pc.pc_set_kv_splits(ctx, splits)
        pc.pc_set_cluster_merge(ctx, cluster)
        pc.pc_set_attend_impl(ctx, impl)
        segs = [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)] + ([(L.cur_k, L.cur_v, L.q_pos)] if with_cur else [])
        segs = [s for s in segs if len(s[0])]
        out, lse = pc.pc_attend_frame(ctx, dst, D.current if with_cur else None, D.q, D.q_pos, want_lse=True)
        want, want_lse = oracle.attend(L.q, L.q_pos, segs, cfg.rope_base, want_lse=True)
        assert pc.pc_poll_status(ctx) == pc.PC_OK, what
        assert np.abs(host(out).astype(np.float64) - want).max() <= 2e-2, what
        assert np.abs(host(lse) - want_lse).max() <= 2e-2, what
        if hkv * cfg.head_dim % 256 == 0:
            n_keys = sum(len(s[0]) for s in segs)
            got = host(pc.pc_attend_mass(ctx, lse, n_keys)).astype(np.float64)
            want_mass = oracle.attend_mass(L.q, L.q_pos, [(s[0], s[2]) for s in segs], cfg.rope_base)
            assert pc.pc_poll_status(ctx) == pc.PC_OK, what
            assert (np.abs(got - want_mass) <= 1e-2 * want_mass + 1e-3 / n_keys).all(), what
        ctx.close()
