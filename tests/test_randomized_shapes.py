"""Seeded random shapes through the whole path on the GPU, every stage against the oracle: head groupings from 2/2 to
32/8, frames of 1 to 550 tokens, 0 to 200 text tokens, all four decay kernels, budgets from nothing to everything, with
and without the current frame, 1-4 key ranges (or the automatic choice), both merge forms, the tensor-core and the
CUDA-core attention kernel, and the attention mass where the tensor-core path takes the shape."""
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


def attention_within_bounds(got: np.ndarray, want: np.ndarray, want_abs: np.ndarray) -> bool:
    """2e-2 wherever a bf16 result can meet it, and everywhere a bound made of what the arithmetic can add.  With a few
    dozen keys and V's outlier channels a result can pass 4, where bf16 numbers are 2^-5 apart: storing it alone then costs
    up to 1.6e-2 (seen: 4.1048 stored as 4.125), so the absolute bound is asked of results below 4 only.  Element-wise:
    one bf16 spacing of the result (storing it), plus 2^-6 * sum_j p_j |v_j| (want_abs: the oracle's attention over |V|),
    plus 1e-3.  The middle term: a probability reaches the tensor core with three bf16 roundings behind it, its own and
    those of the rotated query and key (through the logit), 2^-9 relative each; over thousands of keys they cancel, over a
    handful they do not.  Seen over 300 random cases: at most 2^-7.3 of the sum (3 to 12 keys), below 2^-8 from 30 keys on."""
    from .test_gpu_parity import bf16_ulp
    err = np.abs(got - want)
    return bool((err[np.abs(want) < 4.0] <= 2e-2).all() and (err <= bf16_ulp(want) + 2.0 ** -6 * want_abs + 1e-3).all())


def abs_v(segs):
    return [(k, np.abs(v), p) for k, v, p in segs]


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
        impl = [0, 0, 1][rng.integers(3)]
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
        assert attention_within_bounds(host(out).astype(np.float64), want, oracle.attend(L.q, L.q_pos, abs_v(segs), cfg.rope_base)), what
        assert np.abs(host(lse) - want_lse).max() <= 2e-2, what
        if hkv * cfg.head_dim % 256 == 0 and impl == 0:
            n_keys = sum(len(s[0]) for s in segs)
            got = host(pc.pc_attend_mass(ctx, lse, n_keys)).astype(np.float64)
            want_mass = oracle.attend_mass(L.q, L.q_pos, [(s[0], s[2]) for s in segs], cfg.rope_base)
            assert pc.pc_poll_status(ctx) == pc.PC_OK, what
            assert (np.abs(got - want_mass) <= 5e-3 * want_mass + 1e-3 / n_keys).all(), what
        ctx.close()


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_fused_steps_against_the_separate_calls_and_the_oracle(seed):
    """pc_frame_step on random shapes: the bits of pc_score -> pc_compact -> pc_attend_frame (scores, indices, packed
    rows, output, log-sum-exp), twice in a row (the second step finds the anchors' rotated keys kept), with and without
    anchors, with and without a rebase; the output also against the oracle's attention over the oracle's pack of the
    selected rows."""
    rng = np.random.default_rng(100 + seed)
    same = lambda a, b: torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    for case in range(5):
        hq, hkv = HEADS[rng.integers(len(HEADS))]
        grid = (int(rng.integers(1, 20)), int(rng.integers(1, 30)))
        n_frames, n_text = int(rng.integers(1, 7)), int(rng.integers(1, 200))
        n = grid[0] * grid[1]
        total = int(rng.integers(0, n_frames * n + 1))
        keep_full = int(rng.integers(0, 3)) if total >= 2 * n else 0
        kind = list(DECAY)[rng.integers(4)]
        delta_t = int(rng.integers(0, 2)) * 4
        anchors = bool(rng.integers(4))                      # one case in four has no anchors
        cfg = replace(wl.small_bf16(n_frames=n_frames, grid=grid, n_text=n_text, total=total, kind=kind, param=DECAY[kind],
                                    keep_full=min(keep_full, n_frames), seed=3000 + 10 * seed + case), n_q_heads=hq, n_kv_heads=hkv)
        what = f"{cfg.name} heads {hq}/{hkv} text {n_text} budget {total}/{keep_full} decay {kind} delta_t {delta_t} anchors {anchors}"
        L = wl.make_layer(cfg)
        if not anchors:
            L.anchor_k, L.anchor_v, L.anchor_pos = L.anchor_k[:0], L.anchor_v[:0], L.anchor_pos[:0]
        D = DeviceLayer(L)
        b = cfg.budget
        budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
        n_sel = int(budget.sum())
        if n_sel == 0 and not anchors:
            continue                                         # nothing to attend to: an argument error, covered elsewhere
        ref_ctx, ctx = make_ctx(cfg), make_ctx(cfg)
        scores0, sel0 = pc.pc_score(ref_ctx, D.cache, D.q, D.q_pos, budget)
        dst0 = D.empty_packed(n_sel + 3, poison=5.0)
        pc.pc_compact(ref_ctx, D.cache, sel0, budget, delta_t, dst0)
        out0, lse0 = pc.pc_attend_frame(ref_ctx, dst0, None, D.q, D.q_pos, want_lse=True)
        assert pc.pc_poll_status(ref_ctx) == pc.PC_OK, what
        for step in range(2):
            dst = D.empty_packed(n_sel + 3, poison=5.0)
            out, scores, sel, lse = pc.pc_frame_step(ctx, D.cache, budget, delta_t, dst, D.q, D.q_pos, want_lse=True)
            assert pc.pc_poll_status(ctx) == pc.PC_OK, what
            assert same(scores[:cfg.n_src], scores0[:cfg.n_src]) and same(sel[:n_sel], sel0[:n_sel]), what
            assert same(dst.history.k, dst0.history.k) and same(dst.history.v, dst0.history.v), what
            assert same(dst.history.pos, dst0.history.pos) and dst.history.n_tokens == n_sel, what
            assert same(out, out0) and same(lse, lse0), what
        sel_np = sel.cpu().numpy()[:n_sel]
        wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel_np, delta_t)
        segs = [s for s in [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)] if len(s[0])]
        want, want_lse = oracle.attend(L.q, L.q_pos, segs, cfg.rope_base, want_lse=True)
        assert attention_within_bounds(host(out).astype(np.float64), want, oracle.attend(L.q, L.q_pos, abs_v(segs), cfg.rope_base)), what
        assert np.abs(host(lse) - want_lse).max() <= 2e-2, what
        ref_ctx.close(); ctx.close()


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_random_cache_windows_against_the_reference(seed):
    """Seeded random cache-window runs (window length 1-6, all decay kernels, budgets from a few tokens to several frames,
    kept-whole frames, minimum quotas, cache masks at append time, rebase on and off): the library's window against the
    reference state machine after every frame — regime, token counts, accumulated shift, packed K / V / positions bit for
    bit — both deciding on the same fp32 scores."""
    from oracle import window as ow
    from paper_2601_04359_b200.device import dev, idev, segment

    rng = np.random.default_rng(100 + seed)
    for case in range(8):
        grid = (int(rng.integers(2, 14)), int(rng.integers(2, 20)))
        n = grid[0] * grid[1]
        n_text, n_steps, W = int(rng.integers(0, 100)), int(rng.integers(3, 9)), int(rng.integers(1, 7))
        kind = list(DECAY)[rng.integers(4)]
        total = int(rng.integers(1, 4 * n))
        keep_full = int(rng.integers(0, 2)) if total >= n else 0
        m = int(rng.integers(0, max(1, n // 2))) if rng.integers(2) else 0
        rebase, masked = bool(rng.integers(2)), bool(rng.integers(2))
        hq, hkv = [(24, 8), (8, 8), (4, 2), (6, 2)][rng.integers(4)]
        cfg = replace(wl.small_bf16(n_frames=n_steps + 1, grid=grid, n_text=n_text, total=total, kind=kind, param=DECAY[kind],
                                    keep_full=keep_full, seed=6000 + 10 * seed + case), n_q_heads=hq, n_kv_heads=hkv)
        what = f"grid {grid} W {W} decay {kind} budget {total}/{keep_full}/{m} rebase {rebase} masked {masked} heads {hq}/{hkv}"
        L = wl.make_layer(cfg)
        g = np.random.Generator(np.random.Philox(key=[seed, case]))
        st = lambda x: wl.to_storage(x.astype(np.float32), cfg.dtype)
        cap = total + 2 * n + 8
        ctx = make_ctx(cfg, max_keys=cfg.n_anchor + cap + n)
        mk = lambda: pc.Segment(torch.zeros((cap, hkv, 128), dtype=torch.bfloat16, device="cuda"),
                                torch.zeros((cap, hkv, 128), dtype=torch.bfloat16, device="cuda"),
                                torch.zeros((cap, 4), dtype=torch.int32, device="cuda"), 0)
        win = pc.Window(ctx, W, kind, DECAY[kind], total, keep_full, segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype),
                        mk(), mk(), rebase=rebase, t_step=4, min_quota=m)
        ref = ow.WindowRef(W, kind, DECAY[kind], total, keep_full, rebase=rebase, t_step=4, min_quota=m)
        for f in range(1, n_steps + 1):
            pos = wl.frame_positions(cfg, f, cfg.n_anchor + (f - 1) * n)
            qpos = wl.frame_positions(cfg, f + 1, cfg.n_anchor + f * n)
            pos[:, 0] -= ref.t_shift
            qpos[:, 0] -= ref.t_shift
            k, v = st(g.standard_normal((n, hkv, 128))), st(g.standard_normal((n, hkv, 128)))
            q = st(g.standard_normal((n, hq, 128)))
            if masked and rng.integers(2):
                valid = (rng.random(n) < rng.random()).astype(np.uint8)
                ref.append(k, v, pos, valid=valid)
                win.append_masked(segment(k, v, pos, cfg.dtype), torch.from_numpy(valid).cuda(), int(valid.sum()))
            else:
                ref.append(k, v, pos)
                win.append(segment(k, v, pos, cfg.dtype))
            sk, _, spos, _, _ = ref.source_after_drop()
            s32 = oracle.score_pooled(sk, spos, q, qpos, cfg.rope_base).astype(np.float32) if len(sk) else np.zeros(1, np.float32)
            try:
                want = ref.update(q, qpos, scores32=s32 if len(sk) else None)
            except oracle.OracleError:                              # kept-whole frames exceed the budget: both must refuse
                with pytest.raises(pc.PackCacheError):
                    win.update(dev(q, cfg.dtype), idev(qpos), scores_override=torch.from_numpy(s32).cuda())
                break
            got = win.update(dev(q, cfg.dtype), idev(qpos), scores_override=torch.from_numpy(s32).cuda())
            assert got == want and pc.pc_poll_status(ctx) == pc.PC_OK, what
            counts, shift, _ = win.state()
            assert counts.tolist() == ref.count and shift == ref.t_shift, what
            kk = int(counts.sum())
            if kk:
                cache = win.cache()
                assert np.array_equal(host(cache.history.k)[:kk], ref.k) and np.array_equal(host(cache.history.v)[:kk], ref.v), what
                assert np.array_equal(cache.history.pos.cpu().numpy()[:kk], ref.pos), what
        win.close()
        ctx.close()
