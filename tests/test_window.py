"""The cache window (Fill / Pack / Slide, Sec. 3.4 and Fig. 6; rebase, Eq. 9).

CPU part: the reference state machine in oracle/window.py against what the paper fixes — the allocation pattern printed
after Eq. 7 row by row as the window fills, first-in-first-out eviction, the rebase moving t only — and against
structural invariants.  GPU part: the library's window against the reference, frame by frame, bit for bit on counts,
packed rows and positions when both select on the same fp32 scores, and attention over the window's cache against the
oracle's attention over the reference's cache."""
from __future__ import annotations

import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import window as ow
from paper_2601_04359_b200 import workload as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "allocation_pattern.txt")


def _frames(cfg, n_frames, seed=0):
    """K, V, positions of frames 1..n_frames and the queries of each following frame (tags = global token ids)."""
    rng = np.random.Generator(np.random.Philox(key=[seed, 77]))
    n, hkv, hq, d = cfg.frame_tokens, cfg.n_kv_heads, cfg.n_q_heads, cfg.head_dim
    st = lambda x: wl.to_storage(x.astype(np.float32), cfg.dtype)
    out = []
    for f in range(1, n_frames + 2):
        pos = wl.frame_positions(cfg, f, cfg.n_anchor + (f - 1) * n)
        out.append(dict(k=st(rng.standard_normal((n, hkv, d))), v=st(rng.standard_normal((n, hkv, d))), pos=pos,
                        q=st(rng.standard_normal((n, hq, d)))))
    return out


def _printed_pattern():
    rows = {}
    for line in open(GOLDEN):
        if line.strip() and not line.startswith("#"):
            w, vals = line.split(":")
            rows[int(w)] = [Fraction(x) for x in vals.split()]
    return rows


def test_window_fills_by_the_printed_allocation_pattern():
    """With a budget of one frame (B_one = N) and the closed-form decay, the cache after 1, 2, 3, 4 frames holds
    N x [1], [1/2, 1/2], [1/2, 1/4, 1/4], [1/2, 1/4, 1/8, 1/8] tokens, newest first: the pattern printed after Eq. 7."""
    cfg = wl.CONFIGS["tiny"]
    n = cfg.frame_tokens
    fr = _frames(cfg, 6)
    ref = ow.WindowRef(4, oracle.CLOSED_HALF, 0.5, n, 0)
    rows = _printed_pattern()
    for f in range(4):
        ref.append(fr[f]["k"], fr[f]["v"], fr[f]["pos"])
        regime = ref.update(fr[f + 1]["q"], fr[f + 1]["pos"])
        assert regime == (ow.FILL if f == 0 else ow.PACK)
        assert ref.count[::-1] == [int(n * b) for b in rows[f + 1]]
        assert sum(ref.count) == n
    # sliding: the window stays at four frames under the W = 4 row, the oldest frame leaves
    for f in range(4, 6):
        ref.append(fr[f]["k"], fr[f]["v"], fr[f]["pos"])
        assert ref.update(fr[f + 1]["q"], fr[f + 1]["pos"]) == ow.SLIDE
        assert ref.count[::-1] == [int(n * b) for b in rows[4]]
        frames_present = sorted(set(((ref.pos[:, 3] - cfg.n_anchor) // n).tolist()))
        assert frames_present == list(range(f - 3, f + 1))                 # tags prove which frames survive (FIFO)


def test_window_rebase_moves_t_only_and_kept_sets_shrink():
    cfg = wl.CONFIGS["tiny"]
    n = cfg.frame_tokens
    fr = _frames(cfg, 7, seed=3)
    plain = ow.WindowRef(3, oracle.HALFLIFE, 1.0, 96, 1)
    moved = ow.WindowRef(3, oracle.HALFLIFE, 1.0, 96, 1, rebase=True, t_step=4)
    kept_before = {}
    for f in range(7):
        for w in (plain, moved):
            pos = fr[f]["pos"].copy()
            pos[:, 0] -= w.t_shift                                          # the caller builds positions in the shifted frame
            qpos = fr[f + 1]["pos"].copy()
            qpos[:, 0] -= w.t_shift
            w.append(fr[f]["k"], fr[f]["v"], pos)
            w.update(fr[f + 1]["q"], qpos)
        assert plain.count == moved.count and moved.t_shift == 4 * max(0, f + 1 - 3)
        # same tokens either way (rotary logits depend on position differences only), t lower by the shift, h / w / tag equal
        assert np.array_equal(plain.pos[:, 1:], moved.pos[:, 1:])
        assert np.array_equal(plain.pos[:, 0] - moved.t_shift, moved.pos[:, 0])
        assert np.array_equal(plain.k, moved.k)
        # a frame's kept tokens only ever shrink: re-selection is from what the last pack kept
        tags = set(plain.pos[:, 3].tolist())
        for g, old in kept_before.items():
            now = {t for t in tags if (t - cfg.n_anchor) // n == g}
            assert now <= old
        kept_before = {g: {t for t in tags if (t - cfg.n_anchor) // n == g} for g in range(f + 1)}
        assert sum(plain.count) <= 96 and len(plain.count) <= 3


def test_window_minimum_quota_lets_the_oldest_frames_leave():
    """b_min of Sec. 3.4: every frame that stays keeps at least m tokens; when W * m exceeds the budget only floor(B / m)
    frames can be served and the oldest leave first (first in, first out) — as whole frames, counted in the rebase."""
    cfg = wl.CONFIGS["tiny"]
    n = cfg.frame_tokens                                                      # 64 tokens per frame
    fr = _frames(cfg, 8, seed=5)
    W, B, m = 6, 128, 48                                                      # floor(128 / 48) = 2 frames can be served
    ref = ow.WindowRef(W, oracle.CLOSED_HALF, 0.5, B, 0, rebase=True, t_step=4, min_quota=m)
    left_total = 0
    for f in range(8):
        pos = fr[f]["pos"].copy(); pos[:, 0] -= ref.t_shift
        qpos = fr[f + 1]["pos"].copy(); qpos[:, 0] -= ref.t_shift
        before = len(ref.count) + 1
        ref.append(fr[f]["k"], fr[f]["v"], pos)
        regime = ref.update(fr[f + 1]["q"], qpos)
        left_total += before - len(ref.count)
        assert ref.t_shift == 4 * left_total                                  # every frame that left moved t by one step
        if f == 0:
            assert regime == ow.FILL and ref.count == [n]
            continue
        assert len(ref.count) == 2 and sum(ref.count) == B and min(ref.count) >= m
        frames_of = (ref.pos[:, 3] - cfg.n_anchor) // n
        assert sorted(set(frames_of.tolist())) == [f - 1, f]                  # the two newest frames, nothing older
        assert regime == (ow.FILL if f == 1 else ow.SLIDE)                    # two whole frames are exactly the budget
    # a quota that every frame of the window can have changes nothing about who stays
    easy = ow.WindowRef(W, oracle.CLOSED_HALF, 0.5, B, 0, min_quota=8)        # 6 * 8 <= 128
    for f in range(8):
        easy.append(fr[f]["k"], fr[f]["v"], fr[f]["pos"])
        easy.update(fr[f + 1]["q"], fr[f + 1]["pos"])
        assert len(easy.count) == min(f + 1, W) and (f == 0 or min(easy.count) >= 8)
        assert sum(easy.count) == min(B, (f + 1) * n)


# ------------------------------------------------------------------------------------------------ GPU
@pytest.mark.gpu
@pytest.mark.parametrize("rebase", [False, True])
def test_window_matches_reference_frame_by_frame(rebase):
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import dev, host, idev, make_ctx, segment

    cfg = wl.small_bf16(n_frames=8, grid=(9, 15), n_text=37, total=300, kind=wl.HALFLIFE, param=2.0, keep_full=1, seed=9)
    n, W, total = cfg.frame_tokens, 5, 300
    L = wl.make_layer(cfg)                                                  # anchors only
    fr = _frames(cfg, 8, seed=5)
    ctx = make_ctx(cfg, max_keys=cfg.n_anchor + total + 3 * n)
    cap = total + 2 * n
    td = torch.bfloat16
    mk = lambda: pc.Segment(torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 7.0, dtype=td, device="cuda"),
                            torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 7.0, dtype=td, device="cuda"),
                            torch.full((cap, 4), -9, dtype=torch.int32, device="cuda"), 0)
    anchors = segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype)
    win = pc.Window(ctx, W, pc.PC_HALFLIFE, 2.0, total, 1, anchors, mk(), mk(), rebase=rebase, t_step=4)
    ref = ow.WindowRef(W, oracle.HALFLIFE, 2.0, total, 1, rebase=rebase, t_step=4)
    regimes = []
    for f in range(8):
        pos = fr[f]["pos"].copy(); pos[:, 0] -= ref.t_shift
        qpos = fr[f + 1]["pos"].copy(); qpos[:, 0] -= ref.t_shift
        ref.append(fr[f]["k"], fr[f]["v"], pos)
        win.append(segment(fr[f]["k"], fr[f]["v"], pos, cfg.dtype))
        # both sides select on the same fp32 scores (the oracle's); the GPU's own scores are checked separately below
        sk, _, spos, scounts, _ = ref.source_after_drop()
        s32 = oracle.score_pooled(sk, spos, fr[f + 1]["q"], qpos, cfg.rope_base).astype(np.float32)
        want_regime = ref.update(fr[f + 1]["q"], qpos, scores32=s32)
        got_regime = win.update(dev(fr[f + 1]["q"], cfg.dtype), idev(qpos), scores_override=torch.from_numpy(s32).cuda())
        assert got_regime == want_regime
        regimes.append(got_regime)
        counts, shift, _ = win.state()
        assert counts.tolist() == ref.count and shift == ref.t_shift
        cache = win.cache()
        m = int(counts.sum())
        assert np.array_equal(host(cache.history.k)[:m], ref.k) and np.array_equal(host(cache.history.v)[:m], ref.v)
        assert np.array_equal(cache.history.pos.cpu().numpy()[:m], ref.pos)
        # attention of the next frame's queries over the window's cache
        out = pc.pc_attend_frame(ctx, cache, None, dev(fr[f + 1]["q"], cfg.dtype), idev(qpos))
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        want = oracle.attend(fr[f + 1]["q"], qpos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (ref.k, ref.v, ref.pos)], cfg.rope_base)
        assert np.abs(host(out).astype(np.float64) - want).max() <= 2e-2
    assert regimes[0] == pc.PC_WINDOW_FILL and pc.PC_WINDOW_PACK in regimes and regimes[-1] == pc.PC_WINDOW_SLIDE
    win.close(); ctx.close()


@pytest.mark.gpu
def test_window_on_its_own_scores_keeps_valid_state():
    """Without an override the window scores on the GPU: counts follow the plan, every kept token is a token of the
    frame it is filed under, and each frame's kept set only shrinks."""
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import dev, idev, make_ctx, segment

    cfg = wl.small_bf16(n_frames=8, grid=(9, 15), n_text=37, total=300, kind=wl.LINEAR, param=0.0, keep_full=0, seed=2)
    n, W, total = cfg.frame_tokens, 4, 260
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 7, seed=8)
    ctx = make_ctx(cfg, max_keys=cfg.n_anchor + total + 3 * n)
    cap = total + 2 * n
    mk = lambda: pc.Segment(torch.zeros((cap, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((cap, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((cap, 4), dtype=torch.int32, device="cuda"), 0)
    win = pc.Window(ctx, W, pc.PC_LINEAR, 0.0, total, 0, segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype), mk(), mk())
    kept = {}
    counts_before = []
    for f in range(7):
        win.append(segment(fr[f]["k"], fr[f]["v"], fr[f]["pos"], cfg.dtype))
        regime = win.update(dev(fr[f + 1]["q"], cfg.dtype), idev(fr[f + 1]["pos"]))
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        counts, shift, _ = win.state()
        avail = (counts_before + [n])[-W:] if regime != pc.PC_WINDOW_FILL else None
        if avail is not None:
            assert counts.tolist() == oracle.plan_budget(oracle.LINEAR, 0.0, total, 0, avail).tolist()
        tags = win.cache().history.pos.cpu().numpy()[:int(counts.sum()), 3]
        frames_of = (tags - cfg.n_anchor) // n
        first = f + 1 - len(counts)
        want_frames = np.repeat(np.arange(first, first + len(counts)), counts)
        assert np.array_equal(frames_of, want_frames) and len(set(tags.tolist())) == len(tags)
        now = {g: set(tags[frames_of == g].tolist()) for g in range(first, f + 1)}
        for g, s in now.items():
            assert g not in kept or s <= kept[g]
        kept = now
        counts_before = counts.tolist()
    win.close(); ctx.close()


def test_masked_append_removes_positions_in_the_reference():
    """Cache mask of Eq. 1 at write time: masked positions never enter the cache (their tags never appear), the frame's
    count is the number of unmasked positions, order and coordinates of the kept ones are untouched."""
    cfg = wl.CONFIGS["tiny"]
    n = cfg.frame_tokens
    fr = _frames(cfg, 3, seed=6)
    rng = np.random.default_rng(4)
    ref = ow.WindowRef(4, oracle.CLOSED_HALF, 0.5, 10 ** 6, 0)             # budget never binds: only the mask removes
    kept_tags = []
    for f in range(3):
        valid = (rng.random(n) < 0.6).astype(np.uint8)
        ref.append(fr[f]["k"], fr[f]["v"], fr[f]["pos"], valid=valid)
        assert ref.update(fr[f + 1]["q"], fr[f + 1]["pos"]) == ow.FILL
        kept_tags += fr[f]["pos"][valid != 0, 3].tolist()
        assert ref.count[-1] == int(valid.sum())
    assert ref.pos[:, 3].tolist() == kept_tags
    assert np.array_equal(ref.k, np.concatenate([fr[f]["k"] for f in range(3)])[np.isin(
        np.concatenate([fr[f]["pos"][:, 3] for f in range(3)]), kept_tags)])


@pytest.mark.gpu
def test_window_masked_append_matches_reference():
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import dev, host, idev, make_ctx, segment

    cfg = wl.small_bf16(n_frames=6, grid=(33, 35), n_text=37, total=900, kind=wl.HALFLIFE, param=2.0, keep_full=1, seed=12)
    n, W, total = cfg.frame_tokens, 3, 900                                   # 1155 tokens per frame: more than one scan chunk
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 5, seed=13)
    ctx = make_ctx(cfg, max_keys=cfg.n_anchor + total + 3 * n)
    cap = total + 2 * n
    mk = lambda: pc.Segment(torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=torch.bfloat16, device="cuda"),
                            torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=torch.bfloat16, device="cuda"),
                            torch.full((cap, 4), -3, dtype=torch.int32, device="cuda"), 0)
    win = pc.Window(ctx, W, pc.PC_HALFLIFE, 2.0, total, 1, segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype), mk(), mk())
    ref = ow.WindowRef(W, oracle.HALFLIFE, 2.0, total, 1)
    rng = np.random.default_rng(1)
    for f in range(5):
        valid = (rng.random(n) < (0.7 if f % 2 else 0.35)).astype(np.uint8)
        if f == 2:
            valid[:] = 0; valid[[0, 511, 1024, n - 1]] = 1                   # nearly empty, with survivors at chunk edges
        ref.append(fr[f]["k"], fr[f]["v"], fr[f]["pos"], valid=valid)
        win.append_masked(segment(fr[f]["k"], fr[f]["v"], fr[f]["pos"], cfg.dtype), torch.from_numpy(valid).cuda(), int(valid.sum()))
        sk, _, spos, _, _ = ref.source_after_drop()
        s32 = oracle.score_pooled(sk, spos, fr[f + 1]["q"], fr[f + 1]["pos"], cfg.rope_base).astype(np.float32)
        want = ref.update(fr[f + 1]["q"], fr[f + 1]["pos"], scores32=s32)
        got = win.update(dev(fr[f + 1]["q"], cfg.dtype), idev(fr[f + 1]["pos"]), scores_override=torch.from_numpy(s32).cuda())
        assert got == want and pc.pc_poll_status(ctx) == pc.PC_OK
        counts, _, _ = win.state()
        assert counts.tolist() == ref.count
        cache = win.cache()
        m = int(counts.sum())
        assert np.array_equal(host(cache.history.k)[:m], ref.k) and np.array_equal(cache.history.pos.cpu().numpy()[:m], ref.pos)
        assert np.array_equal(host(cache.history.v)[:m], ref.v)
    # a count that does not match the mask is recorded, not trusted
    valid = np.ones(n, np.uint8)
    win.append_masked(segment(fr[0]["k"], fr[0]["v"], fr[0]["pos"], cfg.dtype), torch.from_numpy(valid).cuda(), n - 5)
    assert pc.pc_poll_status(ctx) == pc.PC_ERR_INVALID_ARG
    win.close(); ctx.close()


@pytest.mark.gpu
def test_masked_append_respects_the_smaller_buffer_like_append():
    """Two history buffers of unequal size: the caller's score / index scratch has the size of the smaller one, so a
    masked append that would grow the active (larger) buffer past it must be refused before anything is enqueued, as
    the plain append is."""
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import make_ctx, segment

    cfg = wl.small_bf16(n_frames=4, grid=(8, 9), n_text=37, total=100, seed=14)
    n = cfg.frame_tokens                                                     # 72 tokens per frame
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 4, seed=15)
    ctx = make_ctx(cfg)
    mk = lambda cap: pc.Segment(torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=torch.bfloat16, device="cuda"),
                                torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=torch.bfloat16, device="cuda"),
                                torch.full((cap, 4), -3, dtype=torch.int32, device="cuda"), 0)
    big, small = mk(4 * n), mk(2 * n + 10)                                   # scratch: 2n + 10 tokens
    win = pc.Window(ctx, 8, pc.PC_HALFLIFE, 2.0, 10 ** 6, 0, segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype), big, small)
    ones = torch.ones(n, dtype=torch.uint8, device="cuda")
    seg = lambda f: segment(fr[f]["k"], fr[f]["v"], fr[f]["pos"], cfg.dtype)
    win.append_masked(seg(0), ones, n)
    win.append_masked(seg(1), ones, n)
    guard = big.k[2 * n:].clone()
    with pytest.raises(pc.PackCacheError) as e:                              # 3n > 2n + 10 although the buffer holds 4n
        win.append_masked(seg(2), ones, n)
    assert e.value.status == pc.PC_ERR_CAPACITY
    with pytest.raises(pc.PackCacheError) as e:
        win.append(seg(2))
    assert e.value.status == pc.PC_ERR_CAPACITY
    torch.cuda.synchronize()
    assert torch.equal(big.k[2 * n:], guard) and win.state()[0].tolist() == [n, n]      # nothing was enqueued or counted
    keep = torch.zeros(n, dtype=torch.uint8, device="cuda"); keep[:10] = 1
    win.append_masked(seg(2), keep, 10)                                      # 2n + 10 still fits
    assert pc.pc_poll_status(ctx) == pc.PC_OK and win.state()[0].tolist() == [n, n, 10]
    win.close(); ctx.close()


@pytest.mark.gpu
def test_window_minimum_quota_matches_reference():
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import dev, host, idev, make_ctx, segment

    cfg = wl.small_bf16(n_frames=8, grid=(9, 15), n_text=37, total=300, kind=wl.HALFLIFE, param=2.0, keep_full=0, seed=31)
    n, W, total, m = cfg.frame_tokens, 5, 300, 90                             # floor(300 / 90) = 3 of the 5 frames can be served
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 7, seed=32)
    ctx = make_ctx(cfg, max_keys=cfg.n_anchor + total + 3 * n)
    cap = total + 2 * n
    mk = lambda: pc.Segment(torch.zeros((cap, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((cap, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((cap, 4), dtype=torch.int32, device="cuda"), 0)
    win = pc.Window(ctx, W, pc.PC_HALFLIFE, 2.0, total, 0, segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype), mk(), mk(),
                    rebase=True, t_step=4, min_quota=m)
    ref = ow.WindowRef(W, oracle.HALFLIFE, 2.0, total, 0, rebase=True, t_step=4, min_quota=m)
    for f in range(7):
        pos = fr[f]["pos"].copy(); pos[:, 0] -= ref.t_shift
        qpos = fr[f + 1]["pos"].copy(); qpos[:, 0] -= ref.t_shift
        ref.append(fr[f]["k"], fr[f]["v"], pos)
        win.append(segment(fr[f]["k"], fr[f]["v"], pos, cfg.dtype))
        sk, _, spos, _, _ = ref.source_after_drop()
        s32 = oracle.score_pooled(sk, spos, fr[f + 1]["q"], qpos, cfg.rope_base).astype(np.float32)
        want = ref.update(fr[f + 1]["q"], qpos, scores32=s32)
        got = win.update(dev(fr[f + 1]["q"], cfg.dtype), idev(qpos), scores_override=torch.from_numpy(s32).cuda())
        assert got == want and pc.pc_poll_status(ctx) == pc.PC_OK
        counts, shift, _ = win.state()
        assert counts.tolist() == ref.count and shift == ref.t_shift
        assert len(ref.count) <= 3 and (f == 0 or min(ref.count) >= m)
        cache = win.cache()
        k = int(counts.sum())
        assert np.array_equal(host(cache.history.k)[:k], ref.k) and np.array_equal(cache.history.pos.cpu().numpy()[:k], ref.pos)
    assert ref.t_shift > 0
    win.close(); ctx.close()


@pytest.mark.gpu
@pytest.mark.parametrize("rebase", [False, True])
def test_window_step_from_host_buffers_reproduces_the_device_side_window(rebase):
    """The resident-cache step (frame and queries in pinned host memory, cache on the device, update and attention
    fused) against the separate device-side calls (append, update, attend) on a second window fed the same frames:
    regimes, token counts, shift, packed cache and attention output must agree bit for bit through Fill, Pack and
    Slide, and the output must match the oracle over the reference window's cache."""
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import dev, host, idev, make_ctx, segment
    from .test_gpu_parity import check_bf16_attention

    cfg = wl.small_bf16(n_frames=6, grid=(9, 15), n_text=37, total=300, kind=wl.HALFLIFE, param=2.0, keep_full=1, seed=21)
    n, W, total = cfg.frame_tokens, 3, 300
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 6, seed=22)
    cap = total + 2 * n
    mk = lambda: pc.Segment(torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=torch.bfloat16, device="cuda"),
                            torch.full((cap, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=torch.bfloat16, device="cuda"),
                            torch.full((cap, 4), -3, dtype=torch.int32, device="cuda"), 0)
    anchors = segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype)
    ctx_a, ctx_b = make_ctx(cfg, max_keys=cfg.n_anchor + cap), make_ctx(cfg, max_keys=cfg.n_anchor + cap)
    win_a = pc.Window(ctx_a, W, pc.PC_HALFLIFE, 2.0, total, 1, anchors, mk(), mk(), rebase=rebase)
    win_b = pc.Window(ctx_b, W, pc.PC_HALFLIFE, 2.0, total, 1, anchors, mk(), mk(), rebase=rebase)
    td = torch.bfloat16
    pin = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(dt) if dt else torch.from_numpy(np.ascontiguousarray(a))).pin_memory()
    ws = {"q": torch.empty((n, cfg.n_q_heads, cfg.head_dim), dtype=td, device="cuda"),
          "q_pos": torch.empty((n, 4), dtype=torch.int32, device="cuda"),
          "out": torch.empty((n, cfg.n_q_heads, cfg.head_dim), dtype=td, device="cuda")}
    out_host = torch.empty((n, cfg.n_q_heads, cfg.head_dim), dtype=td).pin_memory()
    seen = set()
    for f in range(6):
        shift = win_a.state()[1]
        pos = fr[f]["pos"].copy(); pos[:, 0] -= shift                       # frames arrive in the shifted frame of reference
        qpos = fr[f + 1]["pos"].copy(); qpos[:, 0] -= shift
        # (a) device-side calls
        win_a.append(segment(fr[f]["k"], fr[f]["v"], pos, cfg.dtype))
        qd, qpd = dev(fr[f + 1]["q"], cfg.dtype), idev(qpos)
        regime_a = win_a.update(qd, qpd)
        out_a = pc.pc_attend_frame(ctx_a, win_a.cache(), None, qd, qpd)
        # (b) one call from host buffers: the frame, the queries and their positions in, the output back
        regime_b = win_b.step_host({"k": pin(fr[f]["k"], td), "v": pin(fr[f]["v"], td), "pos": pin(pos)},
                                   pin(fr[f + 1]["q"], td), pin(qpos), out_host, ws)
        assert regime_a == regime_b and pc.pc_poll_status(ctx_a) == pc.PC_OK and pc.pc_poll_status(ctx_b) == pc.PC_OK
        seen.add(regime_a)
        ca, sa, _ = win_a.state(); cb, sb, _ = win_b.state()
        assert ca.tolist() == cb.tolist() and sa == sb
        A, B = win_a.cache(), win_b.cache()
        m = int(ca.sum())
        assert torch.equal(A.history.k[:m], B.history.k[:m]) and torch.equal(A.history.v[:m], B.history.v[:m])
        assert torch.equal(A.history.pos[:m], B.history.pos[:m])
        assert torch.equal(out_a.cpu(), out_host)
        want = oracle.attend(fr[f + 1]["q"], qpos, [(L.anchor_k, L.anchor_v, L.anchor_pos),
                                                   (host(B.history.k)[:m], host(B.history.v)[:m], B.history.pos.cpu().numpy()[:m])],
                             cfg.rope_base)
        check_bf16_attention(out_host.float().numpy().astype(np.float64), want)
    assert seen == {pc.PC_WINDOW_FILL, pc.PC_WINDOW_PACK, pc.PC_WINDOW_SLIDE}
    win_a.close(); win_b.close(); ctx_a.close(); ctx_b.close()


@pytest.mark.gpu
def test_sliding_window_comparator_is_a_window_of_one_frame():
    """The sliding-window comparator of the latency curves attends to the anchors and the newest frame.  That is the
    cache window with W = 1 and room for a whole frame: after every update it must hold exactly the newest frame's
    rows, and attention over it must give the bits of attention over (anchors, that frame)."""
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import dev, idev, make_ctx, segment

    cfg = wl.small_bf16(n_frames=4, grid=(9, 15), n_text=37, total=10 ** 6, keep_full=0, seed=23)
    n = cfg.frame_tokens
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 4, seed=24)
    ctx, ctx2 = make_ctx(cfg), make_ctx(cfg)
    mk = lambda: pc.Segment(torch.zeros((2 * n, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((2 * n, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda"),
                            torch.zeros((2 * n, 4), dtype=torch.int32, device="cuda"), 0)
    anchors = segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype)
    win = pc.Window(ctx, 1, pc.PC_HALFLIFE, 2.0, n, 1, anchors, mk(), mk())           # one frame, kept whole
    for f in range(4):
        newest = segment(fr[f]["k"], fr[f]["v"], fr[f]["pos"], cfg.dtype)
        win.append(newest)
        q, qp = dev(fr[f + 1]["q"], cfg.dtype), idev(fr[f + 1]["pos"])
        regime, out = win.step(q, qp)
        assert regime == (pc.PC_WINDOW_FILL if f == 0 else pc.PC_WINDOW_SLIDE)
        cache = win.cache()
        assert win.state()[0].tolist() == [n]
        assert torch.equal(cache.history.k[:n], newest.k) and torch.equal(cache.history.v[:n], newest.v)
        assert torch.equal(cache.history.pos[:n], newest.pos)
        want = pc.pc_attend_frame(ctx2, pc.Cache(anchors, newest, np.array([n], np.int32)), None, q, qp)
        assert torch.equal(out, want)
        assert pc.pc_poll_status(ctx) == pc.PC_OK and pc.pc_poll_status(ctx2) == pc.PC_OK
    win.close(); ctx.close(); ctx2.close()


@pytest.mark.gpu
def test_window_step_from_host_buffers_leaves_the_window_alone_when_the_plan_fails():
    """The step's plan is tried before anything is enqueued: when it cannot be made (here the two frames that are to be
    kept whole exceed the token budget), the call returns the error, the frame is not appended and no buffer is touched;
    the window goes on working."""
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200.device import make_ctx, segment

    cfg = wl.small_bf16(n_frames=3, grid=(8, 9), n_text=37, total=100, keep_full=2, seed=25)
    n = cfg.frame_tokens                                                     # 72 tokens per frame, budget 100, 2 frames whole
    L = wl.make_layer(cfg)
    fr = _frames(cfg, 3, seed=26)
    ctx = make_ctx(cfg)
    td = torch.bfloat16
    mk = lambda: pc.Segment(torch.full((4 * n, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=td, device="cuda"),
                            torch.full((4 * n, cfg.n_kv_heads, cfg.head_dim), 5.0, dtype=td, device="cuda"),
                            torch.full((4 * n, 4), -3, dtype=torch.int32, device="cuda"), 0)
    a, b = mk(), mk()
    win = pc.Window(ctx, 4, pc.PC_HALFLIFE, 2.0, 100, 2, segment(L.anchor_k, L.anchor_v, L.anchor_pos, cfg.dtype), a, b)
    pin = lambda x, dt=None: (torch.from_numpy(np.ascontiguousarray(x)).to(dt) if dt else torch.from_numpy(np.ascontiguousarray(x))).pin_memory()
    ws = {"q": torch.empty((n, cfg.n_q_heads, cfg.head_dim), dtype=td, device="cuda"),
          "q_pos": torch.empty((n, 4), dtype=torch.int32, device="cuda"),
          "out": torch.empty((n, cfg.n_q_heads, cfg.head_dim), dtype=td, device="cuda")}
    out_host = torch.full((n, cfg.n_q_heads, cfg.head_dim), 9.0, dtype=td).pin_memory()
    frame = lambda f, m=n: {"k": pin(fr[f]["k"][:m], td), "v": pin(fr[f]["v"][:m], td), "pos": pin(fr[f]["pos"][:m])}
    assert win.step_host(frame(0), pin(fr[1]["q"], td), pin(fr[1]["pos"]), out_host, ws) == pc.PC_WINDOW_FILL
    first_out = out_host.clone()
    before = (win.state()[0].tolist(), a.k.clone(), b.k.clone())
    with pytest.raises(pc.PackCacheError) as e:                             # 72 + 72 kept whole > 100
        win.step_host(frame(1), pin(fr[2]["q"], td), pin(fr[2]["pos"]), out_host, ws)
    assert e.value.status == pc.PC_ERR_BUDGET
    torch.cuda.synchronize()
    assert win.state()[0].tolist() == before[0] == [n] and torch.equal(a.k, before[1]) and torch.equal(b.k, before[2])
    assert torch.equal(out_host, first_out) and pc.pc_poll_status(ctx) == pc.PC_OK
    assert win.step_host(frame(1, 20), pin(fr[2]["q"], td), pin(fr[2]["pos"]), out_host, ws) == pc.PC_WINDOW_FILL     # 92 fit
    assert win.state()[0].tolist() == [n, 20] and pc.pc_poll_status(ctx) == pc.PC_OK
    win.close(); ctx.close()
