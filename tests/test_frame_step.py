"""The fused frame step (pc_frame_step) against the three separate calls, bit for bit, and against the oracle.

The one call must give what pc_score -> pc_compact -> pc_attend_frame give on the same inputs: scores, selected
indices, packed rows and positions, attention output and log-sum-exp, all identical bits.  On the tensor-core path
it gets there by other kernels (the query pass leaves the rotated queries, the pack kernel the rotated keys, the
anchors' rotated keys are kept from step to step), so the comparison covers those, too: the second step of each case
runs with the anchors' keys kept from the first, a third one after the anchors changed in place."""
from __future__ import annotations

from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import workload as wl
from paper_2601_04359_b200.device import DeviceLayer, dev, host, make_ctx, score_tolerance

from .test_gpu_parity import _check_attention, _valid_topk

pytestmark = pytest.mark.gpu


def _separate(ctx, D, budget, delta_t, n_sel):
    scores, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    dst = D.empty_packed(n_sel + 3, poison=5.0)
    pc.pc_compact(ctx, D.cache, sel, budget, delta_t, dst)
    out, lse = pc.pc_attend_frame(ctx, dst, None, D.q, D.q_pos, want_lse=True)
    return scores.clone(), sel.clone(), dst, out.clone(), lse.clone()


def _same(a: torch.Tensor, b: torch.Tensor) -> bool:
    return torch.equal(a.view(torch.uint8), b.view(torch.uint8))


CASES = {
    "tiny_fp32": lambda: wl.CONFIGS["tiny"],
    "small_bf16": lambda: wl.small_bf16(),
    "ragged_bf16": lambda: wl.small_bf16(n_frames=3, grid=(11, 13), n_text=130, total=260, kind=wl.LINEAR, param=0.0,
                                         keep_full=0, seed=5),
    "several_tiles": lambda: wl.small_bf16(n_frames=4, grid=(12, 21), n_text=130, total=700, keep_full=1, seed=31),
    "no_anchors": lambda: wl.small_bf16(n_frames=3, grid=(9, 15), n_text=37, total=200, keep_full=0, seed=32),
    # key rows of 1536, 3072 and 4096 bytes (6, 12 and 16 KV heads): the other widths the pack kernel rotates
    "rows_1536": lambda: replace(wl.small_bf16(n_frames=2, grid=(7, 9), n_text=20, total=70, keep_full=0, seed=33), n_q_heads=12, n_kv_heads=6),
    "rows_3072": lambda: replace(wl.small_bf16(n_frames=2, grid=(7, 9), n_text=20, total=70, keep_full=1, seed=34), n_q_heads=24, n_kv_heads=12),
    "rows_4096": lambda: replace(wl.small_bf16(n_frames=2, grid=(7, 9), n_text=20, total=70, keep_full=0, seed=35), n_q_heads=32, n_kv_heads=16),
}


@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("delta_t", [0, 8])
def test_fused_step_gives_the_bits_of_the_separate_calls(case, delta_t):
    cfg = CASES[case]()
    L = wl.make_layer(cfg)
    if case == "no_anchors":
        L.anchor_k, L.anchor_v, L.anchor_pos = L.anchor_k[:0], L.anchor_v[:0], L.anchor_pos[:0]
    D = DeviceLayer(L)
    b = cfg.budget
    budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    n_sel = int(budget.sum())
    ref_ctx, ctx = make_ctx(cfg), make_ctx(cfg)
    scores0, sel0, dst0, out0, lse0 = _separate(ref_ctx, D, budget, delta_t, n_sel)
    assert pc.pc_poll_status(ref_ctx) == pc.PC_OK

    for step in range(2):        # the second step finds the anchors' rotated keys in the context
        dst = D.empty_packed(n_sel + 3, poison=5.0)
        out, scores, sel, lse = pc.pc_frame_step(ctx, D.cache, budget, delta_t, dst, D.q, D.q_pos, want_lse=True)
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        assert _same(scores[:cfg.n_src], scores0[:cfg.n_src]) and _same(sel[:n_sel], sel0[:n_sel])
        assert _same(dst.history.k, dst0.history.k) and _same(dst.history.v, dst0.history.v)
        assert _same(dst.history.pos, dst0.history.pos) and dst.history.n_tokens == n_sel
        assert _same(out, out0) and _same(lse, lse0)

    # against the oracle, on the GPU's own selection (valid top-k of the GPU's own scores)
    ref = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)
    assert (np.abs(host(scores)[:cfg.n_src].astype(np.float64) - ref) <= score_tolerance(ref, L.frame_count)).all()
    sel_np = sel.cpu().numpy()[:n_sel]
    _valid_topk(host(scores)[:cfg.n_src], sel_np, L.frame_count, budget)
    wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel_np, delta_t)
    segs = [s for s in [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)] if len(s[0])]
    want, want_lse = oracle.attend(L.q, L.q_pos, segs, cfg.rope_base, want_lse=True)
    _check_attention(cfg, host(out).astype(np.float64), want)
    assert np.abs(host(lse) - want_lse).max() <= (2e-2 if cfg.dtype == wl.BF16 else 1e-4)

    if len(L.anchor_k):
        # anchors rewritten in place: the kept keys are stale until the context is told
        new_k = wl.to_storage(np.random.default_rng(9).standard_normal(L.anchor_k.shape).astype(np.float32), cfg.dtype)
        D.cache.anchors.k.copy_(dev(new_k, cfg.dtype))
        pc.pc_forget_anchors(ctx)
        dst = D.empty_packed(n_sel + 3, poison=5.0)
        out2, _, _ = pc.pc_frame_step(ctx, D.cache, budget, delta_t, dst, D.q, D.q_pos)
        _, _, _, out_ref, _ = _separate(ref_ctx, D, budget, delta_t, n_sel)
        assert pc.pc_poll_status(ctx) == pc.PC_OK and _same(out2, out_ref) and not _same(out2, out0)
        want2 = oracle.attend(L.q, L.q_pos, [(new_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)], cfg.rope_base)
        _check_attention(cfg, host(out2).astype(np.float64), want2)
    ref_ctx.close(); ctx.close()


def test_fused_step_interleaved_with_other_attention_calls():
    """pc_attend_frame and pc_attend_prepare reuse the context's key scratch: a fused step after them must rebuild the
    anchors' keys, and a prepared key set does not survive a fused step."""
    cfg = wl.small_bf16(n_frames=3, grid=(11, 13), n_text=130, total=260, seed=40)
    L = wl.make_layer(cfg, with_current=True)
    D = DeviceLayer(L)
    b = cfg.budget
    budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    n_sel = int(budget.sum())
    ctx = make_ctx(cfg)
    dst = D.empty_packed(n_sel)
    first, _, _ = pc.pc_frame_step(ctx, D.cache, budget, 0, dst, D.q, D.q_pos)
    first = first.clone()
    full = pc.pc_attend_frame(ctx, D.cache, D.current, D.q, D.q_pos).clone()      # overwrites the scratch
    again, _, _ = pc.pc_frame_step(ctx, D.cache, budget, 0, dst, D.q, D.q_pos)
    assert _same(first, again)
    pc.pc_attend_prepare(ctx, D.cache, D.current)
    assert _same(pc.pc_attend_prepared(ctx, D.q, D.q_pos), full)
    again, _, _ = pc.pc_frame_step(ctx, D.cache, budget, 0, dst, D.q, D.q_pos)
    assert _same(first, again)
    with pytest.raises(pc.PackCacheError):
        pc.pc_attend_prepared(ctx, D.q, D.q_pos)
    assert pc.pc_poll_status(ctx) == pc.PC_OK
    ctx.close()


def test_fused_step_with_an_empty_budget_attends_to_the_anchors_only():
    cfg = wl.small_bf16(n_frames=2, grid=(8, 9), total=0, keep_full=0, seed=41)
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    budget = np.zeros(cfg.n_frames, np.int32)
    ctx = make_ctx(cfg)
    dst = D.empty_packed(4)
    out, _, _ = pc.pc_frame_step(ctx, D.cache, budget, 0, dst, D.q, D.q_pos)
    assert pc.pc_poll_status(ctx) == pc.PC_OK and dst.history.n_tokens == 0
    want = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos)], cfg.rope_base)
    _check_attention(cfg, host(out).astype(np.float64), want)
    ctx.close()


def test_fused_step_at_the_benchmark_size_matches_the_separate_calls():
    cfg = wl.CONFIGS["lumos47"]
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    b = cfg.budget
    budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    n_sel = int(budget.sum())
    ref_ctx, ctx = make_ctx(cfg), make_ctx(cfg)
    scores0, sel0, dst0, out0, lse0 = _separate(ref_ctx, D, budget, 0, n_sel)
    dst = D.empty_packed(n_sel + 3, poison=5.0)
    for step in range(2):
        out, scores, sel, lse = pc.pc_frame_step(ctx, D.cache, budget, 0, dst, D.q, D.q_pos, want_lse=True)
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        assert _same(scores, scores0) and _same(sel[:n_sel], sel0[:n_sel]) and _same(dst.history.k, dst0.history.k)
        assert _same(dst.history.pos, dst0.history.pos) and _same(out, out0) and _same(lse, lse0)
    ref_ctx.close(); ctx.close()


def test_fused_step_rejects_bad_arguments_before_enqueueing_anything():
    """Host-detectable errors return at once: a destination that is too small, a null output, too many queries for
    the context, a budget above a frame's tokens, a destination that overlaps the source; none of them leaves a device-side status or touches the outputs."""
    cfg = wl.small_bf16(n_frames=3, grid=(8, 9), total=100, seed=42)
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    b = cfg.budget
    budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    n_sel = int(budget.sum())
    ctx = make_ctx(cfg)
    out = torch.full_like(D.q, 7.0)
    small = D.empty_packed(n_sel - 1)
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_frame_step(ctx, D.cache, budget, 0, small, D.q, D.q_pos, out=out)
    assert e.value.status == pc.PC_ERR_CAPACITY
    dst = D.empty_packed(n_sel, poison=3.0)
    over = budget.copy(); over[0] = L.frame_count[0] + 1
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_frame_step(ctx, D.cache, over, 0, D.empty_packed(int(over.sum())), D.q, D.q_pos, out=out)
    assert e.value.status == pc.PC_ERR_BUDGET
    tight = make_ctx(cfg, max_q=cfg.n_q - 1)
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_frame_step(tight, D.cache, budget, 0, dst, D.q, D.q_pos, out=out)
    assert e.value.status == pc.PC_ERR_CAPACITY
    lib = pc.load()
    import ctypes as C
    cs, cd = D.cache.c(), dst.c()
    bud = np.ascontiguousarray(budget, np.int32)
    st = lib.pc_frame_step(ctx.handle, C.byref(cs), bud.ctypes.data_as(C.POINTER(C.c_int32)), 0, C.byref(cd), D.q.data_ptr(),
                           D.q_pos.data_ptr(), cfg.n_q, None, None, None, None, None)          # no output buffer
    assert st == pc.PC_ERR_INVALID_ARG
    # what only the pack stage would notice is refused before the scoring stage runs: a destination that is the source
    scores = torch.full((cfg.n_src,), 5.0, dtype=torch.float32, device="cuda")
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_frame_step(ctx, D.cache, budget, 0, D.cache, D.q, D.q_pos, scores=scores, out=out)
    assert e.value.status == pc.PC_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert pc.pc_poll_status(ctx) == pc.PC_OK and pc.pc_poll_status(tight) == pc.PC_OK
    assert (out == 7.0).all() and (host(dst.history.k) == 3.0).all() and (scores == 5.0).all()
    ctx.close(); tight.close()


def test_attention_mass_after_a_fused_step_equals_the_mass_after_the_separate_calls():
    """pc_attend_mass reads the rotated keys and queries the last attention call left in the context; after a fused step
    those were written by the query pass, the pack kernel and the kept anchor keys, and must serve it just the same."""
    cfg = wl.small_bf16(n_frames=3, grid=(11, 13), n_text=130, total=260, seed=43)
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    b = cfg.budget
    budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    n_sel = int(budget.sum())
    n_keys = cfg.n_anchor + n_sel
    ref_ctx, ctx = make_ctx(cfg), make_ctx(cfg)
    _, sel0, dst0, _, lse0 = _separate(ref_ctx, D, budget, 0, n_sel)
    want = pc.pc_attend_mass(ref_ctx, lse0, n_keys).clone()
    for step in range(2):
        dst = D.empty_packed(n_sel + 3)
        _, _, _, lse = pc.pc_frame_step(ctx, D.cache, budget, 0, dst, D.q, D.q_pos, want_lse=True)
        got = pc.pc_attend_mass(ctx, lse, n_keys)
        assert pc.pc_poll_status(ctx) == pc.PC_OK and _same(got, want)
    sel_np = sel0.cpu().numpy()[:n_sel]
    wk, _, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel_np, 0)
    ref = oracle.attend_mass(L.q, L.q_pos, [(L.anchor_k, L.anchor_pos), (wk, wp)], cfg.rope_base)
    assert (np.abs(host(got).astype(np.float64) - ref) <= 5e-3 * ref + 1e-3 / n_keys).all()
    ref_ctx.close(); ctx.close()
