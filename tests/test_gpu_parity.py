"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer results (budgets, selected indices, packed rows and positions) must match bit for bit; fp32 scores
within 1e-4 relative; attention within 1e-4 relative (fp32) or 2e-2 max-abs (bf16, unit-variance inputs)."""
from __future__ import annotations

from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import workload as wl
from paper_2601_04359_b200.device import DeviceLayer, dev, host, idev, make_ctx, score_tolerance, segment

pytestmark = pytest.mark.gpu

BF16_ATOL = 2e-2
BF16_KERNEL_ATOL = 4e-3   # what the kernel may add beyond the rounding of its bf16 output (see check_bf16_attention)
F32_RTOL = 1e-4


def _plan(cfg, n_frames=None):
    b = cfg.budget
    avail = [cfg.frame_tokens] * (n_frames if n_frames is not None else cfg.n_frames)
    got = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, avail)
    assert got.tolist() == oracle.plan_budget(b.kind, b.param, b.total, b.keep_full, avail).tolist()
    return got


def _ok(ctx):
    assert pc.pc_poll_status(ctx) == pc.PC_OK


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bfloat16 numbers at |x| (8 significant bits), floored at the spacing of 2^-6."""
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(x), 2.0 ** -6))) - 7)


def check_bf16_attention(got: np.ndarray, want: np.ndarray):
    """The stated bound (2e-2 max-abs) and a sharper element-wise one.  The output is a bf16 number, so half a spacing of
    error comes from storing it: on the V outlier channels (values near 4, spacing 2^-5) that alone is 1.6e-2 and
    nearly fills the stated bound.  What the kernel itself adds (bf16 rounding of the rotated operands and of the
    probabilities) is bounded apart: |got - want| <= ulp_bf16(want) + 4e-3."""
    err = np.abs(got - want)
    assert err.max() <= BF16_ATOL
    assert (err <= bf16_ulp(want) + BF16_KERNEL_ATOL).all(), float((err - bf16_ulp(want)).max())


def _check_attention(cfg, got: np.ndarray, want: np.ndarray):
    if cfg.dtype == wl.BF16:
        check_bf16_attention(got, want)
    else:
        scale = np.abs(want).max()
        assert np.abs(got - want).max() <= F32_RTOL * scale


def _pipeline(cfg, impl=None, with_current=False, delta_t=0):
    """plan -> score -> select -> pack -> attend, each stage checked against the oracle."""
    L = wl.make_layer(cfg, with_current=with_current)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    if impl is not None:
        pc.pc_set_attend_impl(ctx, impl)
    budget = _plan(cfg)

    # scores: fp32 within 1e-4 relative of the fp64 mean logit
    scores, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    ref = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)
    got = host(scores)[:cfg.n_src].astype(np.float64)
    assert (np.abs(got - ref) <= score_tolerance(ref, L.frame_count)).all()
    # the GPU's own selection must be a valid top-k of the GPU's own scores
    sel_np = sel.cpu().numpy()[:budget.sum()]
    _valid_topk(host(scores)[:cfg.n_src], sel_np, L.frame_count, budget)

    # selection: bit-exact when both sides see the same fp32 scores (the oracle's, rounded to fp32)
    ref32 = ref.astype(np.float32)
    _, sel2 = pc.pc_score(ctx, D.cache, None, None, budget, scores_override=torch.from_numpy(ref32).cuda())
    want_sel = oracle.select(ref32, L.frame_count, budget)
    assert sel2.cpu().numpy()[:len(want_sel)].tolist() == want_sel.tolist()

    # pack: bit copies of the selected rows, positions carried, t rebased
    dst = D.empty_packed(int(budget.sum()) + 5, poison=3.0)
    pc.pc_compact(ctx, D.cache, sel2, budget, delta_t, dst)
    wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, want_sel, delta_t)
    n = len(want_sel)
    assert np.array_equal(host(dst.history.k)[:n], wk) and np.array_equal(host(dst.history.v)[:n], wv)
    assert np.array_equal(dst.history.pos.cpu().numpy()[:n], wp)
    assert (host(dst.history.k)[n:] == 3.0).all() and (dst.history.pos.cpu().numpy()[n:] == -7).all()
    assert dst.history.n_tokens == n

    # attention over anchors ++ packed (++ current)
    segs = [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)]
    if with_current:
        segs.append((L.cur_k, L.cur_v, L.q_pos))
    want, want_lse = oracle.attend(L.q, L.q_pos, segs, cfg.rope_base, want_lse=True)
    out, lse = pc.pc_attend_frame(ctx, dst, D.current if with_current else None, D.q, D.q_pos, want_lse=True)
    _ok(ctx)
    _check_attention(cfg, host(out).astype(np.float64), want)
    assert np.abs(host(lse) - want_lse).max() <= (2e-2 if cfg.dtype == wl.BF16 else 1e-4)
    ctx.close()


def _valid_topk(scores, sel, frame_count, budget):
    """Property check at any size: per frame, ascending unique indices of the right count, and no unselected token
    beats a selected one under (score desc, index asc)."""
    base = out = 0
    for n, t in zip(frame_count, budget):
        s = sel[out:out + t]
        assert (np.diff(s) > 0).all() and (s >= base).all() and (s < base + n).all()
        if 0 < t < n:
            mask = np.zeros(n, bool)
            mask[s - base] = True
            fr = scores[base:base + n]
            worst_in = min(zip(fr[mask], -(np.nonzero(mask)[0])))        # lowest score, then highest index
            best_out = max(zip(fr[~mask], -(np.nonzero(~mask)[0])))      # highest score, then lowest index
            assert worst_in > best_out
        base += n
        out += t


# ------------------------------------------------------------------------------------------- whole pipeline
def test_tiny_fp32_pipeline_closed_half():
    _pipeline(wl.CONFIGS["tiny"])


def test_tiny_fp32_pipeline_geometric_capped():
    _pipeline(wl.with_budget(wl.CONFIGS["tiny"], kind=wl.GEOMETRIC, param=0.5), with_current=True, delta_t=4)


@pytest.mark.parametrize("impl", [0, 1])
def test_small_bf16_pipeline(impl):
    _pipeline(wl.small_bf16(), impl=impl)


@pytest.mark.parametrize("impl", [0, 1])
def test_small_bf16_pipeline_with_current_and_rebase(impl):
    _pipeline(wl.small_bf16(n_frames=3, grid=(11, 13), n_text=130, total=260, kind=wl.LINEAR, param=0.0, keep_full=0,
                            seed=5), impl=impl, with_current=True, delta_t=8)


def test_unlimited_budget_equals_full_cache_attention():
    cfg = wl.with_budget(wl.small_bf16(n_frames=2, grid=(8, 9)), total=10 ** 6, keep_full=0)
    L = wl.make_layer(cfg, with_current=True)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    assert budget.tolist() == L.frame_count.tolist()
    _, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    assert sel.cpu().numpy().tolist() == list(range(cfg.n_src))
    dst = D.empty_packed(cfg.n_src)
    pc.pc_compact(ctx, D.cache, sel, budget, 0, dst)
    a = pc.pc_attend_frame(ctx, dst, D.current, D.q, D.q_pos)
    b = pc.pc_attend_frame(ctx, D.cache, D.current, D.q, D.q_pos)
    _ok(ctx)
    assert torch.equal(a, b)
    k = np.concatenate([L.anchor_k, L.hist_k, L.cur_k]); v = np.concatenate([L.anchor_v, L.hist_v, L.cur_v])
    pos = np.concatenate([L.anchor_pos, L.hist_pos, L.q_pos])
    n = cfg.frame_tokens
    block = np.concatenate([np.zeros(cfg.n_text), np.ones(n)] + [np.full(n, 2 + f) for f in range(cfg.n_frames + 1)])
    q_all = np.zeros((len(k),) + L.q.shape[1:], np.float32)
    q_all[-cfg.n_q:] = L.q
    full = oracle.full_block_causal_attention(q_all, k, v, pos, block.astype(np.int32))[-cfg.n_q:]
    assert np.abs(host(a) - full).max() <= BF16_ATOL


# ------------------------------------------------------------------------------------------- split-KV merge
@pytest.mark.parametrize("cluster", [True, False])
def test_attention_key_ranges_merge_like_one_range(cluster):
    """Every split count (1-4 key ranges), merged inside the kernel through cluster shared memory or by the separate
    merge kernel, against the oracle; anchors and history of ragged length, with and without the current frame."""
    cfg = wl.small_bf16(n_frames=4, grid=(12, 21), n_text=130, total=700, keep_full=1, seed=11)
    L = wl.make_layer(cfg, with_current=True)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    pc.pc_set_cluster_merge(ctx, cluster)
    segs = [(L.anchor_k, L.anchor_v, L.anchor_pos), (L.hist_k, L.hist_v, L.hist_pos), (L.cur_k, L.cur_v, L.q_pos)]
    want, want_lse = oracle.attend(L.q, L.q_pos, segs, cfg.rope_base, want_lse=True)
    outs = []
    for n in (1, 2, 3, 4):
        pc.pc_set_kv_splits(ctx, n)
        out, lse = pc.pc_attend_frame(ctx, D.cache, D.current, D.q, D.q_pos, want_lse=True)
        _ok(ctx)
        assert np.abs(host(out).astype(np.float64) - want).max() <= BF16_ATOL
        assert np.abs(host(lse) - want_lse).max() <= 2e-2
        outs.append(host(out))
    for o in outs[1:]:                       # the split only changes fp32 rounding order: at most a bf16 ulp or two
        assert (np.abs(o - outs[0]) <= 2.0 ** -6 * np.maximum(np.abs(outs[0]), 0.5)).all()
    ctx.close()


# ------------------------------------------------------------------------------------------- prepared key set
@pytest.mark.parametrize("cfg_name", ["tiny", "small_bf16"])
def test_prepared_attention_equals_attend_frame_over_several_passes(cfg_name):
    """A frame generated over several passes: the key set is prepared once (keys rotated once), each pass brings its own
    queries.  Every pass must reproduce pc_attend_frame on the same inputs bit for bit, and match the oracle."""
    cfg = wl.CONFIGS["tiny"] if cfg_name == "tiny" else wl.small_bf16(n_frames=3, grid=(11, 13), n_text=130, total=260, seed=4)
    L = wl.make_layer(cfg, with_current=True)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    with pytest.raises(pc.PackCacheError):
        pc.pc_attend_prepared(ctx, D.q, D.q_pos)                       # nothing prepared yet
    pc.pc_attend_prepare(ctx, D.cache, D.current)
    rng = np.random.default_rng(3)
    segs = [(L.anchor_k, L.anchor_v, L.anchor_pos), (L.hist_k, L.hist_v, L.hist_pos), (L.cur_k, L.cur_v, L.q_pos)]
    passes = []
    for step in range(3):
        q = wl.to_storage(rng.standard_normal(L.q.shape).astype(np.float32), cfg.dtype)
        qd = dev(q, cfg.dtype)
        got, lse = pc.pc_attend_prepared(ctx, qd, D.q_pos, want_lse=True)
        want = oracle.attend(q, L.q_pos, segs, cfg.rope_base)
        _check_attention(cfg, host(got).astype(np.float64), want)
        passes.append((qd, got.clone(), lse.clone()))
    _ok(ctx)
    for qd, got, lse in passes:                                        # the one-call form gives the same bits
        ref, ref_lse = pc.pc_attend_frame(ctx, D.cache, D.current, qd, D.q_pos, want_lse=True)
        assert torch.equal(ref, got) and torch.equal(ref_lse, lse)
    if cfg.dtype == wl.BF16:
        with pytest.raises(pc.PackCacheError):                         # pc_attend_frame reused the scratch: prepare again
            pc.pc_attend_prepared(ctx, D.q, D.q_pos)
    ctx.close()


# ------------------------------------------------------------------------------------------- CUDA graph
@pytest.mark.parametrize("fused", [False, True])
def test_frame_step_replays_from_a_cuda_graph(fused):
    """Three layers' frame steps (score, select, pack, attend, launched with programmatic dependencies: eight kernels
    each through the three separate calls, six through the fused step with one context per layer) captured once into a
    CUDA graph.  A replay must give the bits of the eager calls, also after the inputs were overwritten in place (a
    new frame's queries and history in the same buffers)."""
    cfgs = [wl.small_bf16(n_frames=4, grid=(12, 21), n_text=130, total=500, keep_full=1, seed=30 + i) for i in range(3)]
    Ls = [wl.make_layer(c) for c in cfgs]
    Ds = [DeviceLayer(L) for L in Ls]
    cfg = cfgs[0]
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    n_sel = int(budget.sum())
    scores = torch.empty(cfg.n_src, dtype=torch.float32, device="cuda")
    sel = torch.empty(n_sel, dtype=torch.int32, device="cuda")
    dsts = [D.empty_packed(n_sel) for D in Ds]
    outs = [torch.empty_like(D.q) for D in Ds]

    ctxs = [ctx] + [make_ctx(cfg) for _ in Ds[1:]]

    def frame(stream):
        for D, dst, out, c in zip(Ds, dsts, outs, ctxs):
            if fused:
                pc.pc_frame_step(c, D.cache, budget, 0, dst, D.q, D.q_pos, scores=scores, sel_idx=sel, out=out, stream=stream)
            else:
                pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget, scores=scores, sel_idx=sel, stream=stream)
                pc.pc_compact(ctx, D.cache, sel, budget, 0, dst, stream=stream)
                pc.pc_attend_frame(ctx, dst, None, D.q, D.q_pos, out=out, stream=stream)

    frame(torch.cuda.current_stream())                              # warm-up: one-time attribute and occupancy queries
    torch.cuda.synchronize()
    eager = [o.clone() for o in outs]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        frame(torch.cuda.current_stream())
    for o in outs:
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for c in ctxs:
        _ok(c)
    for o, e in zip(outs, eager):
        assert torch.equal(o, e)
    want = oracle.attend(Ls[1].q, Ls[1].q_pos, [(Ls[1].anchor_k, Ls[1].anchor_v, Ls[1].anchor_pos),
                                                tuple(host(t) if t.dtype != torch.int32 else t.cpu().numpy()
                                                      for t in (dsts[1].history.k[:n_sel], dsts[1].history.v[:n_sel], dsts[1].history.pos[:n_sel]))],
                         cfg.rope_base)
    assert np.abs(host(outs[1]).astype(np.float64) - want).max() <= BF16_ATOL
    # new contents in the same buffers: layers swap their queries and history
    for a, b in ((0, 1), (1, 2)):
        for name in ("q",):
            ta, tb = getattr(Ds[a], name), getattr(Ds[b], name)
            tmp = ta.clone(); ta.copy_(tb); tb.copy_(tmp)
        ha, hb = Ds[a].cache.history, Ds[b].cache.history
        for ta, tb in ((ha.k, hb.k), (ha.v, hb.v)):
            tmp = ta.clone(); ta.copy_(tb); tb.copy_(tmp)
    graph.replay()
    torch.cuda.synchronize()
    replayed = [o.clone() for o in outs]
    frame(torch.cuda.current_stream())
    torch.cuda.synchronize()
    for c in ctxs:
        _ok(c)
    for o, e in zip(outs, replayed):
        assert torch.equal(o, e)
    assert not torch.equal(replayed[0], eager[0])
    for c in ctxs:
        c.close()


# ------------------------------------------------------------------------------------------- select
def _select_case(frame_count, budget, scores, cfg=None):
    cfg = cfg or wl.CONFIGS["tiny"]
    ctx = make_ctx(cfg, max_keys=max(int(np.sum(frame_count)), 1) + 16)
    n = int(np.sum(frame_count))
    z = torch.zeros((max(n, 1), cfg.n_kv_heads, cfg.head_dim), device="cuda")
    cache = pc.Cache(pc.Segment.empty(), pc.Segment(z, z, torch.zeros((max(n, 1), 4), dtype=torch.int32, device="cuda"), n),
                     np.asarray(frame_count, np.int32))
    _, sel = pc.pc_score(ctx, cache, None, None, budget, scores_override=torch.from_numpy(scores).cuda())
    _ok(ctx)
    want = oracle.select(scores, frame_count, budget)
    assert sel.cpu().numpy()[:len(want)].tolist() == want.tolist()
    ctx.close()


def test_select_ties_and_edges():
    rng = np.random.default_rng(0)
    for trial in range(12):
        F = int(rng.integers(1, 9))
        fc = rng.integers(0, 1700, size=F)
        if trial == 0:
            fc[0] = 0
        bud = np.array([int(rng.integers(0, n + 1)) for n in fc])
        if trial % 3 == 0:
            bud[-1] = fc[-1]
        if trial % 4 == 0:
            bud[0] = 0
        n = int(fc.sum())
        if n == 0:
            continue
        s = wl.tie_scores(rng, n) if trial % 2 else rng.standard_normal(n).astype(np.float32)
        if trial % 5 == 0:
            s[rng.random(n) < 0.2] = -np.inf
        _select_case(fc, bud, s)


def test_select_all_equal_and_tiny_values():
    _select_case([1008], [300], np.zeros(1008, np.float32))
    s = np.full(600, 1e-40, np.float32)            # denormals and signed zeros keep their order
    s[::3] = -1e-40
    s[1::7] = -0.0
    s[2::11] = 0.0
    _select_case([600], [333], s)


def test_select_full_size_headline_shape():
    cfg = wl.CONFIGS["lumos47"]
    rng = np.random.default_rng(1)
    fc = [cfg.frame_tokens] * cfg.n_frames
    budget = _plan(cfg)
    _select_case(fc, budget, rng.standard_normal(cfg.n_src).astype(np.float32), cfg)
    _select_case(fc, budget, wl.tie_scores(rng, cfg.n_src, levels=41), cfg)


# ------------------------------------------------------------------------------------------- score
def test_score_valid_mask_and_pooling_at_scale():
    cfg = wl.small_bf16(n_frames=4, grid=(12, 21), total=300, keep_full=0)
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    valid = (np.random.default_rng(0).random(cfg.n_src) < 0.7).astype(np.uint8)
    scores, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget, valid=torch.from_numpy(valid).cuda())
    _ok(ctx)
    ref = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, valid=valid)
    got = host(scores).astype(np.float64)
    assert np.array_equal(np.isneginf(got), valid == 0)
    m = valid == 1
    assert (np.abs(got[m] - ref[m]) <= score_tolerance(ref, L.frame_count)[m]).all()
    _valid_topk(host(scores), sel.cpu().numpy()[:budget.sum()], L.frame_count, budget)
    assert valid[sel.cpu().numpy()[:budget.sum()]].all()       # budgets fit inside the valid tokens here
    ctx.close()


@pytest.mark.parametrize("heads", [(96, 8), (48, 16), (32, 8)])
def test_score_with_wide_query_rows(heads):
    """The query pass keeps a token's rotated row in shared memory as fp32: 96 heads x 128 is exactly 48 KB, the most a
    launch gets without asking for more (the block's own static words come on top); 48 and 32 heads sit below."""
    from dataclasses import replace
    cfg = replace(wl.small_bf16(n_frames=2, grid=(5, 7), n_text=20, total=30, keep_full=0, seed=41), n_q_heads=heads[0], n_kv_heads=heads[1])
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    scores, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    _ok(ctx)
    ref = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)
    assert (np.abs(host(scores)[:cfg.n_src].astype(np.float64) - ref) <= score_tolerance(ref, L.frame_count)).all()
    _valid_topk(host(scores)[:cfg.n_src], sel.cpu().numpy()[:budget.sum()], L.frame_count, budget)
    ctx.close()


# ------------------------------------------------------------------------------------------- errors
def test_host_detected_errors():
    cfg = wl.CONFIGS["tiny"]
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    bad = budget.copy(); bad[0] = cfg.frame_tokens + 1
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_score(ctx, D.cache, D.q, D.q_pos, bad)
    assert e.value.status == pc.PC_ERR_BUDGET
    _, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_compact(ctx, D.cache, sel, budget, 0, D.empty_packed(int(budget.sum()) - 1))
    assert e.value.status == pc.PC_ERR_CAPACITY
    with pytest.raises(pc.PackCacheError) as e:                   # destination aliases the source
        pc.pc_compact(ctx, D.cache, sel, budget, 0, D.cache)
    assert e.value.status == pc.PC_ERR_INVALID_ARG
    with pytest.raises(pc.PackCacheError) as e:                   # misaligned query pointer
        shifted = torch.zeros(D.q.numel() + 4, device="cuda")[1:1 + D.q.numel()].view(D.q.shape)
        pc.pc_attend_frame(ctx, D.cache, None, shifted, D.q_pos, out=torch.empty_like(D.q))
    assert e.value.status == pc.PC_ERR_INVALID_ARG
    wrong = pc.Cache(D.cache.anchors, D.cache.history, np.array([64] * 5, np.int32))   # frame table does not sum up
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_score(ctx, wrong, D.q, D.q_pos, budget[:5])
    assert e.value.status == pc.PC_ERR_INVALID_ARG
    small = make_ctx(cfg, max_keys=100)
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_attend_frame(small, D.cache, None, D.q, D.q_pos)
    assert e.value.status == pc.PC_ERR_CAPACITY
    with pytest.raises(pc.PackCacheError):
        pc.Context(5, 2, 64, pc.PC_F32, 10000.0, (8, 8, 8), 8, 8)
    with pytest.raises(pc.PackCacheError):
        pc.Context(4, 2, 48, pc.PC_F32, 10000.0, (8, 8, 8), 8, 8)
    # key rows the scoring kernels are not built for are refused by the call, with nothing enqueued:
    # 32 KV heads x 128 bf16 = 8192 bytes, 5 x 128 bf16 = 1280 bytes (not a multiple of 512), 1 x 128 bf16 = 256 bytes
    for hq, hkv in [(32, 32), (5, 5), (2, 1)]:
        odd = pc.Context(hq, hkv, 128, pc.PC_BF16, 10000.0, (64, 64, 64), 8, 64)
        k = torch.zeros((16, hkv, 128), dtype=torch.bfloat16, device="cuda")
        q = torch.zeros((8, hq, 128), dtype=torch.bfloat16, device="cuda")
        pos = torch.zeros((16, 4), dtype=torch.int32, device="cuda")
        cache = pc.Cache(pc.Segment.empty(), pc.Segment(k, k.clone(), pos, 16), [16])
        with pytest.raises(pc.PackCacheError) as e:
            pc.pc_score(odd, cache, q, pos[:8], np.array([4], np.int32))
        assert e.value.status == pc.PC_ERR_UNSUPPORTED and pc.pc_poll_status(odd) == pc.PC_OK
        odd.close()
    _ok(ctx)


def test_device_side_checks_record_instead_of_faulting():
    cfg = wl.CONFIGS["tiny"]
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    _, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    _ok(ctx)
    # an index outside the source is recorded and its row skipped
    bad_sel = sel.clone(); bad_sel[3] = cfg.n_src + 100
    dst = D.empty_packed(int(budget.sum()), poison=9.0)
    pc.pc_compact(ctx, D.cache, bad_sel, budget, 0, dst)
    assert pc.pc_poll_status(ctx) == pc.PC_ERR_INVALID_ARG
    assert (host(dst.history.k)[3] == 9.0).all()
    assert pc.pc_poll_status(ctx) == pc.PC_OK                     # polling clears the word
    # a position outside the rotary tables is recorded (and clamped)
    tight = make_ctx(cfg, max_pos=(16, 16, 16))
    pc.pc_score(tight, D.cache, D.q, D.q_pos, budget)
    assert pc.pc_poll_status(tight) == pc.PC_ERR_INVALID_ARG
    pc.pc_attend_frame(tight, D.cache, None, D.q, D.q_pos)
    assert pc.pc_poll_status(tight) == pc.PC_ERR_INVALID_ARG
    # NaN scores are an error for selection
    s = np.zeros(cfg.n_src, np.float32); s[5] = np.nan
    pc.pc_score(ctx, D.cache, None, None, budget, scores_override=torch.from_numpy(s).cuda())
    assert pc.pc_poll_status(ctx) == pc.PC_ERR_INVALID_ARG


# ------------------------------------------------------------------------------------------- full size
@pytest.mark.parametrize("name", ["lumos12", "lumos24", "lumos47"])
def test_full_size_sampled_against_oracle(name):
    """The benchmark's launch configuration at full size: scores against the pooled fp64 oracle on every token and
    the mean-logit oracle on a sample; selection and packing bit-exact; attention on sampled (query, head) rows."""
    cfg = wl.CONFIGS[name]
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    rng = np.random.default_rng(0)

    scores, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    got = host(scores).astype(np.float64)
    ref = oracle.score_pooled(L.hist_k, L.hist_pos, L.q, L.q_pos)
    tol = score_tolerance(ref, L.frame_count)
    assert (np.abs(got - ref) <= tol).all()
    idx = rng.choice(cfg.n_src, size=24, replace=False)
    naive = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, idx=idx)
    assert (np.abs(got[idx] - naive) <= tol[idx]).all()
    _valid_topk(host(scores), sel.cpu().numpy(), L.frame_count, budget)

    ref32 = ref.astype(np.float32)
    _, sel2 = pc.pc_score(ctx, D.cache, None, None, budget, scores_override=torch.from_numpy(ref32).cuda())
    want_sel = oracle.select(ref32, L.frame_count, budget)
    assert np.array_equal(sel2.cpu().numpy(), want_sel)

    dst = D.empty_packed(int(budget.sum()))
    pc.pc_compact(ctx, D.cache, sel2, budget, 0, dst)
    wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, want_sel, 0)
    assert np.array_equal(host(dst.history.k), wk) and np.array_equal(host(dst.history.v), wv)
    assert np.array_equal(dst.history.pos.cpu().numpy(), wp)

    out, lse = pc.pc_attend_frame(ctx, dst, None, D.q, D.q_pos, want_lse=True)
    _ok(ctx)
    if name == "lumos47":
        # the benchmark's configuration: every (query, head) row, so that every (row tile, head, key range) of the launch
        # the bench times is compared (the oracle takes about 11 s for them on 16 cores)
        rows = np.stack(np.meshgrid(np.arange(cfg.n_q), np.arange(cfg.n_q_heads), indexing="ij"), axis=-1).reshape(-1, 2)
        rows = rows.astype(np.int32)
    else:
        # one row of every (row tile, head) and a random sample on top
        tiles = [(min(t * 128 + int(rng.integers(128)), cfg.n_q - 1), h) for t in range((cfg.n_q + 127) // 128)
                 for h in range(cfg.n_q_heads)]
        rand = np.stack([rng.integers(0, cfg.n_q, size=96), rng.integers(0, cfg.n_q_heads, size=96)], axis=1)
        rows = np.concatenate([np.array(tiles), rand]).astype(np.int32)
        rows[0] = (0, 0); rows[1] = (cfg.n_q - 1, cfg.n_q_heads - 1); rows[2] = (1007, 5); rows[3] = (896, 23)
    want, want_lse = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)], rows=rows,
                                   want_lse=True)
    o = host(out)
    check_bf16_attention(o[rows[:, 0], rows[:, 1]], want)
    assert np.abs(host(lse)[rows[:, 0], rows[:, 1]] - want_lse).max() <= 2e-2
    assert np.isfinite(o).all()
    ctx.close()


def test_full_cache_comparator_at_24_frames():
    """Attention over the uncompacted cache (anchors ++ all 24 history frames, 25,328 keys): the comparator the
    24-frame configuration is measured against, on sampled (query, head) rows."""
    cfg = wl.CONFIGS["lumos24"]
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    out, lse = pc.pc_attend_frame(ctx, D.cache, None, D.q, D.q_pos, want_lse=True)
    _ok(ctx)
    rng = np.random.default_rng(2)
    # one row of every (row tile, head), so that every tile / head / key-range combination of the launch is compared
    rows = np.array([(min(t * 128 + int(rng.integers(128)), cfg.n_q - 1), h) for t in range((cfg.n_q + 127) // 128)
                     for h in range(cfg.n_q_heads)], dtype=np.int32)
    rows[0] = (0, 0); rows[1] = (cfg.n_q - 1, cfg.n_q_heads - 1)
    want, want_lse = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (L.hist_k, L.hist_v, L.hist_pos)],
                                   rows=rows, want_lse=True)
    o = host(out)
    check_bf16_attention(o[rows[:, 0], rows[:, 1]], want)
    assert np.abs(host(lse)[rows[:, 0], rows[:, 1]] - want_lse).max() <= 2e-2
    assert np.isfinite(o).all()
    ctx.close()


@pytest.mark.parametrize("layer,frac,kind,param", [(3, 0.10, wl.HALFLIFE, 2.0), (17, 0.50, wl.LINEAR, 0.0),
                                                   (27, 1.00, wl.HALFLIFE, 8.0)])
def test_layer_stack_cells_sampled(layer, frac, kind, param):
    """Cells of the 28-layer sweep (layer, budget fraction, decay): each layer has its own seeded tensors; budgets
    bit-exact, selection and packing bit-exact on the oracle's scores, attention on sampled rows."""
    base = wl.CONFIGS["stack28"]
    cfg = wl.with_budget(base, kind=kind, param=param, total=int(frac * base.n_src), keep_full=0)
    L = wl.make_layer(cfg, layer=layer)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    budget = _plan(cfg)
    assert budget.sum() == min(cfg.budget.total, cfg.n_src)
    scores, sel = pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget)
    ref = oracle.score_pooled(L.hist_k, L.hist_pos, L.q, L.q_pos)
    assert (np.abs(host(scores).astype(np.float64) - ref) <= score_tolerance(ref, L.frame_count)).all()
    _valid_topk(host(scores), sel.cpu().numpy(), L.frame_count, budget)
    ref32 = ref.astype(np.float32)
    _, sel2 = pc.pc_score(ctx, D.cache, None, None, budget, scores_override=torch.from_numpy(ref32).cuda())
    want_sel = oracle.select(ref32, L.frame_count, budget)
    assert np.array_equal(sel2.cpu().numpy()[:len(want_sel)], want_sel)
    dst = D.empty_packed(int(budget.sum()))
    pc.pc_compact(ctx, D.cache, sel2, budget, 0, dst)
    wk, wv, wp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, want_sel, 0)
    assert np.array_equal(host(dst.history.k), wk) and np.array_equal(dst.history.pos.cpu().numpy(), wp)
    out = pc.pc_attend_frame(ctx, dst, None, D.q, D.q_pos)
    _ok(ctx)
    rng = np.random.default_rng(layer)
    rows = np.stack([rng.integers(0, cfg.n_q, size=32), rng.integers(0, cfg.n_q_heads, size=32)], axis=1).astype(np.int32)
    want = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (wk, wv, wp)], rows=rows)
    check_bf16_attention(host(out)[rows[:, 0], rows[:, 1]], want)
    ctx.close()
