"""Pins for the CPU oracle: each check compares it with something other than itself —
the paper's printed allocation pattern, closed forms and identities, exact rational
arithmetic, brute force, or numpy/scipy routines written in a different formulation."""
from __future__ import annotations

import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2601_04359_b200 import workload as wl
from tests import npref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
BIG = 1 << 20


# --------------------------------------------------------------------------- plan
def _pattern():
    rows = {}
    for line in open(os.path.join(GOLDEN, "allocation_pattern.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w, fr = line.split(":")
        rows[int(w)] = [Fraction(x) for x in fr.split()]
    return rows


def test_plan_matches_printed_pattern():
    # Eq. 7's displayed pattern, scaled by a budget it divides exactly (Eq. 8: t_d = B_one * b_d)
    for W, fr in _pattern().items():
        assert sum(fr) == 1
        for B in (64, 128, 1024):
            t = oracle.plan_budget(oracle.CLOSED_HALF, 0.5, B, 0, [BIG] * W)
            want = [int(B * f) for f in fr][::-1]          # oracle frames are oldest -> newest
            assert t.tolist() == want


def test_plan_tiny_config_worked_example():
    cfg = wl.CONFIGS["tiny"]
    t = oracle.plan_budget(cfg.budget.kind, cfg.budget.param, cfg.budget.total, 0, [64] * 6)
    assert t.tolist() == [4, 4, 8, 16, 32, 64]              # 128 * [1/32, 1/32, 1/16, 1/8, 1/4, 1/2]


def _hamilton(weights, B, avail):
    """Largest-remainder apportionment in exact rationals, with capping; d=1 first."""
    W = len(weights)
    t = [0] * W
    active = set(range(W))
    B = min(B, sum(avail))
    while active and B > 0:
        S = sum(weights[i] for i in active)
        if B >= sum(avail[i] for i in active):
            for i in active:
                t[i] = avail[i]
            break
        quota = {i: Fraction(B) * weights[i] / S for i in active}
        for i in active:
            t[i] = int(quota[i])                           # floor (non-negative)
        left = B - sum(t[i] for i in active)
        order = sorted(active, key=lambda i: (-(quota[i] - int(quota[i])), i))   # ties: nearer first
        for i in order[:left]:
            t[i] += 1
        over = [i for i in active if t[i] > avail[i]]
        if not over:
            break
        for i in over:
            t[i] = avail[i]
            B -= avail[i]
            active.discard(i)
        for i in active:
            t[i] = 0
    return t


@pytest.mark.parametrize("W", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("B", [0, 1, 7, 100, 129, 1000])
def test_plan_equals_exact_rational_apportionment(W, B):
    N = 64
    cases = {
        oracle.GEOMETRIC: (0.5, [Fraction(1, 2) ** d for d in range(1, W + 1)]),
        oracle.CLOSED_HALF: (0.5, [Fraction(1, 2) ** min(d, W - 1) for d in range(1, W + 1)]),
        oracle.LINEAR: (0.0, [Fraction(W + 1 - d) for d in range(1, W + 1)]),
        oracle.HALFLIFE: (1.0, [Fraction(1, 2) ** (d - 1) for d in range(1, W + 1)]),
    }
    for kind, (param, wts) in cases.items():
        got = oracle.plan_budget(kind, param, B, 0, [N] * W).tolist()[::-1]   # nearest first
        assert got == _hamilton(wts, B, [N] * W), (kind, W, B)


def _q32_halflife_weights(W, keep_full, half_life):
    """floor(2^-((d - 1 - keep_full)/h) * 2^32 + 1/2) for d = keep_full + 1 .. W, in 60-digit decimal arithmetic."""
    from decimal import ROUND_FLOOR, Decimal, getcontext
    getcontext().prec = 60
    out = []
    for d in range(keep_full + 1, W + 1):
        g = Decimal(2) ** (Decimal(-(d - 1 - keep_full)) / Decimal(half_life))
        out.append(int((g * (1 << 32) + Decimal("0.5")).to_integral_value(rounding=ROUND_FLOOR)))
    return out


def test_plan_of_the_benchmark_configurations_by_exact_arithmetic():
    """The budget vectors of the measured configurations (12 frames linear at 25 %; 24 frames at half-life 4; 47 frames
    with the two newest whole and 6048 tokens at half-life 4; 47 frames at 10 % and half-life 2) against largest-remainder
    apportionment in exact integers / rationals over weights quantised once to 2^-32."""
    N = 1008
    got = oracle.plan_budget(oracle.LINEAR, 0.0, (12 * N) // 4, 0, [N] * 12).tolist()[::-1]
    assert got == _hamilton([Fraction(13 - d) for d in range(1, 13)], (12 * N) // 4, [N] * 12)
    assert got[0] == 465 and got[-1] == 39                              # 3024 * 12/78 and 3024 * 1/78, rounded by remainder
    got = oracle.plan_budget(oracle.HALFLIFE, 4.0, 6048, 0, [N] * 24).tolist()[::-1]
    assert got == _hamilton([Fraction(w) for w in _q32_halflife_weights(24, 0, 4)], 6048, [N] * 24)
    got = oracle.plan_budget(oracle.HALFLIFE, 4.0, 2 * N + 6048, 2, [N] * 47).tolist()[::-1]
    tail = _hamilton([Fraction(w) for w in _q32_halflife_weights(47, 2, 4)], 6048, [N] * 45)
    assert got == [N, N] + tail and sum(got) == 8064 and sum(1 for t in got if t) == 46
    got = oracle.plan_budget(oracle.HALFLIFE, 2.0, (47 * N) // 10, 0, [N] * 47).tolist()[::-1]
    assert got == _hamilton([Fraction(w) for w in _q32_halflife_weights(47, 0, 2)], (47 * N) // 10, [N] * 47)
    assert got[:2] == [N, N] and sum(1 for t in got if t) == 24          # the two nearest frames are capped, the surplus re-shared


def test_plan_identities():
    rng = np.random.default_rng(1)
    for kind, param in [(oracle.GEOMETRIC, 0.7), (oracle.GEOMETRIC, 0.5), (oracle.LINEAR, 0.0),
                        (oracle.HALFLIFE, 4.0), (oracle.HALFLIFE, 2.0), (oracle.CLOSED_HALF, 0.5)]:
        for W in (1, 3, 12, 24, 47):
            for B in (0, 5, 1008, 3024, 6048, 47 * 1008, 10 ** 6):
                t = oracle.plan_budget(kind, param, B, 0, [1008] * W)
                assert t.sum() == min(B, 1008 * W)                     # Eq. 8: the shares sum to the total
                assert (t >= 0).all() and (t <= 1008).all()
                assert (np.diff(t) >= 0).all()                         # never more for a farther frame
    # ragged availability: still sums, still within what each frame holds
    for _ in range(20):
        W = int(rng.integers(1, 10))
        avail = rng.integers(0, 50, size=W)
        B = int(rng.integers(0, 300))
        t = oracle.plan_budget(oracle.GEOMETRIC, 0.6, B, 0, avail)
        assert t.sum() == min(B, avail.sum()) and (t <= avail).all()


def test_plan_quota_property_follows_eq6():
    # without capping each t_d is within one token of B * g(d) / sum_j g(j)  (Eq. 6 and Eq. 8)
    W, B = 12, 3000
    for kind, param, g in [(oracle.GEOMETRIC, 0.8, lambda d: 0.8 ** d),
                           (oracle.LINEAR, 0.0, lambda d: W + 1 - d),
                           (oracle.HALFLIFE, 3.0, lambda d: 2.0 ** (-(d - 1) / 3.0))]:
        t = oracle.plan_budget(kind, param, B, 0, [BIG] * W)[::-1]
        gs = np.array([g(d) for d in range(1, W + 1)], dtype=np.float64)
        assert np.abs(t - B * gs / gs.sum()).max() < 1.0


def test_plan_halflife_halves():
    t = oracle.plan_budget(oracle.HALFLIFE, 4.0, 200000, 0, [BIG] * 24)[::-1]
    ratio = t[4:] / t[:-4]
    assert np.abs(ratio - 0.5).max() < 2e-3                            # mu_{d+h} = mu_d / 2


def test_plan_keep_full_and_errors():
    t = oracle.plan_budget(oracle.HALFLIFE, 4.0, 2 * 1008 + 6048, 2, [1008] * 47)
    assert t[-2:].tolist() == [1008, 1008] and t.sum() == 8064
    assert t[:-2].sum() == 6048 and (np.diff(t[:-2]) >= 0).all()
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(oracle.HALFLIFE, 4.0, 1000, 2, [1008] * 5)   # kept-whole frames exceed the total
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(oracle.GEOMETRIC, 1.5, 10, 0, [5] * 3)


def test_plan_caps_and_reshares():
    # normalised geometric 1/2 on 6 frames of 64 gives the nearest frame 65 > 64: capped, surplus re-shared
    t = oracle.plan_budget(oracle.GEOMETRIC, 0.5, 128, 0, [64] * 6)[::-1]
    assert t[0] == 64 and t.sum() == 128 and (np.diff(t) <= 0).all()


# --------------------------------------------------------------------------- rope
def test_rope_against_complex_rotation():
    rng = np.random.default_rng(0)
    for d in (64, 128, 6, 2):
        x = rng.standard_normal(d).astype(np.float32)
        pos = [int(v) for v in rng.integers(0, 400, size=3)]
        want = npref.rope_np(x[None, None, :], np.array([pos + [0]]))[0, 0]
        np.testing.assert_allclose(oracle.rope(x, pos), want, rtol=0, atol=1e-12)


def test_rope_textbook_1d_when_one_axis_moves():
    # with only t non-zero, the pairs on the t axis follow 1D rotary with n_t frequencies; others are untouched
    d, base, t = 128, 10000.0, 37
    x = np.random.default_rng(2).standard_normal(d).astype(np.float32)
    y = oracle.rope(x, [t, 0, 0], base)
    n_t = len(range(0, d // 2, 3))
    for i in range(d // 2):
        x0, x1 = float(x[2 * i]), float(x[2 * i + 1])
        if i % 3 == 0:
            ang = t * base ** (-(i // 3) / n_t)
            assert abs(y[2 * i] - (x0 * np.cos(ang) - x1 * np.sin(ang))) < 1e-12
            assert abs(y[2 * i + 1] - (x0 * np.sin(ang) + x1 * np.cos(ang))) < 1e-12
        else:
            assert y[2 * i] == x0 and y[2 * i + 1] == x1


def test_rope_identity_norm_and_relativity():
    rng = np.random.default_rng(3)
    d = 64
    q, k = rng.standard_normal(d).astype(np.float32), rng.standard_normal(d).astype(np.float32)
    assert np.array_equal(oracle.rope(q, [0, 0, 0]), q.astype(np.float64))
    pq, pk, sh = np.array([5, 16, 24]), np.array([1, 40, 8]), np.array([11, 3, 29])
    assert abs(np.linalg.norm(oracle.rope(q, pq)) - np.linalg.norm(q.astype(np.float64))) < 1e-12
    a = oracle.rope(q, pq) @ oracle.rope(k, pk)
    b = oracle.rope(q, pq + sh) @ oracle.rope(k, pk + sh)
    assert abs(a - b) < 1e-11                      # logits depend on position differences only
    c = oracle.rope(q, pq + [1, 0, 0]) @ oracle.rope(k, pk)
    assert abs(a - c) > 1e-6                       # ... and do depend on them


# --------------------------------------------------------------------------- score
def _tiny_layer(seed=0, **kw):
    cfg = wl.CONFIGS["tiny"]
    from dataclasses import replace
    return wl.make_layer(replace(cfg, seed=seed, **kw), with_current=True)


def test_score_is_mean_logit():
    L = _tiny_layer()
    s = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos)
    want = npref.score_np(L.hist_k, L.hist_pos, L.q, L.q_pos)
    np.testing.assert_allclose(s, want, rtol=0, atol=1e-12)


def test_score_single_query_single_head_is_logit_row():
    L = _tiny_layer(seed=5)
    q1, k1 = L.q[:1, :1], L.hist_k[:, :1]
    s = oracle.score(k1, L.hist_pos, q1, L.q_pos[:1])
    lg = npref.logits_np(q1, L.q_pos[:1], k1, L.hist_pos)[0, 0]
    np.testing.assert_allclose(s, lg, rtol=0, atol=1e-12)


def test_score_pooled_identity_subset_and_mask():
    L = _tiny_layer(seed=7)
    s = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos)
    np.testing.assert_allclose(oracle.score_pooled(L.hist_k, L.hist_pos, L.q, L.q_pos), s, rtol=0, atol=1e-12)
    idx = np.array([3, 0, 200, 383])
    np.testing.assert_array_equal(oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, idx=idx), s[idx])
    valid = np.ones(len(s), np.uint8)
    valid[[1, 9]] = 0
    sm = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, valid=valid)
    assert np.isneginf(sm[[1, 9]]).all() and np.array_equal(np.delete(sm, [1, 9]), np.delete(s, [1, 9]))


# --------------------------------------------------------------------------- select
def _brute_select(scores, frame_count, budget):
    out, base = [], 0
    for n, t in zip(frame_count, budget):
        order = sorted(range(base, base + n), key=lambda j: (-float(scores[j]), j))
        out += sorted(order[:t])
        base += n
    return out


def test_select_matches_brute_force_sort():
    rng = np.random.default_rng(4)
    for trial in range(30):
        F = int(rng.integers(1, 6))
        fc = rng.integers(0, 40, size=F)
        bud = np.array([int(rng.integers(0, n + 1)) for n in fc])
        n = int(fc.sum())
        s = rng.standard_normal(n).astype(np.float32) if trial % 2 else wl.tie_scores(rng, n)
        assert oracle.select(s, fc, bud).tolist() == _brute_select(s, fc, bud)


def test_select_edge_cases():
    s = np.zeros(10, np.float32)
    s[3] = -0.0
    assert oracle.select(s, [10], [4]).tolist() == [0, 1, 2, 3]         # all equal: lowest indices, -0 == +0
    assert oracle.select(s, [10], [0]).tolist() == []
    assert oracle.select(s, [10], [10]).tolist() == list(range(10))
    s2 = np.array([1, -np.inf, 3, -np.inf, 2], np.float32)
    assert oracle.select(s2, [5], [3]).tolist() == [0, 2, 4]
    assert oracle.select(s2, [5], [4]).tolist() == [0, 1, 2, 4]
    with pytest.raises(oracle.OracleError):
        oracle.select(np.array([0, np.nan], np.float32), [2], [1])
    with pytest.raises(oracle.OracleError):
        oracle.select(s, [10], [11])


# --------------------------------------------------------------------------- pack
def test_pack_is_a_row_gather_with_rebase():
    L = _tiny_layer(seed=2)
    rng = np.random.default_rng(0)
    sel = np.sort(rng.choice(len(L.hist_k), size=100, replace=False)).astype(np.int32)
    dk, dv, dp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel, delta_t=8)
    assert np.array_equal(dk.view(np.uint32), L.hist_k[sel].view(np.uint32))
    assert np.array_equal(dv.view(np.uint32), L.hist_v[sel].view(np.uint32))
    assert np.array_equal(dp[:, 1:], L.hist_pos[sel][:, 1:])            # h, w, tag never change (Eq. 9)
    assert np.array_equal(dp[:, 0], L.hist_pos[sel][:, 0] - 8)
    assert np.array_equal(dp[:, 3], sel + wl.CONFIGS["tiny"].n_anchor)  # tags prove provenance


# --------------------------------------------------------------------------- attend
def test_attend_matches_library_softmax_attention():
    L = _tiny_layer(seed=1)
    k = np.concatenate([L.anchor_k, L.hist_k[:70]])
    v = np.concatenate([L.anchor_v, L.hist_v[:70]])
    p = np.concatenate([L.anchor_pos, L.hist_pos[:70]])
    out, lse = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos),
                                            (L.hist_k[:70], L.hist_v[:70], L.hist_pos[:70])], want_lse=True)
    want, want_lse = npref.attend_np(L.q, L.q_pos, k, v, p)
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)
    rows = np.array([[0, 0], [63, 3], [17, 2]], np.int32)
    sub = oracle.attend(L.q, L.q_pos, [(k, v, p)], rows=rows)
    np.testing.assert_allclose(sub, want[rows[:, 0], rows[:, 1]], rtol=0, atol=1e-12)


def test_attend_special_cases():
    L = _tiny_layer(seed=9)
    # one key: the output is that key's value row of the head's KV group
    out = oracle.attend(L.q, L.q_pos, [(L.hist_k[:1], L.hist_v[:1], L.hist_pos[:1])])
    G = L.q.shape[1] // L.hist_k.shape[1]
    for h in range(L.q.shape[1]):
        np.testing.assert_allclose(out[:, h], np.broadcast_to(L.hist_v[0, h // G], out[:, h].shape), atol=1e-15)
    # all-zero keys: uniform weights, the mean of the values; lse = log(n)
    zk = np.zeros_like(L.hist_k[:50])
    out, lse = oracle.attend(L.q, L.q_pos, [(zk, L.hist_v[:50], L.hist_pos[:50])], want_lse=True)
    np.testing.assert_allclose(out[5, 3], L.hist_v[:50, 3 // G].astype(np.float64).mean(axis=0), atol=1e-13)
    np.testing.assert_allclose(lse, np.log(50.0), atol=1e-13)
    # the key order does not matter
    perm = np.random.default_rng(0).permutation(120)
    a = oracle.attend(L.q, L.q_pos, [(L.hist_k[:120], L.hist_v[:120], L.hist_pos[:120])])
    b = oracle.attend(L.q, L.q_pos, [(L.hist_k[:120][perm], L.hist_v[:120][perm], L.hist_pos[:120][perm])])
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def _whole_sequence(L):
    cfg = L.cfg
    n = cfg.frame_tokens
    k = np.concatenate([L.anchor_k, L.hist_k, L.cur_k])
    v = np.concatenate([L.anchor_v, L.hist_v, L.cur_v])
    pos = np.concatenate([L.anchor_pos, L.hist_pos, L.q_pos])
    block = np.concatenate([np.zeros(cfg.n_text), np.ones(n)] +
                           [np.full(n, 2 + f) for f in range(cfg.n_frames + 1)]).astype(np.int32)
    return k, v, pos, block


def test_full_block_causal_attention_against_masked_softmax():
    L = _tiny_layer(seed=11)
    k, v, pos, block = _whole_sequence(L)
    rng = np.random.default_rng(0)
    q_all = rng.standard_normal((len(k),) + L.q.shape[1:]).astype(np.float32)
    out = oracle.full_block_causal_attention(q_all, k, v, pos, block)
    mask = block[None, :] <= block[:, None]            # inside a block both ways, causal between blocks (Eq. 2)
    want, _ = npref.attend_np(q_all, pos, k, v, pos, mask=mask)
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)


def test_unlimited_budget_compaction_equals_full_causal_attention():
    # plan -> score -> select -> pack -> attend with a budget that covers the whole history must equal
    # the current frame's rows of attention over the uncompacted sequence
    L = _tiny_layer(seed=13)
    cfg = L.cfg
    k, v, pos, block = _whole_sequence(L)
    q_all = np.zeros((len(k),) + L.q.shape[1:], np.float32)
    q_all[-cfg.n_q:] = L.q
    full = oracle.full_block_causal_attention(q_all, k, v, pos, block)[-cfg.n_q:]
    budget = oracle.plan_budget(oracle.GEOMETRIC, 0.5, 10 ** 9, 0, L.frame_count)
    assert budget.tolist() == L.frame_count.tolist()
    s = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos).astype(np.float32)
    sel = oracle.select(s, L.frame_count, budget)
    assert sel.tolist() == list(range(cfg.n_src))
    pk, pv, pp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel)
    out = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (pk, pv, pp),
                                       (L.cur_k, L.cur_v, L.q_pos)])
    np.testing.assert_allclose(out, full, rtol=0, atol=1e-12)


def test_anchors_survive_and_rebase_leaves_history_logits_unchanged():
    L = _tiny_layer(seed=17)
    cfg = L.cfg
    budget = oracle.plan_budget(cfg.budget.kind, cfg.budget.param, cfg.budget.total, 0, L.frame_count)
    s = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos).astype(np.float32)
    sel = oracle.select(s, L.frame_count, budget)
    assert len(sel) == 128 and (np.diff(sel) > 0).all()
    # the per-frame counts of the selection are the plan
    frame_of = sel // cfg.frame_tokens
    assert np.bincount(frame_of, minlength=cfg.n_frames).tolist() == budget.tolist()
    # shifting history and query by the same number of dropped frames leaves the history logits unchanged
    pk, pv, pp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel, delta_t=0)
    pk2, pv2, pp2 = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel, delta_t=8)
    qp2 = L.q_pos.copy()
    qp2[:, 0] -= 8
    a = oracle.attend(L.q, L.q_pos, [(pk, pv, pp)])
    b = oracle.attend(L.q, qp2, [(pk2, pv2, pp2)])
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-11)


# ------------------------------------------------------------------------------------------- minimum quota (b_min)
def _exact_plan_with_floor(weights, avail, total, m):
    """Exact-rational statement of the minimum-quota rule for frames listed nearest first: the nearest floor(B/m) frames
    take part, each is guaranteed min(m, avail), the rest is shared in proportion to the weights by largest remainder
    (ties to the nearer frame), capping at what a frame holds and re-sharing the surplus."""
    n = len(weights)
    part = list(range(n)) if m == 0 else list(range(min(n, total // m)))
    floor_q = [min(m, avail[i]) if i in part else 0 for i in range(n)]
    room = [avail[i] - floor_q[i] for i in range(n)]
    B = total - sum(floor_q)
    extra = [0] * n
    live = [i for i in part]
    while live and B > 0:
        if B >= sum(room[i] for i in live):
            for i in live:
                extra[i] = room[i]
            break
        S = sum(weights[i] for i in live)
        if S == 0:
            break
        share = {i: Fraction(B * weights[i], S) for i in live}
        for i in live:
            extra[i] = share[i].numerator // share[i].denominator
        left = B - sum(extra[i] for i in live)
        order = sorted(live, key=lambda i: (-(share[i] - extra[i]), i))      # largest remainder, then nearer frame
        for i in order[:left]:
            extra[i] += 1
        over = [i for i in live if extra[i] > room[i]]
        if not over:
            break
        for i in over:
            extra[i] = room[i]
            B -= room[i]
        live = [i for i in live if i not in over]
        for i in live:
            extra[i] = 0
    return [floor_q[i] + extra[i] for i in range(n)]


def test_plan_minimum_quota_against_exact_rationals():
    rng = np.random.default_rng(11)
    for _ in range(200):
        W = int(rng.integers(1, 9))
        avail = [int(x) for x in rng.integers(0, 90, size=W)]
        m = int(rng.integers(0, 40))
        total = int(rng.integers(0, sum(avail) + 40))
        got = oracle.plan_budget(oracle.LINEAR, 0.0, total, 0, avail, min_quota=m).tolist()
        near_first_w = [(W + 1 - d) << 32 for d in range(1, W + 1)]                # linear weights are exact in Q32
        want = _exact_plan_with_floor(near_first_w, avail[::-1], total, m)[::-1]
        assert got == want


def test_plan_minimum_quota_properties():
    n, W = 64, 6
    base = oracle.plan_budget(oracle.CLOSED_HALF, 0.5, 128, 0, [n] * W).tolist()
    assert oracle.plan_budget(oracle.CLOSED_HALF, 0.5, 128, 0, [n] * W, min_quota=0).tolist() == base
    # every frame that takes part keeps at least the quota; the total is unchanged; still non-increasing with distance
    q = oracle.plan_budget(oracle.CLOSED_HALF, 0.5, 128, 0, [n] * W, min_quota=8).tolist()
    assert q == [10, 11, 13, 18, 28, 48] and sum(q) == 128 and min(q) >= 8 and q == sorted(q)
    # guarantees beyond the budget: the window shrinks first in, first out (6 x 3 > 10: the three nearest frames stay)
    t = oracle.plan_budget(oracle.LINEAR, 0.0, 10, 0, [n] * W, min_quota=3).tolist()
    assert t == [0, 0, 0, 3, 3, 4]
    # a frame that holds less than the quota keeps what it holds; kept-whole frames are outside the rule
    u = oracle.plan_budget(oracle.HALFLIFE, 1.0, 100, 1, [2, 64, 64, 64, 64, 64], min_quota=5).tolist()
    assert u[0] == 2 and u[-1] == 64 and sum(u) == 100 and all(x >= 5 for x in u[1:-1])
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(oracle.LINEAR, 0.0, 10, 0, [5], min_quota=-1)


# ---------------------------------------------------------------------------------------------- attention mass (Sec. 3.4)
def test_attend_mass_matches_library_softmax():
    L = _tiny_layer(seed=4)
    k = np.concatenate([L.anchor_k, L.hist_k[:90]])
    p = np.concatenate([L.anchor_pos, L.hist_pos[:90]])
    got = oracle.attend_mass(L.q, L.q_pos, [(L.anchor_k, L.anchor_pos), (L.hist_k[:90], L.hist_pos[:90])])
    np.testing.assert_allclose(got, npref.attend_mass_np(L.q, L.q_pos, k, p), rtol=0, atol=1e-14)
    assert abs(got.sum() - 1.0) < 1e-12                          # every row's probabilities sum to one


def test_attend_mass_is_the_mean_attention_row_read_through_one_hot_values():
    # With v_j = e_j the attention output (pinned on its own above) is the probability row itself, so the mass is its
    # mean over queries and heads: a wrong head-to-group map or normaliser in either function breaks the equality.
    L = _tiny_layer(seed=5)
    n, d = 40, L.q.shape[2]
    k, p = L.hist_k[:n], L.hist_pos[:n]
    v = np.zeros((n, k.shape[1], d), np.float32)
    v[np.arange(n), :, np.arange(n)] = 1.0
    rows = oracle.attend(L.q, L.q_pos, [(k, v, p)])               # [n_q][Hq][d]: entry j = P(row, key j)
    np.testing.assert_allclose(oracle.attend_mass(L.q, L.q_pos, [(k, p)]), rows[:, :, :n].mean(axis=(0, 1)), rtol=0, atol=1e-14)


def test_attend_mass_closed_forms():
    L = _tiny_layer(seed=6)
    hkv, d = L.hist_k.shape[1], L.hist_k.shape[2]
    # identical keys at one position: every key gets 1/n
    k = np.broadcast_to(L.hist_k[:1], (25, hkv, d)).copy()
    p = np.broadcast_to(L.hist_pos[:1], (25, 4)).copy()
    np.testing.assert_allclose(oracle.attend_mass(L.q, L.q_pos, [(k, p)]), 1.0 / 25, rtol=0, atol=1e-15)
    # two keys, one query, one head, no rotation: the logistic function of the logit difference
    rng = np.random.default_rng(3)
    q1 = rng.standard_normal((1, 1, d)).astype(np.float32)
    k2 = rng.standard_normal((2, 1, d)).astype(np.float32)
    z = np.zeros((2, 4), np.int32)
    diff = float((q1[0, 0].astype(np.float64) @ (k2[0, 0].astype(np.float64) - k2[1, 0].astype(np.float64))) / np.sqrt(d))
    got = oracle.attend_mass(q1, z[:1], [(k2, z)])
    np.testing.assert_allclose(got, [1 / (1 + np.exp(-diff)), 1 / (1 + np.exp(diff))], rtol=0, atol=1e-15)
    # a key that every query matches far better than the rest takes nearly all of the mass
    kk = (0.01 * rng.standard_normal((30, hkv, d))).astype(np.float32)
    qq = np.ones_like(L.q)
    kk[7] = 4.0
    zp = np.zeros((30, 4), np.int32)
    m = oracle.attend_mass(qq, np.zeros_like(L.q_pos), [(kk, zp)])
    assert m.argmax() == 7 and m[7] > 0.999
    # the split into segments and the key order do not matter
    perm = rng.permutation(60)
    a = oracle.attend_mass(L.q, L.q_pos, [(L.hist_k[:60], L.hist_pos[:60])])
    b = oracle.attend_mass(L.q, L.q_pos, [(L.hist_k[:60][perm][:20], L.hist_pos[:60][perm][:20]),
                                          (L.hist_k[:60][perm][20:], L.hist_pos[:60][perm][20:])])
    np.testing.assert_allclose(a[perm], b, rtol=0, atol=1e-14)
