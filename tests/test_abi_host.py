"""CPU-side checks of the CUDA library: it loads, exports every symbol the header declares, and its host-only
budget planner agrees bit for bit with the oracle.  No GPU work is issued here."""
from __future__ import annotations

import os
import re

import numpy as np
import pytest

import oracle
from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import workload as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "packcache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pc_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = pc.load()
    names = _declared()
    assert {"pc_create", "pc_destroy", "pc_plan_budget", "pc_score", "pc_compact", "pc_attend_frame",
            "pc_poll_status", "pc_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in packcache.h but not exported"
    assert sorted(pc.EXPORTS) == names


def test_status_strings():
    lib = pc.load()
    seen = {lib.pc_status_string(i).decode() for i in range(7)}
    assert len(seen) == 7 and "ok" in seen


KINDS = [(pc.PC_GEOMETRIC, 0.5), (pc.PC_GEOMETRIC, 0.83), (pc.PC_CLOSED_HALF, 0.5), (pc.PC_LINEAR, 0.0),
         (pc.PC_HALFLIFE, 2.0), (pc.PC_HALFLIFE, 4.0), (pc.PC_HALFLIFE, 8.0)]


@pytest.mark.parametrize("kind,param", KINDS)
def test_plan_budget_bit_exact_with_oracle(kind, param):
    rng = np.random.default_rng(kind * 10 + int(param * 7))
    for W in (1, 2, 6, 12, 24, 47):
        for total in (0, 1, 128, 3024, 6048, 8064, 47 * 1008, 10 ** 7):
            for keep in (0, 2):
                if keep > W or keep * 1008 > total:
                    continue
                avail = [1008] * W
                assert pc.pc_plan_budget(kind, param, total, keep, avail).tolist() == \
                    oracle.plan_budget(kind, param, total, keep, avail).tolist()
    for _ in range(50):
        W = int(rng.integers(1, 20))
        avail = rng.integers(0, 200, size=W)
        total = int(rng.integers(0, 3000))
        assert pc.pc_plan_budget(kind, param, total, 0, avail).tolist() == \
            oracle.plan_budget(kind, param, total, 0, avail).tolist()


def test_plan_budget_for_the_five_configs():
    for name in ("tiny", "lumos12", "lumos24", "lumos47"):
        cfg = wl.CONFIGS[name]
        b = cfg.budget
        avail = [cfg.frame_tokens] * cfg.n_frames
        got = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, avail)
        assert got.tolist() == oracle.plan_budget(b.kind, b.param, b.total, b.keep_full, avail).tolist()
        assert got.sum() == b.total
    # the full-stack sweep: every budget fraction and decay of the 28-layer configuration
    cfg = wl.CONFIGS["stack28"]
    for frac in (0.10, 0.25, 0.50, 1.00):
        for kind, param in [(pc.PC_LINEAR, 0.0), (pc.PC_HALFLIFE, 2.0), (pc.PC_HALFLIFE, 4.0), (pc.PC_HALFLIFE, 8.0)]:
            for F in (1, 5, 24, 47):
                total = int(frac * F * cfg.frame_tokens)
                avail = [cfg.frame_tokens] * F
                assert pc.pc_plan_budget(kind, param, total, 0, avail).tolist() == \
                    oracle.plan_budget(kind, param, total, 0, avail).tolist()


def test_plan_budget_errors():
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_plan_budget(pc.PC_HALFLIFE, 4.0, 1000, 2, [1008] * 5)
    assert e.value.status == pc.PC_ERR_BUDGET
    for bad in [dict(kind=9, param=0.5), dict(kind=pc.PC_GEOMETRIC, param=1.0), dict(kind=pc.PC_HALFLIFE, param=0.0)]:
        with pytest.raises(pc.PackCacheError) as e:
            pc.pc_plan_budget(bad["kind"], bad["param"], 10, 0, [5, 5])
        assert e.value.status == pc.PC_ERR_INVALID_ARG
    with pytest.raises(pc.PackCacheError):
        pc.pc_plan_budget(pc.PC_LINEAR, 0.0, -1, 0, [5])
    with pytest.raises(pc.PackCacheError):
        pc.pc_plan_budget(pc.PC_LINEAR, 0.0, 5, 0, [5], min_quota=-1)
    assert pc.pc_plan_budget(pc.PC_LINEAR, 0.0, 5, 0, []).tolist() == []


@pytest.mark.parametrize("kind,param", KINDS)
def test_plan_budget_with_minimum_quota_bit_exact_with_oracle(kind, param):
    rng = np.random.default_rng(7)
    for _ in range(60):
        W = int(rng.integers(1, 20))
        avail = rng.integers(0, 1200, size=W)
        keep = int(rng.integers(0, 3))
        m = int(rng.integers(0, 200))
        total = int(rng.integers(0, int(avail.sum()) + 300))
        try:
            want = oracle.plan_budget(kind, param, total, keep, avail, min_quota=m).tolist()
        except oracle.OracleError as e:
            assert e.code == oracle.ERR_BUDGET
            with pytest.raises(pc.PackCacheError) as g:
                pc.pc_plan_budget(kind, param, total, keep, avail, min_quota=m)
            assert g.value.status == pc.PC_ERR_BUDGET
            continue
        assert pc.pc_plan_budget(kind, param, total, keep, avail, min_quota=m).tolist() == want
