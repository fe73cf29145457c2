"""The allocation-free scoring entry point against the ordinary one.

Some hosts cannot call cudaMalloc when they need scores (all device memory already belongs to their own arena, or
they cannot afford the device-wide synchronisation an allocation implies) and therefore cannot create a context.
``pc_score_tokens_static`` serves them from a fixed device array inside the library.  Here it is called through the
C ABI twice in a row — a bf16 case, then an fp32 case of another shape, so the second call finds the array full of
the first call's rotary table and pooled-query accumulator — and each result must agree with ``pc_score`` and with the
CPU oracle on the same inputs within the score tolerance used everywhere else (1e-4 relative, floored by the frame's
rms).  That the call allocates nothing is checked at driver level: free device memory (``cudaMemGetInfo``) must not
drop across a call, which a ``cudaMalloc`` inside the library would cause and PyTorch's own counters would not see.

This file sorts last on purpose: a run that stops at the first failure has already run every other test.
"""
from __future__ import annotations

import ctypes as C
import gc

import numpy as np
import pytest
import torch

import oracle

from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import workload as wl
from paper_2601_04359_b200.device import DeviceLayer, host, make_ctx, score_tolerance

pytestmark = pytest.mark.gpu


def _desc(cfg) -> pc.pc_layer_desc:
    return pc.pc_layer_desc(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                            pc.PC_BF16 if cfg.dtype == wl.BF16 else pc.PC_F32, cfg.rope_base,
                            (C.c_int32 * 3)(*cfg.max_pos), 0, 0)


def _free_bytes() -> int:
    """Free device memory as the driver counts it: unlike torch's own counters it sees a cudaMalloc / cudaFree made by the
    library itself."""
    return torch.cuda.mem_get_info()[0]


def _both(cfg, layer, warm: bool):
    """(scores from pc_score, scores from the allocation-free call, the oracle's scores, frame table) for one seeded layer."""
    L = wl.make_layer(cfg, layer=layer)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    want, _ = pc.pc_score(ctx, D.cache, D.q, D.q_pos, np.zeros(cfg.n_frames, np.int32))
    assert pc.pc_poll_status(ctx) == pc.PC_OK
    # buffers exist before the call; the call itself must not need any more memory
    scores = torch.full((cfg.n_src,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    args = (_desc(cfg), D.cache.history.k, D.cache.history.pos, cfg.n_src, D.q, D.q_pos, scores, status)
    if warm:
        # the first call of a kernel instance on a device may load its code and look up the array's address: one call
        # of this very shape first, so that the measured call is an ordinary one
        pc.pc_score_tokens_static(*args)
        scores.fill_(float("nan"))
    gc.collect()                       # tensors of earlier tests must not be freed in the middle of the measurement
    torch.cuda.synchronize()
    before, before_torch = _free_bytes(), torch.cuda.memory_allocated()
    pc.pc_score_tokens_static(*args)
    torch.cuda.synchronize()
    after = _free_bytes()
    assert after >= before, f"the call took {before - after} bytes of device memory"      # nothing allocated at driver level
    assert torch.cuda.memory_allocated() <= before_torch                                   # nor from torch's allocator
    assert status.cpu().tolist() == [0, 0]
    ctx.close()
    ref = oracle.score_pooled(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)
    return host(want)[:cfg.n_src].astype(np.float64), host(scores).astype(np.float64), ref, L.frame_count


def test_static_scratch_scoring_matches_pc_score_on_two_calls_in_a_row():
    first = wl.small_bf16(n_frames=4, grid=(12, 21), total=300, keep_full=0)    # 1008 source tokens, bf16, d = 128
    second = wl.CONFIGS["tiny"]                                                 # fp32, d = 64, other table extents
    for cfg, layer in ((first, 0), (second, 1), (first, 2)):
        want, got, ref, frame_count = _both(cfg, layer, warm=True)
        assert np.isfinite(got).all()
        tol = score_tolerance(ref, frame_count)
        assert (np.abs(got - want) <= tol).all()          # the existing entry point
        assert (np.abs(got - ref) <= tol).all()           # the oracle (fp64, pooled form)


def test_static_scratch_scoring_rejects_shapes_beyond_its_fixed_array():
    cfg = wl.small_bf16()
    z = torch.zeros(16, dtype=torch.float32, device="cuda")
    st = torch.zeros(2, dtype=torch.int32, device="cuda")
    big = pc.pc_layer_desc(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, pc.PC_BF16, cfg.rope_base,
                           (C.c_int32 * 3)(4096, 4096, 4096), 0, 0)                 # rotary table too large
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_score_tokens_static(big, z, z, 1, z, z, z, st)
    assert e.value.status == pc.PC_ERR_CAPACITY
    wide = pc.pc_layer_desc(32, 16, 128, pc.PC_BF16, cfg.rope_base, (C.c_int32 * 3)(64, 64, 64), 0, 0)   # row > 1024
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_score_tokens_static(wide, z, z, 1, z, z, z, st)
    assert e.value.status == pc.PC_ERR_CAPACITY
