"""A bounded device-side wait that runs out, on purpose and in the permitted form.

Every wait of the library's kernels has a limit; when it runs out the kernel records PC_ERR_TIMEOUT, gives up the work
that depended on the wait, lets its copies land, frees what it holds and returns, and the context stays usable.  Here
the limit is set to two milliseconds and the attention kernel's first barrier is told by the host to expect sixteen
bytes more than its copies will ever deliver, so the wait on it cannot be satisfied: nothing traps, nothing spins
without a limit, no address is bad.  The next ordinary call on the same context must work and match the oracle."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
from paper_2601_04359_b200 import binding as pc
from paper_2601_04359_b200 import workload as wl
from paper_2601_04359_b200.device import DeviceLayer, host, make_ctx

from .test_gpu_parity import check_bf16_attention

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_survives():
    cfg = wl.small_bf16(n_frames=2, grid=(8, 9), seed=60)
    L = wl.make_layer(cfg)
    D = DeviceLayer(L)
    ctx = make_ctx(cfg)
    good = pc.pc_attend_frame(ctx, D.cache, None, D.q, D.q_pos).clone()
    assert pc.pc_poll_status(ctx) == pc.PC_OK

    pc.pc_set_wait_limit_us(ctx, 2000)
    pc.pc_test_expect_extra_bytes(ctx, 16)
    pc.pc_attend_frame(ctx, D.cache, None, D.q, D.q_pos)          # every CTA's first wait runs out after 2 ms
    assert pc.pc_poll_status(ctx) == pc.PC_ERR_TIMEOUT
    assert pc.pc_poll_status(ctx) == pc.PC_OK                      # polling cleared the word

    pc.pc_test_expect_extra_bytes(ctx, 0)
    pc.pc_set_wait_limit_us(ctx, 0)
    again = pc.pc_attend_frame(ctx, D.cache, None, D.q, D.q_pos)
    assert pc.pc_poll_status(ctx) == pc.PC_OK
    assert (again.view(dtype=good.dtype) == good).all()
    want = oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (L.hist_k, L.hist_v, L.hist_pos)], cfg.rope_base)
    check_bf16_attention(host(again).astype(np.float64), want)
    ctx.close()
