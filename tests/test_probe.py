"""The streaming-read yardstick: it must really read every byte it is timed on, so its output is checked — one word per
row, the xor of the row's 32-bit words — for row widths that take the unrolled and the looped path and an odd row count.
The multiply-add yardstick: a 128 x 128 x 16 bf16 multiply-add is 524,288 flop, and an SM's tensor core does 8,192 per
clock, so a multiply-add that was really executed cannot take fewer than 64 cycles; one that was only issued takes about 12."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from paper_2601_04359_b200 import binding as pc

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_rows,row_bytes", [(1, 512), (37, 2048), (1000, 2048), (65, 1024), (9, 4096)])
def test_stream_read_returns_the_xor_of_every_row(n_rows, row_bytes):
    rng = np.random.default_rng(n_rows)
    data = rng.integers(0, 2 ** 32, size=(n_rows, row_bytes // 4), dtype=np.uint64).astype(np.uint32)
    rows = torch.from_numpy(data.view(np.int32)).cuda()
    out = torch.zeros(n_rows, dtype=torch.int32, device="cuda")
    pc.pc_probe_stream_read(rows, out)
    torch.cuda.synchronize()
    want = np.bitwise_xor.reduce(data, axis=1)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want)


def test_stream_read_rejects_rows_that_are_not_whole_512_byte_runs():
    rows = torch.zeros((4, 100), dtype=torch.int32, device="cuda")          # 400 bytes per row
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_probe_stream_read(rows, torch.zeros(4, dtype=torch.int32, device="cuda"))
    assert e.value.status == pc.PC_ERR_INVALID_ARG


def test_mma_rate_probe_cannot_beat_the_tensor_core():
    from paper_2601_04359_b200 import workload as wl
    from paper_2601_04359_b200.device import make_ctx
    ctx = make_ctx(wl.small_bf16())
    rates = {form: pc.pc_probe_mma_rate(ctx, form, rounds=500) for form in ("qk", "pv", "mix")}
    assert pc.pc_poll_status(ctx) == pc.PC_OK
    for form, (cycles, ghz) in rates.items():
        assert 63.5 <= cycles <= 100.0, (form, cycles)          # executed, and at a rate a tensor core can have
        assert 0.8 <= ghz <= 2.3, (form, ghz)
    assert rates["qk"][0] >= rates["pv"][0] - 0.5                 # two operands from shared memory cannot be cheaper than one
    one_cta = pc.pc_probe_mma_rate(ctx, "mix", rounds=200, n_cta=1)
    assert 63.5 <= one_cta[0] <= 100.0
    with pytest.raises(pc.PackCacheError) as e:
        pc.pc_probe_mma_rate(ctx, "mix", rounds=0)
    assert e.value.status == pc.PC_ERR_INVALID_ARG
    ctx.close()
