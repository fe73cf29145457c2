"""The streaming-read yardstick: it must really read every byte it is timed on, so its output is checked — one word per
row, the xor of the row's 32-bit words — for row widths that take the unrolled and the looped path and an odd row count."""
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
