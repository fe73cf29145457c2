"""The multi-rank path of the benchmark on CPU: two `gloo` ranks.  The path shards by replication (each rank its own
seeded layers, no collective on the data path), so what has to hold is: ranks draw disjoint layers, the job time is the
maximum over ranks, replicas add throughput and not latency, and under a two-rank launch of the reference arm only rank 0
works and prints.  The KV-head split of one layer (the one multi-GPU form in which ranks have to agree on something) is
covered by two ranks that score their head slices with the oracle and reduce the scores."""
from __future__ import annotations

import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = bench.rank_layer_ids(rank, 4)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, dist)          # rank 1 is the slow one
    dist.barrier()
    out.put((rank, gathered, slowest))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_layers_and_take_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, gathered, slowest in got:
        assert gathered == [[0, 1, 2, 3], [4, 5, 6, 7]]                # disjoint, seeded per rank
        assert slowest == 15.0                                         # every rank reports the maximum
    # a frame's latency is the slowest rank's step; what two replicas add is throughput, reported apart from it
    assert abs(bench.replica_frames_per_s(15.0, world) - 2000.0 / 15.0) < 1e-9
    assert bench.max_over_ranks(3.0, None) == 3.0


def test_reference_arm_under_two_ranks_prints_once():
    env = dict(os.environ, WORLD_SIZE="2", OMP_NUM_THREADS="2")
    outs = []
    for rank in (0, 1):
        env["RANK"] = env["LOCAL_RANK"] = str(rank)
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                            "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-500:]
        outs.append(r.stdout.strip())
    assert outs[1] == ""                                               # rank 1 exits without work
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def _kv_worker(rank, world, port, out):
    """A rank of the KV-head split on CPU: the oracle scores its head slice, the ranks' scores are reduced, and every
    rank selects on the reduced vector."""
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2601_04359_b200 import kv_split
    from paper_2601_04359_b200 import workload as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.small_bf16(n_frames=3, grid=(6, 7), n_text=20, total=60, keep_full=0, seed=70)
    L = wl.make_layer(cfg)
    kv0, kv1, q0, q1 = kv_split.head_slice(rank, world, cfg.n_q_heads, cfg.n_kv_heads)
    local = oracle.score(L.hist_k[:, kv0:kv1], L.hist_pos, L.q[:, q0:q1], L.q_pos, cfg.rope_base)
    s = torch.from_numpy(local.astype(np.float32))
    kv_split.reduce_scores(s, q1 - q0, cfg.n_q_heads, dist)
    b = cfg.budget
    budget = oracle.plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    sel = oracle.select(s.numpy(), L.frame_count, budget)
    dist.barrier()
    out.put((rank, s.numpy().tobytes(), sel.tolist()))
    dist.destroy_process_group()


def test_kv_head_split_ranks_agree_on_the_selection():
    """Two gloo ranks, each with half of the KV heads: the reduced score vectors are bit-identical on both ranks, equal
    the scores over all heads (to fp32 rounding), and give the same kept tokens as the unsplit selection."""
    import oracle
    from paper_2601_04359_b200 import kv_split
    from paper_2601_04359_b200 import workload as wl
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_kv_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, s0, sel0), (_, s1, sel1) = got
    assert s0 == s1 and sel0 == sel1                                   # same bits, same kept tokens on every rank
    cfg = wl.small_bf16(n_frames=3, grid=(6, 7), n_text=20, total=60, keep_full=0, seed=70)
    L = wl.make_layer(cfg)
    full = oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base)
    reduced = np.frombuffer(s0, dtype=np.float32)
    assert np.abs(reduced - full).max() <= 1e-5 * np.abs(full).max()
    b = cfg.budget
    budget = oracle.plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    assert sel0 == oracle.select(reduced, L.frame_count, budget).tolist()
    assert kv_split.head_slice(1, 2, 24, 8) == (4, 8, 12, 24)
    with pytest.raises(ValueError):
        kv_split.head_slice(0, 3, 24, 8)


def test_recorded_dram_traffic_is_dropped_when_the_kernel_source_changes(tmp_path):
    """The bench line's roofline.traffic comes from a record that names the git blob of the attention kernel's source:
    it is reported while that file is unchanged and becomes null as soon as the file differs."""
    src = os.path.join(ROOT, "paper_2601_04359_b200", "csrc", "pc_attend_tc.cu")
    rec = json.load(open(os.path.join(ROOT, "profiles", "attend_dram_traffic.json")))
    assert bench.attend_traffic() in (None, rec["dram_bytes_read"] + rec["dram_bytes_write"])
    changed = tmp_path / "pc_attend_tc.cu"
    changed.write_bytes(open(src, "rb").read() + b"\n// touched\n")
    assert bench.attend_traffic(src=str(changed)) is None
    same = tmp_path / "same.cu"
    same.write_bytes(b"x")
    import hashlib
    fake = tmp_path / "rec.json"
    fake.write_text(json.dumps({"dram_bytes_read": 5, "dram_bytes_write": 7,
                                "source_blob": hashlib.sha1(b"blob 1\0x").hexdigest()}))
    assert bench.attend_traffic(rec=str(fake), src=str(same)) == 12
    assert bench.attend_traffic(rec=str(tmp_path / "missing.json"), src=str(same)) is None
