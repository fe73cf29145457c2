#!/usr/bin/env python
"""Benchmark of the PackCache hot path on B200: late-frame attention + compaction latency.

A step is one pass of the whole path for one frame of the 48-frame workload (47 history frames of 1008 tokens,
1136 anchors, 24 query / 8 KV heads of 128, bf16): plan the per-frame budgets, score the history, select per frame,
pack the retained rows, and attend the 1008 current-frame queries over anchors ++ packed history.  Steps rotate over
several layers' K/V (each layer its own seeded tensors, about 0.2 GB per layer) so that every step's inputs come
from HBM, not from L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One JSON line is printed by rank 0.  With --impl reference the CPU oracle is timed instead (bounded samples).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "late_frame_attn_plus_compaction_latency"
UNIT = "ms/frame"
WORKLOAD = "lumos47"
N_LAYERS = 4          # rotated input sets; 4 x ~0.2 GB > L2 (--layers changes it for small profiler captures)
KERNELS_PER_STEP = 6  # k_qprep, k_score, k_select, k_pack, k_attend_tc, k_combine (anchors' rotated keys are kept per layer)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------------------- ranks
def _cpu_model() -> str:
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.lower().startswith("model name"):
                return ln.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def rank_layer_ids(rank: int, n_layers: int):
    """Layers a rank draws: disjoint seeded layers per rank (weak scaling by replication, nothing exchanged on the data
    path)."""
    return [rank * n_layers + i for i in range(n_layers)]


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """The slowest rank's time: a job of N replicas takes as long as its slowest member."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_frames_per_s(ms_step_max: float, world: int) -> float:
    """Aggregate throughput of `world` independent replicas: each finishes one frame per step of the slowest rank.  The
    latency of a frame does not fall with replicas, so it is reported apart from this."""
    return world * 1e3 / ms_step_max


# --------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed regions run."""

    def __init__(self, index: int, uuid: str = ""):
        self.samples, self.reasons, self.max_mhz, self._stop = [], set(), None, threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if uuid else b"")
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "sw_power_cap": 0x4, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                util = nv.nvmlDeviceGetUtilizationRates(self.h).gpu
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((mhz, util))
                for n, bit in names.items():
                    if r & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.02)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        mhz = [m for m, _ in self.samples]
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(mhz)}


# --------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(cfg, layer, n_score: int, n_rows: int, s32=None):
    """Time the oracle on a bounded sample of one frame step and extrapolate to the whole frame.
    Returns (ms_per_frame, description)."""
    import oracle
    L = layer
    b = cfg.budget
    rng = np.random.default_rng(0)
    t0 = time.perf_counter()
    budget = oracle.plan_budget(b.kind, b.param, b.total, b.keep_full, L.frame_count)
    t_plan = time.perf_counter() - t0
    n_score, n_rows = min(n_score, cfg.n_src), min(n_rows, cfg.n_q * cfg.n_q_heads)
    idx = np.sort(rng.choice(cfg.n_src, size=n_score, replace=False))
    t0 = time.perf_counter()
    oracle.score(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base, idx=idx)
    t_score = (time.perf_counter() - t0) * (cfg.n_src / n_score)
    # the remaining stages need all scores: take them from the oracle's pooled form (not timed)
    if s32 is None:
        s32 = oracle.score_pooled(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base).astype(np.float32)
    t0 = time.perf_counter()
    sel = oracle.select(s32, L.frame_count, budget)
    t_select = time.perf_counter() - t0
    t0 = time.perf_counter()
    pk, pv, pp = oracle.pack(L.hist_k, L.hist_v, L.hist_pos, sel, 0)
    t_pack = time.perf_counter() - t0
    flat = np.sort(rng.choice(cfg.n_q * cfg.n_q_heads, size=n_rows, replace=False))     # distinct (query, head) rows
    rows = np.stack([flat // cfg.n_q_heads, flat % cfg.n_q_heads], axis=1)
    t0 = time.perf_counter()
    oracle.attend(L.q, L.q_pos, [(L.anchor_k, L.anchor_v, L.anchor_pos), (pk, pv, pp)], cfg.rope_base,
                  rows=rows.astype(np.int32))
    t_att = (time.perf_counter() - t0) * (cfg.n_q * cfg.n_q_heads / n_rows)
    total = t_plan + t_score + t_select + t_pack + t_att
    whole = n_score == cfg.n_src and n_rows == cfg.n_q * cfg.n_q_heads
    what = (f"{n_score}/{cfg.n_src} tokens scored and {n_rows}/{cfg.n_q * cfg.n_q_heads} attention rows, "
            f"select and pack in full; " + ("the whole frame, nothing scaled" if whole else "scaled to one frame"))
    return total * 1e3, what


def bench_config(cfg, n_sel: int, world: int) -> dict:
    """The `config` object of the JSON line, the same for both arms (the reference arm runs the CUDA arm's configuration)."""
    return {"workload": WORKLOAD, "n_frames": cfg.n_frames, "frame_tokens": cfg.frame_tokens,
            "n_anchor": cfg.n_anchor, "retained": int(n_sel), "keys_attended": int(cfg.n_anchor + n_sel), "n_q": cfg.n_q,
            "heads": f"{cfg.n_q_heads}q/{cfg.n_kv_heads}kv", "head_dim": cfg.head_dim,
            "budget": "2 newest frames whole + 6048 at half-life 4", "mode": "one-shot compaction every frame",
            "l2": f"inputs rotate over {N_LAYERS} layers (~{0.2 * N_LAYERS:.1f} GB; L2 is 126 MB)", "parallelism": f"replicas x{world}"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2601_04359_b200 import workload as wl
    cfg = wl.CONFIGS[WORKLOAD]
    L = wl.make_layer(cfg, 0)
    n_iter = args.steps + args.warmup
    n_score = max(8, min(2000, 12000 // n_iter))
    n_rows = max(32, min(4096, 24000 // n_iter))
    s32 = oracle.score_pooled(L.hist_k, L.hist_pos, L.q, L.q_pos, cfg.rope_base).astype(np.float32)
    vals = []
    for i in range(n_iter):
        ms, what = oracle_sample(cfg, L, n_score, n_rows, s32)
        if i >= args.warmup:
            vals.append(ms)
    v = float(np.mean(vals))
    cores = oracle.max_threads()
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": v, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": bench_config(cfg, cfg.budget.total, max(args.gpus, 1)),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------- CUDA arm
def attend_traffic(rec=None, src=None):
    """DRAM bytes of one k_attend_tc launch from the ncu capture recorded under profiles/, or None when the kernel's
    source has changed since that capture (the record carries the git blob id of the file it was taken on)."""
    import hashlib
    rec = rec or os.path.join(ROOT, "profiles", "attend_dram_traffic.json")
    src = src or os.path.join(ROOT, "paper_2601_04359_b200", "csrc", "pc_attend_tc.cu")
    try:
        r = json.load(open(rec))
        data = open(src, "rb").read()
        blob = hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()
        return r["dram_bytes_read"] + r["dram_bytes_write"] if r.get("source_blob") == blob else None
    except (OSError, ValueError, KeyError):
        return None


def run_cuda(args):
    import torch
    from paper_2601_04359_b200 import binding as pc
    from paper_2601_04359_b200 import workload as wl
    from paper_2601_04359_b200.device import DeviceLayer, make_ctx

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pc.load()

    global N_LAYERS
    N_LAYERS = args.layers
    cfg = wl.CONFIGS[WORKLOAD]
    b = cfg.budget
    # every rank draws its own layers (weak scaling: independent layers, no exchange on the data path)
    host_layers = [wl.make_layer(cfg, layer=i) for i in rank_layer_ids(rank, N_LAYERS)]
    layers = [DeviceLayer(L) for L in host_layers]
    # one context per layer, as a model would hold them: each keeps its layer's rotated anchor keys between frames
    ctxs = [make_ctx(cfg) for _ in layers]
    ctx = ctxs[0]
    n_sel = b.total
    dsts = [D.empty_packed(n_sel) for D in layers]
    scores = torch.empty(cfg.n_src, dtype=torch.float32, device="cuda")
    sel = torch.empty(n_sel, dtype=torch.int32, device="cuda")
    out = torch.empty_like(layers[0].q)
    avail = layers[0].L.frame_count
    stream = torch.cuda.current_stream()
    N = cfg.frame_tokens

    def step(i, n_frames=None):
        D, dst = layers[i % N_LAYERS], dsts[i % N_LAYERS]
        src = D.cache
        if n_frames is not None:                     # an earlier frame of the generation: the first n_frames of the history
            src = pc.Cache(D.cache.anchors, pc.Segment(D.cache.history.k, D.cache.history.v, D.cache.history.pos, n_frames * N),
                           avail[:n_frames])
        budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, src.frame_count)
        pc.pc_frame_step(ctxs[i % N_LAYERS], src, budget, 0, dst, D.q, D.q_pos, scores=scores, sel_idx=sel, out=out,
                         stream=stream)

    def step_separate(i):
        D, dst = layers[i % N_LAYERS], dsts[i % N_LAYERS]
        budget = pc.pc_plan_budget(b.kind, b.param, b.total, b.keep_full, avail)
        pc.pc_score(ctx, D.cache, D.q, D.q_pos, budget, scores=scores, sel_idx=sel, stream=stream)
        pc.pc_compact(ctx, D.cache, sel, budget, 0, dst, stream=stream)
        pc.pc_attend_frame(ctx, dst, None, D.q, D.q_pos, out=out, stream=stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, n, first=0):
        """Device time of n calls of fn(i) between two events on the launching stream, per call, max over ranks."""
        barrier()
        e0.record(stream)
        for i in range(n):
            fn(first + i)
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / n, dist, "cuda")

    sampler = ClockSampler(local, "GPU-" + str(torch.cuda.get_device_properties(local).uuid))
    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    assert all(pc.pc_poll_status(c) == pc.PC_OK for c in ctxs), "device-side error during warm-up"

    # ---- timed region: K steps between two events on the launching stream, repeated; the median region is the value.
    # The clock is sampled while these regions run, and only then.
    sampler.start()
    regions = [timed(step, args.steps) for _ in range(max(args.repeats, 1))]
    clocks = sampler.stop()
    ms_step = float(np.median(regions))
    assert all(pc.pc_poll_status(c) == pc.PC_OK for c in ctxs), "device-side error in the timed region"

    # ---- per-kernel durations (CUDA events recorded by the library at kernel boundaries, same steps again)
    for c in ctxs:
        pc.pc_set_timing(c, True)
    acc = {k: [] for k in pc.STAGES}
    for i in range(min(args.steps, 200)):
        step(i)
        for k, v in pc.pc_get_timing(ctxs[i % N_LAYERS]).items():
            if v >= 0:
                acc[k].append(v)
    kern_ms = {k: (float(np.mean(v)) if v else None) for k, v in acc.items()}
    # An event between two kernels drains the stream, so the kernel behind it starts from an idle GPU and its span
    # overstates it.  With the mark in front of a kernel left out, the span of that kernel and the one before it, minus the
    # earlier kernel's own span, is the kernel's duration as it runs in the untimed step (launch overlapped as there).
    plan = {"score": (["QPOOL"], "SCORE0", "SCORE", "qpool"), "select": (["SCORE"], "QPOOL", "SELECT", "score"),
            "pack": (["SELECT", "PACK0"], "SCORE", "PACK", "select"), "attend": (["PACK", "ATT0"], "PACK0", "ATTEND", "pack"),
            "combine": (["ATTEND"], "ATT0", "COMBINE", "attend")}
    pipelined = {}
    for name, (skip, a, b_, before) in plan.items():
        for c in ctxs:
            pc.pc_set_timing_skip(c, skip)
        spans = []
        for i in range(min(args.steps, 100)):
            step(i)
            v = pc.pc_get_span(ctxs[i % N_LAYERS], a, b_)
            if i >= 3 and v >= 0:
                spans.append(v)
        pipelined[name] = (float(np.mean(spans)) - kern_ms[before]) if spans and kern_ms[before] else None
    for c in ctxs:
        pc.pc_set_timing_skip(c, [])
        pc.pc_set_timing(c, False)

    # ---- yardstick for the HBM-bound kernels: a kernel that only streams the history keys the scoring kernel reads (same
    # access pattern, no arithmetic), by an event pair per launch and back to back, over the rotating layers
    probe_out = torch.empty(cfg.n_src, dtype=torch.int32, device="cuda")
    stream_fn = lambda i: pc.pc_probe_stream_read(layers[i % N_LAYERS].cache.history.k, probe_out, stream=stream)
    for i in range(4):
        stream_fn(i)
    singles = []
    for i in range(40):
        torch.cuda.synchronize()
        e0.record(stream); stream_fn(i); e1.record(stream)
        torch.cuda.synchronize()
        singles.append(e0.elapsed_time(e1))
    stream_single_ms = float(np.median(singles))
    stream_b2b_ms = timed(stream_fn, 100)

    # ---- yardstick for the attention kernel: its tensor-core issue stream alone (no loads, no softmax), one CTA per SM, a few
    # milliseconds per form: cycles per 128 x 128 x 16 multiply-add and the SM clock under that load
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    mma = {form: pc.pc_probe_mma_rate(ctx, form, rounds=2000) for form in ("qk", "pv", "mix")}
    assert pc.pc_poll_status(ctx) == pc.PC_OK

    # ---- the same frame through the three separate calls (pc_score, pc_compact, pc_attend_frame: eight launches)
    for i in range(3):
        step_separate(i)
    sep_ms = timed(step_separate, min(args.steps, 200))

    # ---- the last four frames of the generation (44 to 47 history frames), one-shot compaction each, and the same four
    # frames attending to the whole cache instead
    late = {}
    if not args.no_extra_pass:
        depths = [cfg.n_frames - 3 + k for k in range(4)]
        for F in depths:
            step(0, F)
        late_pack = sum(timed(lambda i, F=F: step(i, F), 50) for F in depths)

        def full(i, F):
            D = layers[i % N_LAYERS]
            src = pc.Cache(D.cache.anchors, pc.Segment(D.cache.history.k, D.cache.history.v, D.cache.history.pos, F * N), avail[:F])
            pc.pc_attend_frame(ctx, src, None, D.q, D.q_pos, out=out, stream=stream)
        for F in depths:
            full(0, F)
        late_full = sum(timed(lambda i, F=F: full(i, F), 20) for F in depths)
        late = {"history_frames": depths, "packcache_ms": late_pack, "full_cache_ms": late_full, "ratio": late_full / late_pack,
                "what": "sum over the last four frames of the 48-frame generation: plan + score + select + pack + attend on "
                        "the compacted cache against attention over the whole cache"}

    # ---- one further attention pass over an unchanged cache (a frame is generated over several diffusion steps that all
    # attend to the same keys): keys rotated once by pc_attend_prepare, each pass rotates only its queries
    pass_ms = None
    if not args.no_extra_pass:
        pc.pc_attend_prepare(ctx, dsts[0], None, stream=stream)
        prepared = lambda i: pc.pc_attend_prepared(ctx, layers[i % N_LAYERS].q, layers[i % N_LAYERS].q_pos, out=out, stream=stream)
        for i in range(5):
            prepared(i)
        pass_ms = timed(prepared, min(args.steps, 200))
        assert pc.pc_poll_status(ctx) == pc.PC_OK

    # ---- attention mass of every key of the packed cache (the score that attention-guided retention ranks by), computed
    # once per frame after the frame's last attention pass, from the rotated operands and normalisers that pass left behind
    mass_ms = None
    if not args.no_extra_pass:
        n_keys = cfg.n_anchor + n_sel
        lse = torch.empty(cfg.n_q, cfg.n_q_heads, dtype=torch.float32, device="cuda")
        mass = torch.empty(n_keys, dtype=torch.float32, device="cuda")
        n_mass = min(args.steps, 100)
        es = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_mass)]
        for i in range(-3, n_mass):
            pc.pc_attend_frame(ctx, dsts[i % N_LAYERS], None, layers[i % N_LAYERS].q, layers[i % N_LAYERS].q_pos, out=out, lse=lse,
                               stream=stream)
            if i >= 0:
                es[i][0].record(stream)
            pc.pc_attend_mass(ctx, lse, n_keys, mass=mass, stream=stream)
            if i >= 0:
                es[i][1].record(stream)
        barrier()
        mass_ms = max_over_ranks(float(np.mean([a.elapsed_time(b_) for a, b_ in es])), dist, "cuda")
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        assert abs(float(mass.sum()) - 1.0) < 1e-3

    # ---- the frame step with the cache resident in the window (Slide regime: the source of each pack is what the last
    # pack kept plus the newest frame, about 9 k tokens instead of the whole 47-frame history), first with the new
    # frame and the queries already on the device, then end to end from pinned host memory
    cap = n_sel + 2 * N
    td = torch.bfloat16
    mkbuf = lambda: pc.Segment(torch.empty((cap, cfg.n_kv_heads, cfg.head_dim), dtype=td, device="cuda"),
                               torch.empty((cap, cfg.n_kv_heads, cfg.head_dim), dtype=td, device="cuda"),
                               torch.empty((cap, 4), dtype=torch.int32, device="cuda"), 0)
    win = pc.Window(ctx, cfg.n_frames, b.kind, b.param, b.total, b.keep_full, layers[0].cache.anchors, mkbuf(), mkbuf())

    def frame_of(i):
        D = layers[i % N_LAYERS]
        f = i % cfg.n_frames
        h = D.cache.history
        return D, pc.Segment(h.k[f * N:(f + 1) * N], h.v[f * N:(f + 1) * N], h.pos[f * N:(f + 1) * N], N)

    regime_seen = []

    def inc_step(i):
        D, fr = frame_of(i)
        win.append(fr, stream=stream)
        regime_seen.append(win.step(D.q, D.q_pos, out=out, stream=stream)[0])

    inc_ms, inc_src, e2e_ms, h2d, d2h, n_e2e = None, None, None, 0, 0, 0
    if not args.no_incremental:
        for i in range(cfg.n_frames + 3):                       # fill the window, then a few sliding steps
            inc_step(i)
        barrier()
        assert regime_seen[-1] == pc.PC_WINDOW_SLIDE and pc.pc_poll_status(ctx) == pc.PC_OK
        inc_src = int(win.state()[0].sum()) + N
        inc_ms = timed(inc_step, min(args.steps, 200), cfg.n_frames + 3)
        assert pc.pc_poll_status(ctx) == pc.PC_OK

    # ---- end to end through the host-buffer entry point of the window: every step uploads the finished frame's K, V and
    # positions and the new frame's queries and positions from pinned memory, and downloads the attention output
    if not args.no_incremental and not args.no_e2e:
        pin = lambda x: x.cpu().pin_memory()
        hosts = []
        for i in range(8):
            D, fr = frame_of(i)
            hosts.append(({"k": pin(fr.k), "v": pin(fr.v), "pos": pin(fr.pos)}, pin(D.q), pin(D.q_pos)))
        out_host = torch.empty(out.shape, dtype=td).pin_memory()
        ws = {"q": torch.empty_like(layers[0].q), "q_pos": torch.empty_like(layers[0].q_pos), "out": out}
        fr0, q0, qp0 = hosts[0]
        h2d = sum(x.numel() * x.element_size() for x in (fr0["k"], fr0["v"], fr0["pos"], q0, qp0))
        d2h = out_host.numel() * out_host.element_size()

        def e2e_step(i):
            fr, q, qp = hosts[i % len(hosts)]
            assert win.step_host(fr, q, qp, out_host, ws, stream=stream) == pc.PC_WINDOW_SLIDE
        for i in range(3):
            e2e_step(i)
        n_e2e = max(3, min(args.steps, 100))
        barrier()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)
        barrier()
        e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3 / n_e2e, dist, "cuda")      # each step ends with a stream wait
        assert pc.pc_poll_status(ctx) == pc.PC_OK
    win.close()

    # ---- the one-shot step end to end (the whole history uploaded every frame: a copy benchmark, kept for reference)
    full_ms, full_h2d = None, 0
    if not args.no_e2e and args.full_upload:
        L0 = host_layers[0]
        pinn = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(dt) if dt else
                                   torch.from_numpy(np.ascontiguousarray(a))).pin_memory()
        hostbuf = {"q": pinn(L0.q, td), "q_pos": pinn(L0.q_pos), "anchor_k": pinn(L0.anchor_k, td),
                   "anchor_v": pinn(L0.anchor_v, td), "anchor_pos": pinn(L0.anchor_pos), "hist_k": pinn(L0.hist_k, td),
                   "hist_v": pinn(L0.hist_v, td), "hist_pos": pinn(L0.hist_pos), "frame_count": L0.frame_count,
                   "out": torch.empty(L0.q.shape, dtype=td).pin_memory()}
        ws1 = {"q": torch.empty_like(layers[0].q), "q_pos": torch.empty_like(layers[0].q_pos), "scores": scores,
               "sel_idx": sel, "out": out}
        ws_src = pc.Cache(pc.Segment(torch.empty_like(layers[0].cache.anchors.k), torch.empty_like(layers[0].cache.anchors.v),
                                     torch.empty_like(layers[0].cache.anchors.pos), 0),
                          pc.Segment(torch.empty_like(layers[0].cache.history.k), torch.empty_like(layers[0].cache.history.v),
                                     torch.empty_like(layers[0].cache.history.pos), 0), L0.frame_count)
        full_h2d = sum(hostbuf[k].numel() * hostbuf[k].element_size() for k in
                       ("q", "q_pos", "anchor_k", "anchor_v", "anchor_pos", "hist_k", "hist_v", "hist_pos"))
        one = lambda i: pc.pc_frame_step_host(ctx, hostbuf, ws_src, dsts[0], ws1, b.kind, b.param, b.total, b.keep_full, 0, stream)
        one(0)
        barrier()
        t0 = time.perf_counter()
        for i in range(5):
            one(i)
        barrier()
        full_ms = max_over_ranks((time.perf_counter() - t0) * 1e3 / 5, dist, "cuda")
    status = pc.pc_poll_status(ctx)
    assert status == pc.PC_OK, f"device-side status {status}"

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (attention: a dense contraction on the tensor cores)
    peaks = _peaks()
    n_keys = cfg.n_anchor + n_sel
    flops = 4.0 * cfg.n_q * n_keys * cfg.head_dim * cfg.n_q_heads
    # the attention kernel's duration as it runs in the untimed step (the mark in front of it left out); its span between
    # two marks of its own, which also holds a launch from an idle GPU, rides along
    att_span_ms = kern_ms["attend"]
    att_ms = pipelined.get("attend") or att_span_ms
    achieved = flops / (att_ms * 1e-3) / 1e12
    row = cfg.n_kv_heads * cfg.head_dim * 2
    score_bytes = cfg.n_src * (row + 16 + 4)
    pack_bytes = n_sel * (5 * row + 32 + 4)          # K and V rows read, K, V and rotated K written, positions, index
    hbm = lambda nbytes, ms: (nbytes / (ms * 1e-3) / 1e9) if ms else None

    def hbm_entry(nbytes, ms, ms_pipe):
        return {"GBps": hbm(nbytes, ms), "bytes": nbytes, "frac": (hbm(nbytes, ms) or 0) / peaks["hbm_gbs"], "ms": ms,
                "GBps_pipelined": hbm(nbytes, ms_pipe), "frac_pipelined": (hbm(nbytes, ms_pipe) or 0) / peaks["hbm_gbs"],
                "ms_pipelined": ms_pipe}
    both_ms = (kern_ms["score"] + kern_ms["pack"]) if kern_ms["score"] and kern_ms["pack"] else None
    both_pipe = (pipelined["score"] + pipelined["pack"]) if pipelined.get("score") and pipelined.get("pack") else None
    stages = {k: (round(v, 5) if v is not None else None) for k, v in kern_ms.items()}
    line = {
        "metric": METRIC, "value": ms_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": bench_config(cfg, n_sel, world),
        "timed_regions": {"count": len(regions), "steps_each": args.steps, "median_ms_per_step": ms_step,
                          "min_ms_per_step": float(min(regions)), "max_ms_per_step": float(max(regions))},
        "replicas": {"frames_per_s": replica_frames_per_s(ms_step, world), "what": "every rank steps its own layers; per-frame latency is "
                     "the slowest rank's, the job's aggregate is this throughput"},
        "clocks": clocks,
        "e2e": {"value": e2e_ms, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
                "copies_declared": True,
                "mode": "Slide regime, cache resident on the device: pc_window_step_host uploads the finished frame's K, V, "
                        "positions and the new frame's queries from pinned memory, updates the window, attends, downloads O",
                "full_upload": {"value": full_ms, "h2d_bytes_per_step": full_h2d,
                                "what": "pc_frame_step_host: the whole 47-frame history re-uploaded every frame (copy-bound)"}},
        "gpu_launches": KERNELS_PER_STEP * args.steps * len(regions),
        "roofline": {"kernel": "k_attend_tc", "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"], "traffic": attend_traffic(),
                     "peak_source": f"{peaks['source']} (burst; sustained {peaks['bf16_tflops_sustained']})",
                     "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                     "flops_per_launch": flops, "ms_per_launch": att_ms, "ms_per_launch_single_kernel_span": att_span_ms,
                     "frac_by_single_kernel_span": flops / (att_span_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                     "mma_yardstick": {
                         "cycles_per_mma": {k: round(v[0], 2) for k, v in mma.items()}, "sm_ghz_under_load": {k: round(v[1], 3) for k, v in mma.items()},
                         "tflops_mix_never_waiting": 524288.0 * sm_count * mma["mix"][1] * 1e9 / mma["mix"][0] / 1e12,
                         "frac_of_yardstick": achieved / (524288.0 * sm_count * mma["mix"][1] * 1e9 / mma["mix"][0] / 1e12),
                         "what": "pc_probe_mma_rate: the kernel's own tcgen05.mma stream (Q K^T from shared memory, P V with P in "
                                 "tensor memory, and both in the kernel's order) issued back to back on every SM with nothing else "
                                 "running; 524,288 flop per multiply-add x SMs x clock / cycles is what the tensor cores deliver "
                                 "to this instruction mix when they never wait"},
                     "how": "flops / the kernel's mean duration by CUDA events on the launching stream: the event mark in front "
                            "of the kernel left out, span of the pack kernel and this one minus the pack kernel's own span (the "
                            "duration as in the untimed step); the kernel runs inside a long power-capped step, for which the "
                            "sustained peak is the like-for-like denominator, the burst peak the conservative one used for frac"},
        "kernels_ms": stages,
        "kernels_ms_pipelined": {k: (round(v, 5) if v is not None else None) for k, v in pipelined.items()},
        "separate_calls": {"ms_per_frame": sep_ms, "what": "the same frame through pc_score, pc_compact and pc_attend_frame "
                           "(eight launches: Q read twice, rotary pre-pass over anchors and packed history)"},
        "late4": late,
        "extra_pass": {"ms_per_pass": pass_ms, "what": "one more attention pass of the frame over the unchanged packed cache "
                       "(pc_attend_prepared: query rotation, attention, merge; keys were rotated once per frame)"},
        "attention_mass": {"ms": mass_ms, "keys": cfg.n_anchor + n_sel,
                           "what": "pc_attend_mass after an attention pass over the packed cache: K Q^T on tensor cores, "
                                   "column sums of the normalised probabilities (three launches)"},
        "incremental": {"ms_per_frame": inc_ms, "source_tokens": inc_src,
                        "mode": "cache window in the Slide regime (pc_window_append + pc_window_step): append the newest frame, "
                                "drop the oldest, re-plan, score and re-select from packed + new, pack, attend (same keys attended)"},
        "hbm_kernels": {
            "score": hbm_entry(score_bytes, kern_ms["score"], pipelined.get("score")),
            "pack": hbm_entry(pack_bytes, kern_ms["pack"], pipelined.get("pack")),
            "score_plus_pack": hbm_entry(score_bytes + pack_bytes, both_ms, both_pipe) if both_ms else None,
            "how": "bytes / kernel duration.  `frac`: between the library's CUDA event marks around the kernel alone; an event "
                   "between two kernels drains the stream, so this span also holds a launch from an idle GPU (see "
                   "stream_read_yardstick for what a plain streaming read of the score kernel's bytes reaches that way).  `frac_pipelined`: the mark in front of the kernel left out, the common span of the "
                   "kernel and the one before it minus that kernel's own span: the duration as in the untimed step",
            "stream_read_yardstick": {
                "bytes": cfg.n_src * row,
                "single_launch": {"ms": stream_single_ms, "frac": hbm(cfg.n_src * row, stream_single_ms) / peaks["hbm_gbs"]},
                "back_to_back": {"ms": stream_b2b_ms, "frac": hbm(cfg.n_src * row, stream_b2b_ms) / peaks["hbm_gbs"]},
                "what": "pc_probe_stream_read over the same history keys: what a kernel that only streams the scoring kernel's "
                        "bytes reaches here, timed by an event pair around one launch from an idle GPU and back to back"},
            "peak": peaks["hbm_gbs"], "peak_source": peaks["source"]},
    }
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        t0 = time.perf_counter()
        # size the sample with a short probe so that the timed part is about 15 s of oracle work on this host's cores
        # (on 16 cores that is the whole frame: every token scored, every attention row)
        probe_ms, _ = oracle_sample(cfg, host_layers[0], n_score=400, n_rows=800)
        frac = min(1.0, 15e3 / max(probe_ms, 1.0))
        v, what = oracle_sample(cfg, host_layers[0], n_score=max(400, int(frac * cfg.n_src)),
                                n_rows=max(800, int(frac * cfg.n_q * cfg.n_q_heads)))
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                                "sample": what, "sample_seconds": round(time.perf_counter() - t0, 1)}
        # the same oracle on one thread, from a small sample (a few seconds), and the host's CPU model
        n_threads = oracle.max_threads()
        oracle.set_threads(1)
        v1, what1 = oracle_sample(cfg, host_layers[0], n_score=60, n_rows=120)
        oracle.set_threads(n_threads)
        line["cpu_baseline"]["single_thread"] = {"value": v1, "unit": UNIT, "sample": what1}
        line["cpu_baseline"]["cpu_model"] = _cpu_model()
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--repeats", type=int, default=25, help="timed regions of --steps steps each; the median is reported")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer legs (profiler captures)")
    ap.add_argument("--full-upload", action="store_true", help="also time the one-shot host step that re-uploads the whole history")
    ap.add_argument("--no-incremental", action="store_true", help="skip the cache-window leg (profiler captures)")
    ap.add_argument("--no-extra-pass", action="store_true", help="skip the prepared-attention leg (profiler captures)")
    ap.add_argument("--layers", type=int, default=N_LAYERS, help="rotated input sets (default 4, > L2)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand with --gpus N: relaunch as one rank per GPU
        os.execvp(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node",
                                   str(args.gpus), "--master-addr", "127.0.0.1", "--master-port", "29511"] + sys.argv)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
