"""Per-frame latency curves of the cache strategies on one GPU (synthetic lumos-shaped layer).

    python -m paper_2601_04359_b200.sweep [--reps 20] [--layers 28]

Three strategies, as in the paper's comparison (Sec. 3.3 / Sec. 4): the full KV cache (every history frame attended), a
sliding window (anchors plus the most recent frame), and PackCache (anchors plus the compacted history: the two newest
frames whole and 6048 tokens over the rest at half-life 4, one-shot compaction every frame).  For each history depth the
script times one layer's frame step (compaction, where there is one, plus attention of the 1008 current-frame queries)
with CUDA events and prints one JSON line per depth, then the budget x decay grid of the 28-layer configuration at 47
history frames, then a summary.  `--layers` only scales the per-layer time to a stack of identical layers.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as pc
from . import workload as wl
from .device import DeviceLayer, make_ctx


def _time(fn, reps, stream):
    for _ in range(3):
        fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--layers", type=int, default=28)
    ap.add_argument("--depths", type=str, default="1,2,3,4,6,8,12,16,24,32,40,44,45,46,47")
    ap.add_argument("--stack", type=int, default=0, help="also time one frame through this many distinct layers (5.6 GB at 28)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("the sweep needs a CUDA device; there is no CPU fallback")
    cfg = wl.CONFIGS["lumos47"]
    N = cfg.frame_tokens
    D = DeviceLayer(wl.make_layer(cfg))
    ctx = make_ctx(cfg)
    stream = torch.cuda.current_stream()
    scores = torch.empty(cfg.n_src, dtype=torch.float32, device="cuda")
    sel = torch.empty(cfg.n_src, dtype=torch.int32, device="cuda")
    out = torch.empty_like(D.q)
    dst = D.empty_packed(cfg.n_src)
    h = D.cache.history

    def history(first_frame, n_frames):
        a, b = first_frame * N, (first_frame + n_frames) * N
        return pc.Cache(D.cache.anchors, pc.Segment(h.k[a:b], h.v[a:b], h.pos[a:b], n_frames * N), np.full(n_frames, N, np.int32))

    def pack_step(cache, kind, param, total, keep_full):
        avail = cache.frame_count
        budget = pc.pc_plan_budget(kind, param, min(total, int(avail.sum())), min(keep_full, len(avail)), avail)
        if budget.sum() == avail.sum():                       # nothing to drop: attend the cache as it is
            pc.pc_attend_frame(ctx, cache, None, D.q, D.q_pos, out=out, stream=stream)
            return
        pc.pc_score(ctx, cache, D.q, D.q_pos, budget, scores=scores, sel_idx=sel, stream=stream)
        pc.pc_compact(ctx, cache, sel, budget, 0, dst, stream=stream)
        pc.pc_attend_frame(ctx, dst, None, D.q, D.q_pos, out=out, stream=stream)

    rows = []
    for F in [int(x) for x in args.depths.split(",")]:
        full = history(cfg.n_frames - F, F)                   # the F most recent frames
        last = history(cfg.n_frames - 1, 1)
        t_full = _time(lambda: pc.pc_attend_frame(ctx, full, None, D.q, D.q_pos, out=out, stream=stream), args.reps, stream)
        t_slide = _time(lambda: pc.pc_attend_frame(ctx, last, None, D.q, D.q_pos, out=out, stream=stream), args.reps, stream)
        t_pack = _time(lambda: pack_step(full, pc.PC_HALFLIFE, 4.0, 2 * N + 6048, 2), args.reps, stream)
        row = {"history_frames": F, "keys_full": cfg.n_anchor + F * N, "ms_full": round(t_full, 4), "ms_packcache": round(t_pack, 4),
               "ms_sliding": round(t_slide, 4), "speedup_vs_full": round(t_full / t_pack, 2)}
        rows.append(row)
        print(json.dumps(row), flush=True)
    assert pc.pc_poll_status(ctx) == pc.PC_OK

    grid = []
    full47 = history(0, cfg.n_frames)
    for frac in (0.10, 0.25, 0.50, 1.00):
        for name, kind, param in (("linear", pc.PC_LINEAR, 0.0), ("halflife2", pc.PC_HALFLIFE, 2.0), ("halflife4", pc.PC_HALFLIFE, 4.0),
                                  ("halflife8", pc.PC_HALFLIFE, 8.0)):
            total = int(frac * cfg.n_src)
            t = _time(lambda: pack_step(full47, kind, param, total, 0), args.reps, stream)
            cell = {"budget_frac": frac, "decay": name, "retained": min(total, cfg.n_src), "ms_per_layer_frame": round(t, 4),
                    f"ms_per_frame_{args.layers}_layers": round(t * args.layers, 3)}
            grid.append(cell)
            print(json.dumps(cell), flush=True)
    assert pc.pc_poll_status(ctx) == pc.PC_OK
    if args.stack > 0:
        # one frame of the whole stack: every layer has its own seeded K / V / Q (its own compaction, its own attention)
        stack = [D] + [DeviceLayer(wl.make_layer(cfg, layer=i)) for i in range(1, args.stack)]
        dsts = [x.empty_packed(2 * N + 6048) for x in stack]
        avail = np.full(cfg.n_frames, N, np.int32)

        def frame(st):
            for x, d in zip(stack, dsts):
                budget = pc.pc_plan_budget(pc.PC_HALFLIFE, 4.0, 2 * N + 6048, 2, avail)
                pc.pc_score(ctx, x.cache, x.q, x.q_pos, budget, scores=scores, sel_idx=sel, stream=st)
                pc.pc_compact(ctx, x.cache, sel, budget, 0, d, stream=st)
                pc.pc_attend_frame(ctx, d, None, x.q, x.q_pos, out=out, stream=st)

        reps = max(3, args.reps // 4)
        t = _time(lambda: frame(stream), reps, stream)
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        # the same frame captured once into a CUDA graph (8 kernels x layers, programmatic dependencies kept as graph
        # edges) and replayed: the host's planning and launch work leaves the critical path
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            frame(torch.cuda.current_stream())
        tg = _time(graph.replay, reps, torch.cuda.current_stream())
        assert pc.pc_poll_status(ctx) == pc.PC_OK
        print(json.dumps({"stack_layers": args.stack, "history_frames": cfg.n_frames, "ms_per_frame": round(t, 3),
                          "ms_per_layer": round(t / args.stack, 4), "ms_per_frame_cuda_graph": round(tg, 3),
                          "ms_per_layer_cuda_graph": round(tg / args.stack, 4)}), flush=True)
    late = [r for r in rows if r["history_frames"] >= 44]
    print(json.dumps({"summary": "last four frames (44-47 history frames), one layer",
                      "ms_full": round(sum(r["ms_full"] for r in late), 4), "ms_packcache": round(sum(r["ms_packcache"] for r in late), 4),
                      "ms_sliding": round(sum(r["ms_sliding"] for r in late), 4),
                      "speedup_packcache_vs_full": round(sum(r["ms_full"] for r in late) / sum(r["ms_packcache"] for r in late), 2)}))


if __name__ == "__main__":
    main()
