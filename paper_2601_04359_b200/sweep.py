"""Latency of the cache strategies over a whole 48-frame generation on one GPU (synthetic lumos-shaped layer).

    python -m paper_2601_04359_b200.sweep [--reps 10] [--layers 28] [--stack 28] [--markdown]

Three strategies, as in the paper's comparison (Sec. 3.3 / Sec. 4, Fig. 1, Tab. 2): the full KV cache (every history
frame attended), a sliding window (anchors plus the most recent frame: a cache window of one frame), and PackCache
(anchors plus the compacted history: the two newest frames whole and 6048 tokens over the rest at half-life 4,
one-shot compaction every frame through the fused frame step).  For every history depth 1 ... 47 the script times one
layer's frame step (compaction, where there is one, plus attention of the 1008 current-frame queries) with CUDA events
and prints one JSON line with the per-frame time and the running total of each strategy (the per-frame and the
cumulative curve of Fig. 1; TOTAL and LAST of Tab. 2 are the last total and the sum over the last four frames).  Then
the budget x decay grid of the 28-layer configuration (budget 10 / 25 / 50 / 100 % of the history, decay linear or
half-life 2 / 4 / 8) over the depth of the generation: per-frame time at sampled depths, the total over all 47 frames
and the last four.  `--layers` only scales a per-layer time to a stack of identical layers; `--stack N` times one frame
through N distinct layers.  `--markdown` also prints the two tables as markdown.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as pc
from . import workload as wl
from .device import DeviceLayer, make_ctx

GRID_DECAYS = (("linear", pc.PC_LINEAR, 0.0), ("halflife2", pc.PC_HALFLIFE, 2.0), ("halflife4", pc.PC_HALFLIFE, 4.0),
               ("halflife8", pc.PC_HALFLIFE, 8.0))
GRID_FRACS = (0.10, 0.25, 0.50, 1.00)


def _time(fn, reps, stream):
    for _ in range(2):
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
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--layers", type=int, default=28)
    ap.add_argument("--grid-depths", type=str, default="4,8,16,24,32,40,47", help="depths printed for the budget x decay grid")
    ap.add_argument("--stack", type=int, default=0, help="also time one frame through this many distinct layers (5.6 GB at 28)")
    ap.add_argument("--markdown", action="store_true")
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
        pc.pc_frame_step(ctx, cache, budget, 0, dst, D.q, D.q_pos, scores=scores, sel_idx=sel, out=out, stream=stream)

    # ---- the three strategies over the whole generation: per frame and cumulative
    rows, tot = [], {"full": 0.0, "pack": 0.0, "slide": 0.0}
    for F in range(1, cfg.n_frames + 1):
        full = history(cfg.n_frames - F, F)                   # the F most recent frames
        last = history(cfg.n_frames - 1, 1)
        t_full = _time(lambda: pc.pc_attend_frame(ctx, full, None, D.q, D.q_pos, out=out, stream=stream), args.reps, stream)
        t_slide = _time(lambda: pc.pc_attend_frame(ctx, last, None, D.q, D.q_pos, out=out, stream=stream), args.reps, stream)
        t_pack = _time(lambda: pack_step(full, pc.PC_HALFLIFE, 4.0, 2 * N + 6048, 2), args.reps, stream)
        tot["full"] += t_full; tot["pack"] += t_pack; tot["slide"] += t_slide
        row = {"history_frames": F, "keys_full": cfg.n_anchor + F * N, "ms_full": round(t_full, 4), "ms_packcache": round(t_pack, 4),
               "ms_sliding": round(t_slide, 4), "total_full": round(tot["full"], 3), "total_packcache": round(tot["pack"], 3),
               "total_sliding": round(tot["slide"], 3), "speedup_vs_full": round(t_full / t_pack, 2)}
        rows.append(row)
        print(json.dumps(row), flush=True)
    assert pc.pc_poll_status(ctx) == pc.PC_OK
    late = rows[-4:]
    summary = {"summary": "one layer, 47 generated frames after the first (history depth 1 ... 47)",
               "TOTAL_ms": {"full": round(tot["full"], 3), "packcache": round(tot["pack"], 3), "sliding": round(tot["slide"], 3)},
               "LAST4_ms": {"full": round(sum(r["ms_full"] for r in late), 4), "packcache": round(sum(r["ms_packcache"] for r in late), 4),
                            "sliding": round(sum(r["ms_sliding"] for r in late), 4)},
               "speedup_total": round(tot["full"] / tot["pack"], 2),
               "speedup_last4": round(sum(r["ms_full"] for r in late) / sum(r["ms_packcache"] for r in late), 2)}
    print(json.dumps(summary), flush=True)

    # ---- budget x decay grid over the depth of the generation (the budget is a fraction of the history at that depth)
    grid_depths = [int(x) for x in args.grid_depths.split(",")]
    grid = []
    for frac in GRID_FRACS:
        for name, kind, param in GRID_DECAYS:
            per = []
            for F in range(1, cfg.n_frames + 1):
                cache = history(cfg.n_frames - F, F)
                per.append(_time(lambda: pack_step(cache, kind, param, int(frac * F * N), 0), max(3, args.reps // 2), stream))
            cell = {"budget_frac": frac, "decay": name, "ms_at_depth": {str(F): round(per[F - 1], 4) for F in grid_depths},
                    "total_ms_per_layer": round(sum(per), 3), "last4_ms_per_layer": round(sum(per[-4:]), 4),
                    f"total_ms_{args.layers}_layers": round(sum(per) * args.layers, 1)}
            grid.append(cell)
            print(json.dumps(cell), flush=True)
    assert pc.pc_poll_status(ctx) == pc.PC_OK

    stack_line = None
    if args.stack > 0:
        # one frame of the whole stack: every layer has its own seeded K / V / Q, its own context (rotated anchors kept),
        # its own compaction and attention
        stack = [D] + [DeviceLayer(wl.make_layer(cfg, layer=i)) for i in range(1, args.stack)]
        ctxs = [ctx] + [make_ctx(cfg, max_keys=cfg.n_anchor + cfg.n_src) for _ in range(1, args.stack)]
        dsts = [x.empty_packed(2 * N + 6048) for x in stack]
        avail = np.full(cfg.n_frames, N, np.int32)

        def frame(st):
            for x, c, d in zip(stack, ctxs, dsts):
                budget = pc.pc_plan_budget(pc.PC_HALFLIFE, 4.0, 2 * N + 6048, 2, avail)
                pc.pc_frame_step(c, x.cache, budget, 0, d, x.q, x.q_pos, scores=scores, sel_idx=sel, out=out, stream=st)

        reps = max(3, args.reps // 2)
        t = _time(lambda: frame(stream), reps, stream)
        assert all(pc.pc_poll_status(c) == pc.PC_OK for c in ctxs)
        # the same frame captured once into a CUDA graph (6 kernels x layers, programmatic dependencies kept as graph
        # edges) and replayed: the host's planning and launch work leaves the critical path
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            frame(torch.cuda.current_stream())
        tg = _time(graph.replay, reps, torch.cuda.current_stream())
        assert all(pc.pc_poll_status(c) == pc.PC_OK for c in ctxs)
        stack_line = {"stack_layers": args.stack, "history_frames": cfg.n_frames, "ms_per_frame": round(t, 3),
                      "ms_per_layer": round(t / args.stack, 4), "ms_per_frame_cuda_graph": round(tg, 3),
                      "ms_per_layer_cuda_graph": round(tg / args.stack, 4)}
        print(json.dumps(stack_line), flush=True)

    if args.markdown:
        print("\n| history frames | keys (full) | full cache | PackCache | sliding window | full / PackCache | total full | total PackCache | total sliding |")
        print("|---|---|---|---|---|---|---|---|---|")
        for r in rows:
            if r["history_frames"] in (1, 2, 4, 8, 12, 16, 24, 32, 40, 44, 45, 46, 47):
                print(f"| {r['history_frames']} | {r['keys_full']:,} | {r['ms_full']:.3f} | {r['ms_packcache']:.3f} | {r['ms_sliding']:.3f} | "
                      f"{r['speedup_vs_full']:.2f} | {r['total_full']:.2f} | {r['total_packcache']:.2f} | {r['total_sliding']:.2f} |")
        print("\n| budget | decay | " + " | ".join(f"depth {F}" for F in grid_depths) + " | total (47 frames) | last four |")
        print("|---|---|" + "---|" * (len(grid_depths) + 2))
        for c in grid:
            print(f"| {int(c['budget_frac'] * 100)} % | {c['decay']} | " + " | ".join(f"{c['ms_at_depth'][str(F)]:.3f}" for F in grid_depths) +
                  f" | {c['total_ms_per_layer']:.2f} | {c['last4_ms_per_layer']:.3f} |")


if __name__ == "__main__":
    main()
