// pc_attend_frame and the prepare / prepared pair: argument checks and the choice of attention kernel.
#include "pc_common.cuh"

namespace {

// anchors ++ history ++ current, empty segments dropped
pc_status gather_segments(pc_ctx *ctx, const pc_cache *cache, const pc_segment *current, pc_segment *segs, int *n_seg) {
    *n_seg = 0;
    int64_t n_keys = 0;
    const pc_segment *cand[3] = {&cache->anchors, &cache->history, current};
    for (int i = 0; i < 3; ++i) {
        if (!cand[i]) continue;
        pc_status st = pc_check_segment(cand[i], true);
        if (st != PC_OK) return st;
        if (cand[i]->n_tokens == 0) continue;
        segs[(*n_seg)++] = *cand[i];
        n_keys += cand[i]->n_tokens;
    }
    if (n_keys == 0) return PC_ERR_INVALID_ARG;
    if (n_keys > ctx->desc.max_keys) return PC_ERR_CAPACITY;
    return PC_OK;
}

pc_status check_queries(pc_ctx *ctx, const void *q, const int32_t *q_pos, int32_t n_q, void *out, float *lse) {
    if (!q || !q_pos || !out || n_q <= 0) return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(q) || !pc_aligned16(q_pos) || !pc_aligned16(out) || (lse && !pc_aligned16(lse))) return PC_ERR_INVALID_ARG;
    if (n_q > ctx->desc.max_q) return PC_ERR_CAPACITY;
    return PC_OK;
}

bool tensor_core_path(const pc_ctx *ctx) {
    return ctx->attend_impl != 1 && pc_tensor_core_shape(ctx);
}

}  // namespace

extern "C" pc_status pc_attend_frame(pc_ctx *ctx, const pc_cache *cache, const pc_segment *current, const void *q,
                                     const int32_t *q_pos, int32_t n_q, void *out, float *lse, void *stream_) {
    if (!ctx || !cache) return PC_ERR_INVALID_ARG;
    pc_status st = check_queries(ctx, q, q_pos, n_q, out, lse);
    if (st != PC_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    pc_segment segs[PC_MAX_SEGMENTS];
    int n_seg = 0;
    st = gather_segments(ctx, cache, current, segs, &n_seg);
    if (st != PC_OK) return st;
    ctx->last_n_q = 0;
    if (tensor_core_path(ctx)) {
        ctx->prepared_n_seg = 0;                       // the rotated-key scratch is about to be overwritten
        ctx->anchor_rot_n = 0;
        return pc_launch_attend_tc(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream, PC_TC_ALL);
    }
    return pc_launch_attend_simt(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream);
}

extern "C" pc_status pc_attend_prepare(pc_ctx *ctx, const pc_cache *cache, const pc_segment *current, void *stream_) {
    if (!ctx || !cache) return PC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    pc_segment segs[PC_MAX_SEGMENTS];
    int n_seg = 0;
    pc_status st = gather_segments(ctx, cache, current, segs, &n_seg);
    if (st != PC_OK) return st;
    ctx->prepared_n_seg = 0;
    ctx->last_n_q = 0;
    if (tensor_core_path(ctx)) {
        ctx->anchor_rot_n = 0;
        st = pc_launch_attend_tc(ctx, n_seg, segs, nullptr, nullptr, 0, nullptr, nullptr, stream, PC_TC_ROPE_K);
        if (st != PC_OK) return st;
    }
    for (int i = 0; i < n_seg; ++i) ctx->prepared_seg[i] = segs[i];
    ctx->prepared_n_seg = n_seg;
    return PC_OK;
}

extern "C" pc_status pc_attend_prepared(pc_ctx *ctx, const void *q, const int32_t *q_pos, int32_t n_q, void *out, float *lse,
                                        void *stream_) {
    if (!ctx) return PC_ERR_INVALID_ARG;
    if (ctx->prepared_n_seg <= 0) return PC_ERR_INVALID_ARG;      // no key set prepared (or overwritten since)
    pc_status st = check_queries(ctx, q, q_pos, n_q, out, lse);
    if (st != PC_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    ctx->last_n_q = 0;
    if (tensor_core_path(ctx))
        return pc_launch_attend_tc(ctx, ctx->prepared_n_seg, ctx->prepared_seg, q, q_pos, n_q, out, lse, stream,
                                   PC_TC_ROPE_Q | PC_TC_ATTEND);
    return pc_launch_attend_simt(ctx, ctx->prepared_n_seg, ctx->prepared_seg, q, q_pos, n_q, out, lse, stream);
}

// One frame of the steady state in one call: score -> select -> pack -> attend over anchors ++ packed history.  On the
// tensor-core path the intermediate passes of the separate calls disappear: the query pass that pools for the scores also
// leaves the rotated queries, the pack kernel also leaves the rotated keys of what it packs, and the anchors' rotated
// keys stay in the scratch from the first step that saw them, so attention starts without a rotary pre-pass.
extern "C" pc_status pc_frame_step(pc_ctx *ctx, const pc_cache *src, const int32_t *budget, int32_t delta_t, pc_cache *dst,
                                   const void *q, const int32_t *q_pos, int32_t n_q, float *scores, int32_t *sel_idx, void *out,
                                   float *lse, void *stream_) {
    if (!ctx || !src || !dst || !budget) return PC_ERR_INVALID_ARG;
    pc_status st = check_queries(ctx, q, q_pos, n_q, out, lse);
    if (st != PC_OK) return st;
    if (src->n_frames < 0 || (src->n_frames > 0 && !src->frame_count)) return PC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int64_t n_sel = 0;
    for (int f = 0; f < src->n_frames; ++f) {
        if (budget[f] < 0) return PC_ERR_INVALID_ARG;
        n_sel += budget[f];
    }
    if (n_sel > dst->history.capacity) return PC_ERR_CAPACITY;
    st = pc_check_segment(&src->anchors, true);
    if (st != PC_OK) return st;
    const int n_anchor = src->anchors.n_tokens;
    if (n_anchor + n_sel == 0) return PC_ERR_INVALID_ARG;
    if (n_anchor + n_sel > ctx->desc.max_keys) return PC_ERR_CAPACITY;
    const bool tc = tensor_core_path(ctx);
    const int tile = 128;
    const int anchor_tiles = (n_anchor + tile - 1) / tile;
    void *k_rot_dst = nullptr;
    if (tc) {
        if ((size_t)(anchor_tiles + (n_sel + tile - 1) / tile) * tile > ctx->k_rot_rows) return PC_ERR_CAPACITY;
        const size_t row_bytes = (size_t)ctx->desc.n_kv_heads * ctx->desc.head_dim * sizeof(__nv_bfloat16);
        k_rot_dst = static_cast<char *>(ctx->k_rot) + (size_t)anchor_tiles * tile * row_bytes;
        ctx->prepared_n_seg = 0;                       // the scratch no longer holds a key set of pc_attend_prepare
    }
    // what the pack stage would refuse (a destination that overlaps the source, a misaligned or missing buffer) is refused
    // now, before the scoring stage enqueues anything
    st = pc_compact_check(ctx, src, sel_idx, budget, dst, nullptr, nullptr);
    if (st != PC_OK) return st;
    ctx->last_n_q = 0;
    ctx->q_rot_n = 0;
    st = pc_score_impl(ctx, src, q, q_pos, n_q, budget, nullptr, nullptr, scores, sel_idx, tc ? ctx->q_rot : nullptr, stream);
    if (st != PC_OK) return st;
    st = pc_compact_impl(ctx, src, sel_idx, budget, delta_t, dst, k_rot_dst, stream);
    if (st != PC_OK) return st;
    dst->history.n_tokens = (int32_t)n_sel;
    dst->n_frames = src->n_frames;

    pc_segment segs[PC_MAX_SEGMENTS];
    int n_seg = 0;
    if (n_anchor > 0) segs[n_seg++] = src->anchors;
    if (n_sel > 0) segs[n_seg++] = dst->history;
    if (!tc) return pc_launch_attend_simt(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream);
    int what = PC_TC_ATTEND;
    if (ctx->q_rot_n != n_q) what |= PC_TC_ROPE_Q;    // nothing was scored, so no query pass ran: rotate the queries now
    const bool anchors_cached = n_anchor > 0 && ctx->anchor_rot_n == n_anchor && ctx->anchor_rot_k == src->anchors.k &&
                                ctx->anchor_rot_pos == src->anchors.pos;
    if (n_anchor > 0 && !anchors_cached) what |= PC_TC_ROPE_K0;
    ctx->anchor_rot_n = 0;
    st = pc_launch_attend_tc(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream, what);
    if (st != PC_OK) return st;
    if (n_anchor > 0) {
        ctx->anchor_rot_k = src->anchors.k;
        ctx->anchor_rot_pos = src->anchors.pos;
        ctx->anchor_rot_n = n_anchor;
    }
    return PC_OK;
}
