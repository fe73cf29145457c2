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
