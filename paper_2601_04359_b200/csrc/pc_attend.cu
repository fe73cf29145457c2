// pc_attend_frame: argument checks and the choice of attention kernel.
#include "pc_common.cuh"

extern "C" pc_status pc_attend_frame(pc_ctx *ctx, const pc_cache *cache, const pc_segment *current, const void *q,
                                     const int32_t *q_pos, int32_t n_q, void *out, float *lse, void *stream_) {
    if (!ctx || !cache || !q || !q_pos || !out || n_q <= 0) return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(q) || !pc_aligned16(q_pos) || !pc_aligned16(out) || (lse && !pc_aligned16(lse)))
        return PC_ERR_INVALID_ARG;
    if (n_q > ctx->desc.max_q) return PC_ERR_CAPACITY;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    pc_segment segs[PC_MAX_SEGMENTS];
    int n_seg = 0;
    int64_t n_keys = 0;
    const pc_segment *cand[3] = {&cache->anchors, &cache->history, current};
    for (int i = 0; i < 3; ++i) {
        if (!cand[i]) continue;
        pc_status st = pc_check_segment(cand[i], true);
        if (st != PC_OK) return st;
        if (cand[i]->n_tokens == 0) continue;
        segs[n_seg++] = *cand[i];
        n_keys += cand[i]->n_tokens;
    }
    if (n_keys == 0) return PC_ERR_INVALID_ARG;
    if (n_keys > ctx->desc.max_keys) return PC_ERR_CAPACITY;
    if (ctx->desc.dtype == PC_BF16 && ctx->attend_impl == 0 && ctx->desc.head_dim == 128)
        return pc_launch_attend_tc(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream);
    return pc_launch_attend_simt(ctx, n_seg, segs, q, q_pos, n_q, out, lse, stream);
}
