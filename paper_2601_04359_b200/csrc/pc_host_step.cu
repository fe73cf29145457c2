// One whole frame step driven from host memory: copy in, plan, score, select, pack, attend, copy out.
#include <vector>

#include "pc_common.cuh"

extern "C" pc_status pc_frame_step_host(pc_ctx *ctx, const pc_host_frame *in, pc_device_workspace *ws,
                                        const pc_budget_params *params, int32_t delta_t, void *stream_) {
    if (!ctx || !in || !ws || !params) return PC_ERR_INVALID_ARG;
    if (!in->q || !in->q_pos || !in->out || in->n_q <= 0 || in->n_frames < 0 || in->n_anchor < 0) return PC_ERR_INVALID_ARG;
    if (in->n_frames > 0 && !in->frame_count) return PC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const pc_layer_desc &D = ctx->desc;
    const size_t row = (size_t)D.n_kv_heads * D.head_dim * ctx->elem_size;
    const size_t qrow = (size_t)D.n_q_heads * D.head_dim * ctx->elem_size;
    int64_t n_src = 0;
    for (int f = 0; f < in->n_frames; ++f) {
        if (in->frame_count[f] < 0) return PC_ERR_INVALID_ARG;
        n_src += in->frame_count[f];
    }
    if (n_src > ws->src.history.capacity || in->n_anchor > ws->src.anchors.capacity) return PC_ERR_CAPACITY;
    if (!ws->q || !ws->q_pos || !ws->out || (n_src > 0 && (!ws->scores || !ws->sel_idx))) return PC_ERR_INVALID_ARG;
    // every argument is checked before the first copy is enqueued
    if (in->n_anchor > 0 && (!in->anchor_k || !in->anchor_v || !in->anchor_pos || !ws->src.anchors.k || !ws->src.anchors.v ||
                             !ws->src.anchors.pos))
        return PC_ERR_INVALID_ARG;
    if (n_src > 0 && (!in->hist_k || !in->hist_v || !in->hist_pos || !ws->src.history.k || !ws->src.history.v ||
                      !ws->src.history.pos || !ws->dst.history.k || !ws->dst.history.v || !ws->dst.history.pos))
        return PC_ERR_INVALID_ARG;
    if (in->n_q > ctx->desc.max_q) return PC_ERR_CAPACITY;

    std::vector<int32_t> budget((size_t)std::max(in->n_frames, 1));
    pc_status st = pc_plan_budget(params, in->n_frames, in->frame_count, budget.data());
    if (st != PC_OK) return st;
    int64_t n_sel = 0;
    for (int f = 0; f < in->n_frames; ++f) n_sel += budget[f];
    if (n_sel > ws->dst.history.capacity) return PC_ERR_CAPACITY;

    // host -> device: this step's inputs
    PC_CUDA_TRY(cudaMemcpyAsync(ws->q, in->q, (size_t)in->n_q * qrow, cudaMemcpyHostToDevice, stream));
    PC_CUDA_TRY(cudaMemcpyAsync(ws->q_pos, in->q_pos, (size_t)in->n_q * 16, cudaMemcpyHostToDevice, stream));
    if (in->n_anchor > 0) {
        PC_CUDA_TRY(cudaMemcpyAsync(ws->src.anchors.k, in->anchor_k, in->n_anchor * row, cudaMemcpyHostToDevice, stream));
        PC_CUDA_TRY(cudaMemcpyAsync(ws->src.anchors.v, in->anchor_v, in->n_anchor * row, cudaMemcpyHostToDevice, stream));
        PC_CUDA_TRY(cudaMemcpyAsync(ws->src.anchors.pos, in->anchor_pos, (size_t)in->n_anchor * 16, cudaMemcpyHostToDevice, stream));
    }
    if (n_src > 0) {
        PC_CUDA_TRY(cudaMemcpyAsync(ws->src.history.k, in->hist_k, n_src * row, cudaMemcpyHostToDevice, stream));
        PC_CUDA_TRY(cudaMemcpyAsync(ws->src.history.v, in->hist_v, n_src * row, cudaMemcpyHostToDevice, stream));
        PC_CUDA_TRY(cudaMemcpyAsync(ws->src.history.pos, in->hist_pos, (size_t)n_src * 16, cudaMemcpyHostToDevice, stream));
    }
    pc_cache src = ws->src;
    src.anchors.n_tokens = in->n_anchor;
    src.history.n_tokens = (int32_t)n_src;
    src.n_frames = in->n_frames;
    src.frame_count = in->frame_count;
    pc_cache dst = ws->dst;
    dst.anchors = src.anchors;
    dst.history.n_tokens = (int32_t)n_sel;
    dst.n_frames = in->n_frames;
    dst.frame_count = budget.data();
    if (n_src > 0) {
        st = pc_score(ctx, &src, ws->q, ws->q_pos, in->n_q, budget.data(), nullptr, nullptr, ws->scores, ws->sel_idx, stream);
        if (st != PC_OK) return st;
        st = pc_compact(ctx, &src, ws->sel_idx, budget.data(), delta_t, &dst, stream);
        if (st != PC_OK) return st;
    }
    st = pc_attend_frame(ctx, &dst, nullptr, ws->q, ws->q_pos, in->n_q, ws->out, nullptr, stream);
    if (st != PC_OK) return st;
    PC_CUDA_TRY(cudaMemcpyAsync(in->out, ws->out, (size_t)in->n_q * qrow, cudaMemcpyDeviceToHost, stream));
    PC_CUDA_TRY(cudaStreamSynchronize(stream));
    return PC_OK;
}
