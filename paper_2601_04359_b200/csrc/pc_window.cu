// Cache window: the Fill / Pack / Slide regimes (Sec. 3.4, Fig. 6) and the temporal rebase (Eq. 9) as a host-side state
// machine around pc_plan_budget, pc_score and pc_compact; its one kernel turns a cache mask (Eq. 1) into row indices.
#include <vector>

#include "pc_common.cuh"

struct pc_window {
    pc_ctx *ctx;
    pc_window_params p;
    pc_segment anchors;
    pc_segment buf[2];
    int active;
    std::vector<int32_t> count;      // tokens per retained frame, oldest -> newest
    std::vector<int32_t> budget;     // scratch of the last plan
    int64_t t_shift;
    float *scores;
    int32_t *sel_idx;
    int32_t scratch_capacity;
};

extern "C" pc_status pc_window_create(pc_ctx *ctx, const pc_window_params *params, const pc_segment *anchors,
                                      const pc_segment *hist_a, const pc_segment *hist_b, float *scores, int32_t *sel_idx,
                                      pc_window **out) {
    if (!ctx || !params || !anchors || !hist_a || !hist_b || !scores || !sel_idx || !out) return PC_ERR_INVALID_ARG;
    *out = nullptr;
    if (params->window < 1 || params->window >= PC_MAX_FRAMES || params->t_step < 0 || params->budget.total < 0)
        return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(scores) || !pc_aligned16(sel_idx)) return PC_ERR_INVALID_ARG;
    pc_status st = pc_check_segment(anchors, true);
    if (st != PC_OK) return st;
    const pc_segment *hb[2] = {hist_a, hist_b};
    for (int i = 0; i < 2; ++i) {
        if (hb[i]->capacity <= 0 || !hb[i]->k || !hb[i]->v || !hb[i]->pos) return PC_ERR_INVALID_ARG;
        if (!pc_aligned16(hb[i]->k) || !pc_aligned16(hb[i]->v) || !pc_aligned16(hb[i]->pos)) return PC_ERR_INVALID_ARG;
    }
    pc_window *w = new (std::nothrow) pc_window();
    if (!w) return PC_ERR_CUDA;
    w->ctx = ctx;
    w->p = *params;
    w->anchors = *anchors;
    w->buf[0] = *hist_a;
    w->buf[1] = *hist_b;
    w->buf[0].n_tokens = w->buf[1].n_tokens = 0;
    w->active = 0;
    w->t_shift = 0;
    w->scores = scores;
    w->sel_idx = sel_idx;
    w->scratch_capacity = std::min(hist_a->capacity, hist_b->capacity);
    *out = w;
    return PC_OK;
}

extern "C" pc_status pc_window_destroy(pc_window *w) {
    if (!w) return PC_ERR_INVALID_ARG;
    delete w;
    return PC_OK;
}

extern "C" pc_status pc_window_append(pc_window *w, const pc_segment *frame, void *stream_) {
    if (!w || !frame) return PC_ERR_INVALID_ARG;
    pc_status st = pc_check_segment(frame, false);
    if (st != PC_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    pc_segment &A = w->buf[w->active];
    const int n = frame->n_tokens;
    if ((int64_t)A.n_tokens + n > A.capacity || (int64_t)A.n_tokens + n > w->scratch_capacity) return PC_ERR_CAPACITY;
    if ((int)w->count.size() + 1 > PC_MAX_FRAMES) return PC_ERR_CAPACITY;
    const size_t row = (size_t)w->ctx->desc.n_kv_heads * w->ctx->desc.head_dim * w->ctx->elem_size;
    char *k = static_cast<char *>(A.k) + (size_t)A.n_tokens * row, *v = static_cast<char *>(A.v) + (size_t)A.n_tokens * row;
    PC_CUDA_TRY(cudaMemcpyAsync(k, frame->k, (size_t)n * row, cudaMemcpyDeviceToDevice, stream));
    PC_CUDA_TRY(cudaMemcpyAsync(v, frame->v, (size_t)n * row, cudaMemcpyDeviceToDevice, stream));
    PC_CUDA_TRY(cudaMemcpyAsync(A.pos + 4 * (size_t)A.n_tokens, frame->pos, (size_t)n * 16, cudaMemcpyDeviceToDevice, stream));
    A.n_tokens += n;
    w->count.push_back(n);
    return PC_OK;
}

namespace {

// Indices of the non-zero bytes of valid[0..n), ascending, into idx; one block, a scan per 1024 bytes.  The host states how
// many there are (it sizes the frame table without a device round trip): a different count is recorded as an error.
__global__ void __launch_bounds__(1024) k_mask_to_index(const uint8_t *__restrict__ valid, int n, int32_t *__restrict__ idx,
                                                        int expected, int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    __shared__ int warp_sums[32];
    __shared__ int carry;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int j0 = 0; j0 < n; j0 += 1024) {
        const int j = j0 + threadIdx.x;
        const int keep = j < n && valid[j] != 0;
        int inc = keep;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        if (lane == 31) warp_sums[w] = inc;
        __syncthreads();
        int base = carry;
        for (int i = 0; i < w; ++i) base += warp_sums[i];
        const int at = base + inc - keep;
        if (keep && at < expected) idx[at] = j;
        __syncthreads();
        if (threadIdx.x == 1023) carry = base + inc;
        __syncthreads();
    }
    if (threadIdx.x == 0 && carry != expected) pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_MASK_COUNT);
}

}  // namespace

extern "C" pc_status pc_window_append_masked(pc_window *w, const pc_segment *frame, const uint8_t *valid, int32_t n_valid,
                                             void *stream_) {
    if (!w || !frame || !valid) return PC_ERR_INVALID_ARG;
    pc_status st = pc_check_segment(frame, false);
    if (st != PC_OK) return st;
    if (n_valid < 0 || n_valid > frame->n_tokens) return PC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    pc_segment &A = w->buf[w->active];
    // the grown buffer must fit the caller's score / index scratch as well (the next update scores every token of it), and
    // the mask's row indices go through that index scratch
    if ((int64_t)A.n_tokens + n_valid > A.capacity || (int64_t)A.n_tokens + n_valid > w->scratch_capacity ||
        frame->n_tokens > w->scratch_capacity)
        return PC_ERR_CAPACITY;
    if ((int)w->count.size() + 1 > PC_MAX_FRAMES) return PC_ERR_CAPACITY;
    if (n_valid > 0) {
        const size_t row = (size_t)w->ctx->desc.n_kv_heads * w->ctx->desc.head_dim * w->ctx->elem_size;
        PC_LAUNCH(k_mask_to_index, dim3(1), dim3(1024), 0, stream, valid, (int)frame->n_tokens, w->sel_idx, (int)n_valid,
                  w->ctx->status);
        st = pc_launch_pack(w->ctx, frame->k, frame->v, frame->pos, w->sel_idx, n_valid, frame->n_tokens, 0,
                            static_cast<char *>(A.k) + (size_t)A.n_tokens * row, static_cast<char *>(A.v) + (size_t)A.n_tokens * row,
                            A.pos + 4 * (size_t)A.n_tokens, nullptr, stream);
        if (st != PC_OK) return st;
    }
    A.n_tokens += n_valid;
    w->count.push_back(n_valid);
    return PC_OK;
}

extern "C" pc_status pc_window_update(pc_window *w, const void *q, const int32_t *q_pos, int32_t n_q,
                                      const float *scores_override, int32_t *regime, void *stream) {
    if (!w) return PC_ERR_INVALID_ARG;
    const int n_frames = (int)w->count.size();
    const int drop = std::max(0, n_frames - w->p.window);          // frames beyond the window leave first (FIFO)
    int64_t dropped_tokens = 0, kept_tokens = 0;
    for (int f = 0; f < n_frames; ++f) (f < drop ? dropped_tokens : kept_tokens) += w->count[f];
    if (drop == 0 && kept_tokens <= w->p.budget.total) {           // Fill: everything still fits
        if (regime) *regime = PC_WINDOW_FILL;
        return PC_OK;
    }
    const int kept = n_frames - drop;
    pc_segment &A = w->buf[w->active], &B = w->buf[w->active ^ 1];
    const size_t row = (size_t)w->ctx->desc.n_kv_heads * w->ctx->desc.head_dim * w->ctx->elem_size;
    // source: the active buffer past the dropped frames
    pc_cache src;
    src.anchors = w->anchors;
    src.history.k = static_cast<char *>(A.k) + (size_t)dropped_tokens * row;
    src.history.v = static_cast<char *>(A.v) + (size_t)dropped_tokens * row;
    src.history.pos = A.pos + 4 * (size_t)dropped_tokens;
    src.history.n_tokens = (int32_t)kept_tokens;
    src.history.capacity = (int32_t)(A.capacity - dropped_tokens);
    src.n_frames = kept;
    src.frame_count = w->count.data() + drop;
    w->budget.assign((size_t)std::max(kept, 1), 0);
    pc_status st = pc_plan_budget(&w->p.budget, kept, src.frame_count, w->budget.data());
    if (st != PC_OK) return st;
    // Frames that the plan leaves with nothing at the old end (a minimum quota starves the oldest frames first) leave the
    // window like frames beyond W: first in, first out, counted in the rebase.
    int lead = 0;
    int64_t lead_tokens = 0;
    while (lead < kept && w->budget[lead] == 0) lead_tokens += src.frame_count[lead++];
    const int32_t *budget = w->budget.data() + lead;
    const int left = drop + lead, stay = kept - lead;
    src.history.k = static_cast<char *>(src.history.k) + (size_t)lead_tokens * row;
    src.history.v = static_cast<char *>(src.history.v) + (size_t)lead_tokens * row;
    src.history.pos += 4 * (size_t)lead_tokens;
    src.history.n_tokens -= (int32_t)lead_tokens;
    src.history.capacity -= (int32_t)lead_tokens;
    src.n_frames = stay;
    src.frame_count += lead;
    if (scores_override) scores_override += lead_tokens;
    int64_t n_sel = 0;
    for (int f = 0; f < stay; ++f) n_sel += budget[f];
    if (n_sel > B.capacity) return PC_ERR_CAPACITY;
    const int32_t delta_t = w->p.rebase ? left * w->p.t_step : 0;  // Eq. 9: t falls by the number of frames that left
    if (stay > 0) {
        st = pc_score(w->ctx, &src, q, q_pos, n_q, budget, nullptr, scores_override, w->scores, w->sel_idx, stream);
        if (st != PC_OK) return st;
        pc_cache dst;
        dst.anchors = w->anchors;
        dst.history = B;
        dst.n_frames = stay;
        dst.frame_count = budget;
        st = pc_compact(w->ctx, &src, w->sel_idx, budget, delta_t, &dst, stream);
        if (st != PC_OK) return st;
    }
    B.n_tokens = (int32_t)n_sel;
    A.n_tokens = 0;
    w->active ^= 1;
    w->count.assign(budget, budget + stay);
    w->t_shift += delta_t;
    if (regime) *regime = left ? PC_WINDOW_SLIDE : PC_WINDOW_PACK;
    return PC_OK;
}

extern "C" pc_status pc_window_cache(pc_window *w, pc_cache *out) {
    if (!w || !out) return PC_ERR_INVALID_ARG;
    out->anchors = w->anchors;
    out->history = w->buf[w->active];
    out->n_frames = (int32_t)w->count.size();
    out->frame_count = w->count.data();
    return PC_OK;
}

extern "C" pc_status pc_window_state(pc_window *w, int32_t *n_frames, int32_t *counts, int64_t *t_shift, int32_t *active) {
    if (!w) return PC_ERR_INVALID_ARG;
    if (n_frames) *n_frames = (int32_t)w->count.size();
    if (counts)
        for (size_t f = 0; f < w->count.size(); ++f) counts[f] = w->count[f];
    if (t_shift) *t_shift = w->t_shift;
    if (active) *active = w->active;
    return PC_OK;
}
