// Cache window: the Fill / Pack / Slide regimes (Sec. 3.4, Fig. 6) and the temporal rebase (Eq. 9) as a host-side state
// machine around pc_plan_budget, pc_score and pc_compact; its one kernel turns a cache mask (Eq. 1) into row indices.
#include <algorithm>
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

namespace {

// What an update has to do, worked out on the host before anything is enqueued.
struct WindowPlan {
    bool fill;               // everything still fits: nothing to do
    pc_cache src;            // source of the pack: the active buffer past the frames that leave
    const int32_t *budget;   // quotas of the frames that stay (points into the window's plan)
    int stay, left;          // frames that stay / leave (beyond the window, or starved by the plan at the old end)
    int64_t n_sel;           // tokens kept
    int32_t delta_t;         // temporal rebase (Eq. 9)
    const float *scores_override;
};

pc_status window_plan(pc_window *w, const float *scores_override, WindowPlan *pl) {
    const int n_frames = (int)w->count.size();
    const int drop = std::max(0, n_frames - w->p.window);          // frames beyond the window leave first (FIFO)
    int64_t dropped_tokens = 0, kept_tokens = 0;
    for (int f = 0; f < n_frames; ++f) (f < drop ? dropped_tokens : kept_tokens) += w->count[f];
    pl->fill = drop == 0 && kept_tokens <= w->p.budget.total;      // Fill: everything still fits
    if (pl->fill) return PC_OK;
    const int kept = n_frames - drop;
    pc_segment &A = w->buf[w->active], &B = w->buf[w->active ^ 1];
    const size_t row = (size_t)w->ctx->desc.n_kv_heads * w->ctx->desc.head_dim * w->ctx->elem_size;
    // source: the active buffer past the dropped frames
    pc_cache &src = pl->src;
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
    pl->budget = w->budget.data() + lead;
    pl->left = drop + lead;
    pl->stay = kept - lead;
    src.history.k = static_cast<char *>(src.history.k) + (size_t)lead_tokens * row;
    src.history.v = static_cast<char *>(src.history.v) + (size_t)lead_tokens * row;
    src.history.pos += 4 * (size_t)lead_tokens;
    src.history.n_tokens -= (int32_t)lead_tokens;
    src.history.capacity -= (int32_t)lead_tokens;
    src.n_frames = pl->stay;
    src.frame_count += lead;
    pl->scores_override = scores_override ? scores_override + lead_tokens : nullptr;
    pl->n_sel = 0;
    for (int f = 0; f < pl->stay; ++f) pl->n_sel += pl->budget[f];
    if (pl->n_sel > B.capacity) return PC_ERR_CAPACITY;
    pl->delta_t = w->p.rebase ? pl->left * w->p.t_step : 0;        // Eq. 9: t falls by the number of frames that left
    return PC_OK;
}

// the other buffer becomes the active one and holds what was kept
void window_commit(pc_window *w, const WindowPlan &pl) {
    pc_segment &A = w->buf[w->active], &B = w->buf[w->active ^ 1];
    B.n_tokens = (int32_t)pl.n_sel;
    A.n_tokens = 0;
    w->active ^= 1;
    w->count.assign(pl.budget, pl.budget + pl.stay);
    w->t_shift += pl.delta_t;
}

}  // namespace

extern "C" pc_status pc_window_update(pc_window *w, const void *q, const int32_t *q_pos, int32_t n_q,
                                      const float *scores_override, int32_t *regime, void *stream) {
    if (!w) return PC_ERR_INVALID_ARG;
    WindowPlan pl;
    pc_status st = window_plan(w, scores_override, &pl);
    if (st != PC_OK) return st;
    if (pl.fill) {
        if (regime) *regime = PC_WINDOW_FILL;
        return PC_OK;
    }
    if (pl.stay > 0) {
        st = pc_score(w->ctx, &pl.src, q, q_pos, n_q, pl.budget, nullptr, pl.scores_override, w->scores, w->sel_idx, stream);
        if (st != PC_OK) return st;
        pc_cache dst;
        dst.anchors = w->anchors;
        dst.history = w->buf[w->active ^ 1];
        dst.n_frames = pl.stay;
        dst.frame_count = pl.budget;
        st = pc_compact(w->ctx, &pl.src, w->sel_idx, pl.budget, pl.delta_t, &dst, stream);
        if (st != PC_OK) return st;
    }
    window_commit(w, pl);
    if (regime) *regime = pl.left ? PC_WINDOW_SLIDE : PC_WINDOW_PACK;
    return PC_OK;
}

extern "C" pc_status pc_window_step(pc_window *w, const void *q, const int32_t *q_pos, int32_t n_q, void *out, float *lse,
                                    int32_t *regime, void *stream) {
    if (!w) return PC_ERR_INVALID_ARG;
    WindowPlan pl;
    pc_status st = window_plan(w, nullptr, &pl);
    if (st != PC_OK) return st;
    if (pl.fill || pl.stay == 0) {
        if (!pl.fill) window_commit(w, pl);
        pc_cache cache;
        cache.anchors = w->anchors;
        cache.history = w->buf[w->active];
        cache.n_frames = (int32_t)w->count.size();
        cache.frame_count = w->count.data();
        st = pc_attend_frame(w->ctx, &cache, nullptr, q, q_pos, n_q, out, lse, stream);
        if (st != PC_OK) return st;
        if (regime) *regime = pl.fill ? PC_WINDOW_FILL : (pl.left ? PC_WINDOW_SLIDE : PC_WINDOW_PACK);
        return PC_OK;
    }
    pc_cache dst;
    dst.anchors = w->anchors;
    dst.history = w->buf[w->active ^ 1];
    dst.n_frames = pl.stay;
    dst.frame_count = pl.budget;
    st = pc_frame_step(w->ctx, &pl.src, pl.budget, pl.delta_t, &dst, q, q_pos, n_q, w->scores, w->sel_idx, out, lse, stream);
    if (st != PC_OK) return st;
    window_commit(w, pl);
    if (regime) *regime = pl.left ? PC_WINDOW_SLIDE : PC_WINDOW_PACK;
    return PC_OK;
}

extern "C" pc_status pc_window_step_host(pc_window *w, const pc_host_window_step *in, const pc_window_step_workspace *ws,
                                         int32_t *regime, void *stream_) {
    if (!w || !in || !ws) return PC_ERR_INVALID_ARG;
    if (!in->q || !in->q_pos || !in->out || in->n_q <= 0 || in->n_frame < 0) return PC_ERR_INVALID_ARG;
    if (!ws->q || !ws->q_pos || !ws->out) return PC_ERR_INVALID_ARG;
    if (in->n_frame > 0 && (!in->frame_k || !in->frame_v || !in->frame_pos)) return PC_ERR_INVALID_ARG;
    if (in->n_q > w->ctx->desc.max_q) return PC_ERR_CAPACITY;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const pc_layer_desc &D = w->ctx->desc;
    const size_t row = (size_t)D.n_kv_heads * D.head_dim * w->ctx->elem_size;
    const size_t qrow = (size_t)D.n_q_heads * D.head_dim * w->ctx->elem_size;
    pc_segment &A = w->buf[w->active];
    const int n = in->n_frame;
    if (n > 0) {
        if ((int64_t)A.n_tokens + n > A.capacity || (int64_t)A.n_tokens + n > w->scratch_capacity) return PC_ERR_CAPACITY;
        if ((int)w->count.size() + 1 > PC_MAX_FRAMES) return PC_ERR_CAPACITY;
    }
    // The plan of the step is tried on the window as it will be with the frame appended (host arithmetic only); if it
    // cannot be made (budget, capacity of the other buffer), the window is left as it was and nothing is enqueued.
    if (n > 0) {
        A.n_tokens += n;
        w->count.push_back(n);
    }
    {
        WindowPlan trial;
        const pc_status st = window_plan(w, nullptr, &trial);
        if (st != PC_OK) {
            if (n > 0) {
                A.n_tokens -= n;
                w->count.pop_back();
            }
            return st;
        }
    }
    // every argument is checked: from here on work is enqueued.  The finished frame goes straight to the end of the
    // active history buffer (no staging copy); the queries follow.
    if (n > 0) {
        const size_t at = (size_t)(A.n_tokens - n);
        PC_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(A.k) + at * row, in->frame_k, (size_t)n * row, cudaMemcpyHostToDevice, stream));
        PC_CUDA_TRY(cudaMemcpyAsync(static_cast<char *>(A.v) + at * row, in->frame_v, (size_t)n * row, cudaMemcpyHostToDevice, stream));
        PC_CUDA_TRY(cudaMemcpyAsync(A.pos + 4 * at, in->frame_pos, (size_t)n * 16, cudaMemcpyHostToDevice, stream));
    }
    PC_CUDA_TRY(cudaMemcpyAsync(ws->q, in->q, (size_t)in->n_q * qrow, cudaMemcpyHostToDevice, stream));
    PC_CUDA_TRY(cudaMemcpyAsync(ws->q_pos, in->q_pos, (size_t)in->n_q * 16, cudaMemcpyHostToDevice, stream));
    pc_status st = pc_window_step(w, ws->q, ws->q_pos, in->n_q, ws->out, nullptr, regime, stream);
    if (st != PC_OK) return st;
    PC_CUDA_TRY(cudaMemcpyAsync(in->out, ws->out, (size_t)in->n_q * qrow, cudaMemcpyDeviceToHost, stream));
    PC_CUDA_TRY(cudaStreamSynchronize(stream));
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
