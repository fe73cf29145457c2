// Context management, the host-side budget planner and status plumbing of the PackCache library.
#include <algorithm>
#include <cmath>
#include <new>
#include <vector>

#include "pc_common.cuh"

bool pc_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

pc_status pc_check_segment(const pc_segment *s, bool allow_empty) {
    if (!s) return PC_ERR_INVALID_ARG;
    if (s->n_tokens < 0 || s->capacity < s->n_tokens) return PC_ERR_INVALID_ARG;
    if (s->n_tokens == 0) return allow_empty ? PC_OK : PC_ERR_INVALID_ARG;
    if (!s->k || !s->v || !s->pos) return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(s->k) || !pc_aligned16(s->v) || !pc_aligned16(s->pos)) return PC_ERR_INVALID_ARG;
    return PC_OK;
}

extern "C" const char *pc_status_string(pc_status s) {
    switch (s) {
    case PC_OK: return "ok";
    case PC_ERR_INVALID_ARG: return "invalid argument";
    case PC_ERR_BUDGET: return "budget exceeds what a frame holds";
    case PC_ERR_CAPACITY: return "capacity exceeded";
    case PC_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case PC_ERR_CUDA: return "CUDA runtime error";
    case PC_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

static int pairs_of_axis(int n_pairs, int axis) { return (n_pairs - axis + 2) / 3; }

static pc_status create_on_device(pc_ctx *c) {
    const pc_layer_desc *desc = &c->desc;
    PC_CUDA_TRY(cudaGetDevice(&c->device));
    PC_CUDA_TRY(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device));

    // rotary tables in fp64 on the host, stored as fp32 (cos, sin)
    const int n_pairs = desc->head_dim / 2;
    size_t total = 0;
    for (int a = 0; a < 3; ++a) {
        c->rope.n_axis[a] = pairs_of_axis(n_pairs, a);
        c->rope.max_pos[a] = desc->max_pos[a];
        c->rope.off[a] = (int32_t)total;
        total += (size_t)desc->max_pos[a] * c->rope.n_axis[a];
    }
    std::vector<float2> tab(total);
    for (int a = 0; a < 3; ++a) {
        const int na = c->rope.n_axis[a];
        for (int m = 0; m < na; ++m) {
            const double freq = std::pow(desc->rope_base, -(double)m / (double)na);
            for (int p = 0; p < desc->max_pos[a]; ++p) {
                const double ang = (double)p * freq;
                tab[c->rope.off[a] + (size_t)p * na + m] = make_float2((float)std::cos(ang), (float)std::sin(ang));
            }
        }
    }
    const int row = desc->n_kv_heads * desc->head_dim;
    PC_CUDA_TRY(cudaMalloc(&c->rope_tab, total * sizeof(float2)));
    PC_CUDA_TRY(cudaMemcpy(c->rope_tab, tab.data(), total * sizeof(float2), cudaMemcpyHostToDevice));
    c->rope.tab = c->rope_tab;
    PC_CUDA_TRY(cudaMalloc(&c->status, 2 * sizeof(int32_t)));
    PC_CUDA_TRY(cudaMemset(c->status, 0, 2 * sizeof(int32_t)));
    PC_CUDA_TRY(cudaMallocHost(&c->host_status, 2 * sizeof(int32_t)));
    PC_CUDA_TRY(cudaMalloc(&c->qpool_fx, ((size_t)PC_FX_REPLICAS * row + 1) * sizeof(long long)));
    PC_CUDA_TRY(cudaMemset(c->qpool_fx, 0, ((size_t)PC_FX_REPLICAS * row + 1) * sizeof(long long)));
    PC_CUDA_TRY(cudaMalloc(&c->qpool, (size_t)row * sizeof(float)));
    if (desc->dtype == PC_BF16) {
        pc_status st = pc_attend_tc_scratch(desc, c->sm_count, &c->k_rot_rows, &c->part_o_floats, &c->part_ml_floats);
        if (st != PC_OK) return st;
        PC_CUDA_TRY(cudaMalloc(&c->k_rot, c->k_rot_rows * row * sizeof(__nv_bfloat16)));
        PC_CUDA_TRY(cudaMemset(c->k_rot, 0, c->k_rot_rows * row * sizeof(__nv_bfloat16)));
        PC_CUDA_TRY(cudaMalloc(&c->q_rot, (size_t)desc->max_q * desc->n_q_heads * desc->head_dim * sizeof(__nv_bfloat16)));
        PC_CUDA_TRY(cudaMalloc(&c->part_o, std::max<size_t>(c->part_o_floats, 1) * sizeof(float)));
        PC_CUDA_TRY(cudaMalloc(&c->part_ml, std::max<size_t>(c->part_ml_floats, 1) * sizeof(float)));
        PC_CUDA_TRY(cudaMalloc(&c->mass_part, c->k_rot_rows * desc->n_kv_heads * 2 * sizeof(float)));
        PC_CUDA_TRY(cudaMalloc(&c->mass_norm, (size_t)((desc->max_q + 127) / 128) * 128 * desc->n_q_heads * sizeof(float)));
    }
    return PC_OK;
}

extern "C" pc_status pc_create(const pc_layer_desc *desc, pc_ctx **out) {
    if (!desc || !out) return PC_ERR_INVALID_ARG;
    *out = nullptr;
    if (desc->head_dim != 64 && desc->head_dim != 128) return PC_ERR_UNSUPPORTED;
    if (desc->dtype != PC_F32 && desc->dtype != PC_BF16) return PC_ERR_UNSUPPORTED;
    if (desc->n_q_heads <= 0 || desc->n_kv_heads <= 0 || desc->n_q_heads % desc->n_kv_heads) return PC_ERR_UNSUPPORTED;
    if (desc->n_kv_heads * desc->head_dim > 4096) return PC_ERR_UNSUPPORTED;
    if (!(desc->rope_base > 1.0)) return PC_ERR_INVALID_ARG;
    if (desc->max_q <= 0 || desc->max_keys <= 0) return PC_ERR_INVALID_ARG;
    for (int a = 0; a < 3; ++a)
        if (desc->max_pos[a] <= 0 || desc->max_pos[a] > (1 << 20)) return PC_ERR_INVALID_ARG;

    pc_ctx *c = new (std::nothrow) pc_ctx();       // value-initialised: every pointer starts out null
    if (!c) return PC_ERR_CUDA;
    c->desc = *desc;
    c->group = desc->n_q_heads / desc->n_kv_heads;
    c->elem_size = desc->dtype == PC_BF16 ? 2 : 4;
    const pc_status st = create_on_device(c);
    if (st != PC_OK) {                             // one way out on failure: whatever was allocated so far is released
        pc_destroy(c);
        return st;
    }
    *out = c;
    return PC_OK;
}

extern "C" pc_status pc_destroy(pc_ctx *c) {
    if (!c) return PC_ERR_INVALID_ARG;
    cudaFree(c->rope_tab);
    cudaFree(c->status);
    if (c->host_status) cudaFreeHost(c->host_status);
    cudaFree(c->qpool_fx);
    cudaFree(c->qpool);
    for (int i = 0; i < PC_N_MARKS; ++i)
        if (c->ev[i]) cudaEventDestroy(c->ev[i]);
    cudaFree(c->k_rot);
    cudaFree(c->q_rot);
    cudaFree(c->part_o);
    cudaFree(c->part_ml);
    cudaFree(c->mass_part);
    cudaFree(c->mass_norm);
    delete c;
    return PC_OK;
}

extern "C" pc_status pc_set_attend_impl(pc_ctx *c, int32_t impl) {
    if (!c || impl < 0 || impl > 1) return PC_ERR_INVALID_ARG;
    c->attend_impl = impl;
    return PC_OK;
}

extern "C" pc_status pc_set_wait_limit_us(pc_ctx *c, uint32_t limit_us) {
    if (!c) return PC_ERR_INVALID_ARG;
    c->wait_limit_us = limit_us;
    return PC_OK;
}

extern "C" pc_status pc_test_expect_extra_bytes(pc_ctx *c, uint32_t n_bytes) {
    if (!c) return PC_ERR_INVALID_ARG;
    c->test_extra_tx = n_bytes;
    return PC_OK;
}

extern "C" pc_status pc_forget_anchors(pc_ctx *c) {
    if (!c) return PC_ERR_INVALID_ARG;
    c->anchor_rot_n = 0;
    return PC_OK;
}

extern "C" pc_status pc_set_kv_splits(pc_ctx *c, int32_t n) {
    if (!c || n < 0 || n > 4) return PC_ERR_INVALID_ARG;
    c->kv_splits = n;
    return PC_OK;
}

extern "C" pc_status pc_set_cluster_merge(pc_ctx *c, int32_t on) {
    if (!c || on < 0 || on > 1) return PC_ERR_INVALID_ARG;
    c->cluster_merge = on;
    return PC_OK;
}

extern "C" pc_status pc_set_timing(pc_ctx *c, int32_t on) {
    if (!c) return PC_ERR_INVALID_ARG;
    if (on)
        for (int i = 0; i < PC_N_MARKS; ++i)
            if (!c->ev[i]) PC_CUDA_TRY(cudaEventCreate(&c->ev[i]));
    c->timing_on = on ? 1 : 0;
    c->ev_mask = 0;
    return PC_OK;
}

extern "C" pc_status pc_get_timing(pc_ctx *c, float *ms) {
    if (!c || !ms) return PC_ERR_INVALID_ARG;
    // (first mark, last mark) of each stage; the attention kernel starts at the rotary pre-pass's end mark when that
    // pre-pass ran in the call, else at the call's first mark
    static const int span[PC_N_STAGES][2] = {{PC_MARK_SCORE0, PC_MARK_QPOOL}, {PC_MARK_QPOOL, PC_MARK_SCORE},
                                             {PC_MARK_SCORE, PC_MARK_SELECT}, {PC_MARK_PACK0, PC_MARK_PACK},
                                             {PC_MARK_ATT0, PC_MARK_ROPE},    {PC_MARK_ROPE, PC_MARK_ATTEND},
                                             {PC_MARK_ATTEND, PC_MARK_COMBINE}, {PC_MARK_MASS0, PC_MARK_MASS}};
    for (int s = 0; s < PC_N_STAGES; ++s) {
        ms[s] = -1.f;
        int a = span[s][0];
        const int b = span[s][1];
        if (s == PC_STAGE_ATTEND && !((c->ev_mask >> a) & 1u)) a = PC_MARK_ATT0;
        if (!((c->ev_mask >> a) & 1u) || !((c->ev_mask >> b) & 1u)) continue;
        PC_CUDA_TRY(cudaEventSynchronize(c->ev[b]));
        PC_CUDA_TRY(cudaEventElapsedTime(&ms[s], c->ev[a], c->ev[b]));
    }
    return PC_OK;
}

extern "C" pc_status pc_set_timing_skip(pc_ctx *c, uint32_t mark_mask) {
    if (!c) return PC_ERR_INVALID_ARG;
    c->ev_skip = mark_mask;
    c->ev_mask = 0;
    return PC_OK;
}

extern "C" pc_status pc_get_span(pc_ctx *c, int32_t a, int32_t b, float *ms) {
    if (!c || !ms || a < 0 || b < 0 || a >= PC_N_MARKS || b >= PC_N_MARKS) return PC_ERR_INVALID_ARG;
    *ms = -1.f;
    if (!((c->ev_mask >> a) & 1u) || !((c->ev_mask >> b) & 1u)) return PC_OK;
    PC_CUDA_TRY(cudaEventSynchronize(c->ev[b]));
    PC_CUDA_TRY(cudaEventElapsedTime(ms, c->ev[a], c->ev[b]));
    return PC_OK;
}

extern "C" pc_status pc_poll_status(pc_ctx *c, void *stream) {
    if (!c) return PC_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    PC_CUDA_TRY(cudaMemcpyAsync(c->host_status, c->status, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    PC_CUDA_TRY(cudaMemsetAsync(c->status, 0, 2 * sizeof(int32_t), s));
    PC_CUDA_TRY(cudaStreamSynchronize(s));
    int code = c->host_status[0];
    if (code < 0 || code > PC_ERR_TIMEOUT) return PC_ERR_CUDA;
    return static_cast<pc_status>(code);
}

// ---------------------------------------------------------------------------------------------------------
// Budget planner (Sec. 3.4, Eq. 5-8).  Fixed-point weights, then integer largest-remainder apportionment with
// capping at what each frame holds.
// ---------------------------------------------------------------------------------------------------------
namespace {

typedef unsigned __int128 u128;

struct Share {
    int frame;         // index oldest -> newest
    uint64_t weight;   // g(dist) in units of 2^-32
    uint64_t rem_hi, rem_lo;
};

uint64_t decay_weight_q32(int kind, double param, int dist, int W, int keep_full) {
    double g = 0.0;
    switch (kind) {
    case PC_GEOMETRIC: g = std::pow(param, (double)dist); break;
    case PC_CLOSED_HALF: g = std::ldexp(1.0, -std::min(dist, W - 1)); break;
    case PC_LINEAR: g = (double)(W + 1 - dist); break;
    case PC_HALFLIFE: g = std::exp2(-(double)(dist - 1 - keep_full) / param); break;
    }
    return (uint64_t)std::floor(g * 4294967296.0 + 0.5);
}

}  // namespace

extern "C" pc_status pc_plan_budget(const pc_budget_params *p, int32_t n_frames, const int32_t *avail, int32_t *budget) {
    if (!p || n_frames < 0 || (n_frames > 0 && (!avail || !budget))) return PC_ERR_INVALID_ARG;
    if (p->total < 0 || p->keep_full < 0 || p->min_quota < 0) return PC_ERR_INVALID_ARG;
    if (p->kind < PC_GEOMETRIC || p->kind > PC_HALFLIFE) return PC_ERR_INVALID_ARG;
    if (p->kind == PC_GEOMETRIC && !(p->param > 0.0 && p->param < 1.0)) return PC_ERR_INVALID_ARG;
    if (p->kind == PC_HALFLIFE && !(p->param > 0.0)) return PC_ERR_INVALID_ARG;
    const int W = n_frames;
    for (int f = 0; f < W; ++f)
        if (avail[f] < 0) return PC_ERR_INVALID_ARG;

    int64_t remaining = p->total;
    std::vector<Share> live;
    for (int f = 0; f < W; ++f) {
        const int dist = W - f;
        budget[f] = 0;
        if (dist <= p->keep_full) {
            budget[f] = avail[f];
            remaining -= avail[f];
        } else {
            live.push_back(Share{f, decay_weight_q32(p->kind, p->param, dist, W, p->keep_full), 0, 0});
        }
    }
    if (remaining < 0) return PC_ERR_BUDGET;

    // Minimum quota (b_min of Sec. 3.4).  `live` runs oldest -> newest.  If every live frame's guarantee does not fit the
    // budget, the oldest frames leave the window (first in, first out) until the guarantees of the rest do; each frame
    // that stays is granted min(min_quota, what it holds) up front, and only its remaining room competes for the rest.
    std::vector<int32_t> granted((size_t)W, 0), room_of((size_t)W, 0);
    for (int f = 0; f < W; ++f) room_of[f] = avail[f];
    if (p->min_quota > 0) {
        const int64_t fits = remaining / p->min_quota;
        if ((int64_t)live.size() > fits) live.erase(live.begin(), live.end() - (size_t)fits);
        for (const Share &s : live) {
            granted[s.frame] = std::min<int32_t>(p->min_quota, avail[s.frame]);
            room_of[s.frame] -= granted[s.frame];
            remaining -= granted[s.frame];
        }
    }
    avail = room_of.data();          // from here on a frame's capacity is what is left above its guarantee

    while (!live.empty() && remaining > 0) {
        u128 weight_sum = 0;
        int64_t room = 0;
        for (const Share &s : live) {
            weight_sum += s.weight;
            room += avail[s.frame];
        }
        if (weight_sum == 0) break;
        if (remaining >= room) {
            for (const Share &s : live) budget[s.frame] = avail[s.frame];
            break;
        }
        int64_t handed = 0;
        for (Share &s : live) {
            const u128 num = (u128)remaining * s.weight;
            budget[s.frame] = (int32_t)(num / weight_sum);
            const u128 rem = num % weight_sum;
            s.rem_hi = (uint64_t)(rem >> 64);
            s.rem_lo = (uint64_t)rem;
            handed += budget[s.frame];
        }
        // left-over units: one each, largest remainder first, equal remainders to the nearer (later) frame
        std::vector<const Share *> order;
        for (const Share &s : live) order.push_back(&s);
        std::sort(order.begin(), order.end(), [](const Share *a, const Share *b) {
            if (a->rem_hi != b->rem_hi) return a->rem_hi > b->rem_hi;
            if (a->rem_lo != b->rem_lo) return a->rem_lo > b->rem_lo;
            return a->frame > b->frame;
        });
        const int64_t left = remaining - handed;
        for (int64_t i = 0; i < left && i < (int64_t)order.size(); ++i) budget[order[i]->frame] += 1;
        // frames granted more than they hold keep what they hold and leave; the rest is shared again
        std::vector<Share> next;
        bool capped = false;
        for (const Share &s : live) {
            if (budget[s.frame] > avail[s.frame]) {
                budget[s.frame] = avail[s.frame];
                remaining -= avail[s.frame];
                capped = true;
            } else {
                next.push_back(s);
            }
        }
        if (!capped) break;
        for (const Share &s : next) budget[s.frame] = 0;
        live.swap(next);
    }
    for (int f = 0; f < W; ++f) budget[f] += granted[f];
    return PC_OK;
}
