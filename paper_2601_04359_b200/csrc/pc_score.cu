// Token scoring and per-frame top-k selection (the "attention-relevant" retention of Sec. 3.4).
//
//   k_qpool  : pooled query  q~[g][c] = sum_{h in group g} (1/n_q) sum_i (R(p_i) q_ih)[c]        (fp32, deterministic)
//   k_score  : s_j = 1/(Hq sqrt(d)) * sum_g q~_g . R(p_j) k_jg   — one pass over the history keys, HBM-bound
//   k_select : per frame the budget[f] best scores (ties to the lower index), ascending indices out
//
// The score of a key equals the mean scaled logit over all queries and heads because the logit is linear in the
// rotated query.  For one rotary pair (a, b) = elements (2i, 2i+1):
//   q_a (k_a cos - k_b sin) + q_b (k_a sin + k_b cos) = cos (q_a k_a + q_b k_b) + sin (q_b k_a - q_a k_b),
// and the angle is the same for every KV head, so the two brackets are summed over heads first and each pair costs
// one table look-up per token.
#include "pc_common.cuh"

namespace {

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int PER16 = 4;
    static __device__ __forceinline__ void unpack(const uint4 &v, float *f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int PER16 = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float *f) {
        f[0] = pc_bf16_lo(v.x); f[1] = pc_bf16_hi(v.x); f[2] = pc_bf16_lo(v.y); f[3] = pc_bf16_hi(v.y);
        f[4] = pc_bf16_lo(v.z); f[5] = pc_bf16_hi(v.z); f[6] = pc_bf16_lo(v.w); f[7] = pc_bf16_hi(v.w);
    }
};

// ---------------------------------------------------------------------------------------------------------
// Pooled query.  Block b owns query tokens b, b + gridDim.x, ...; thread t owns rotary pairs t, t + blockDim.x, ...
// of the [Hq][d/2] pair grid and accumulates them in shared memory (one owner per slot, fixed order).  The last
// block to finish adds the per-block partials in block order, so the result does not depend on scheduling.
// ---------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) k_qpool(const T *__restrict__ q, const int32_t *__restrict__ q_pos, int n_q,
                                               int n_q_heads, int group, int d, pc_rope_dev rope,
                                               float *__restrict__ partial, float *__restrict__ pooled,
                                               unsigned int *ticket, int32_t *status) {
    extern __shared__ float acc[];   // [Hq][d]
    __shared__ bool last;
    const int half = d / 2, n_pairs = n_q_heads * half;
    for (int p = threadIdx.x; p < n_pairs; p += blockDim.x) { acc[2 * p] = 0.f; acc[2 * p + 1] = 0.f; }
    for (int i = blockIdx.x; i < n_q; i += gridDim.x) {
        const int4 pp = *reinterpret_cast<const int4 *>(q_pos + 4 * (size_t)i);
        const T *row = q + (size_t)i * n_q_heads * d;
        for (int p = threadIdx.x; p < n_pairs; p += blockDim.x) {
            const int pair = p % half;
            const float2 cs = pc_rope_cs(rope, pair, pp.x, pp.y, pp.z, status, PC_WHERE_QPOOL_POS);
            float x0, x1;
            if constexpr (sizeof(T) == 2) {
                const uint32_t w = *reinterpret_cast<const uint32_t *>(row + 2 * p);
                x0 = pc_bf16_lo(w); x1 = pc_bf16_hi(w);
            } else {
                const float2 w = *reinterpret_cast<const float2 *>(row + 2 * p);
                x0 = w.x; x1 = w.y;
            }
            acc[2 * p] += x0 * cs.x - x1 * cs.y;
            acc[2 * p + 1] += x0 * cs.y + x1 * cs.x;
        }
    }
    __syncthreads();
    // fold the heads of each group, in head order
    const int n_kv = n_q_heads / group, row_len = n_kv * d;
    for (int e = threadIdx.x; e < row_len; e += blockDim.x) {
        const int g = e / d, c = e % d;
        float s = 0.f;
        for (int u = 0; u < group; ++u) s += acc[(g * group + u) * d + c];
        partial[(size_t)blockIdx.x * row_len + e] = s;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    const float inv_n = 1.f / (float)n_q;
    for (int e = threadIdx.x; e < row_len; e += blockDim.x) {
        float s = 0.f;
        for (unsigned b = 0; b < gridDim.x; ++b) s += __ldcg(partial + (size_t)b * row_len + e);
        pooled[e] = s * inv_n;
    }
    if (threadIdx.x == 0) *ticket = 0u;   // ready for the next call
}

// ---------------------------------------------------------------------------------------------------------
// Score: one warp per token.  A token's K row over all KV heads is CH = Hkv*d/PER16 16-byte chunks; lane l reads
// chunks l, l+32, ... .  Because 32*PER16 is a multiple of d, all of a lane's chunks cover the same PER16/2 rotary
// pairs (of different heads), so the lane sums the two brackets over its chunks and needs PER16/2 table look-ups.
// Two tokens are in flight per warp to keep enough bytes outstanding.
// ---------------------------------------------------------------------------------------------------------
template <typename T, int CPL /* chunks per lane */>
__global__ void __launch_bounds__(256) k_score(const T *__restrict__ k, const int32_t *__restrict__ k_pos,
                                               const uint8_t *__restrict__ valid, int n_src, int d, float scale,
                                               pc_rope_dev rope, const float *__restrict__ pooled,
                                               float *__restrict__ scores, int32_t *status) {
    constexpr int PER = Elem<T>::PER16, NP = PER / 2;
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int n_warps = (gridDim.x * blockDim.x) >> 5;
    const size_t row_bytes = (size_t)CPL * 32 * 16;

    // this lane's slice of the pooled query stays in registers
    float qv[CPL][PER];
#pragma unroll
    for (int c = 0; c < CPL; ++c)
#pragma unroll
        for (int e = 0; e < PER; ++e) qv[c][e] = pooled[(size_t)(c * 32 + lane) * PER + e];
    const int pair0 = ((lane * PER) % d) / 2;

    for (int j0 = warp * 2; j0 < n_src; j0 += n_warps * 2) {
        uint4 raw[2][CPL];
        int4 pp[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int j = min(j0 + t, n_src - 1);
            const char *row = reinterpret_cast<const char *>(k) + (size_t)j * row_bytes;
#pragma unroll
            for (int c = 0; c < CPL; ++c) raw[t][c] = pc_ldg_stream(row + (size_t)(c * 32 + lane) * 16);
            pp[t] = __ldg(reinterpret_cast<const int4 *>(k_pos) + j);
        }
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int j = j0 + t;
            float A[NP], B[NP];
#pragma unroll
            for (int u = 0; u < NP; ++u) { A[u] = 0.f; B[u] = 0.f; }
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                float kv[PER];
                Elem<T>::unpack(raw[t][c], kv);
#pragma unroll
                for (int u = 0; u < NP; ++u) {
                    const float qa = qv[c][2 * u], qb = qv[c][2 * u + 1], ka = kv[2 * u], kb = kv[2 * u + 1];
                    A[u] = fmaf(qa, ka, fmaf(qb, kb, A[u]));
                    B[u] = fmaf(qb, ka, fmaf(-qa, kb, B[u]));
                }
            }
            float s = 0.f;
#pragma unroll
            for (int u = 0; u < NP; ++u) {
                const float2 cs = pc_rope_cs(rope, pair0 + u, pp[t].x, pp[t].y, pp[t].z, status, PC_WHERE_SCORE_POS);
                s = fmaf(cs.x, A[u], fmaf(cs.y, B[u], s));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0 && j < n_src) {
                float r = s * scale;
                if (valid && !valid[j]) r = -INFINITY;
                scores[j] = r;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// Select.  One block per frame.  Scores map to 32-bit keys whose unsigned order is the score order (-0 folded onto
// +0).  An 8-bit-digit radix descent finds the key T of the budget-th best token and how many keys beat it; a final
// ordered sweep keeps every key > T and the lowest-index (budget - beaten) keys == T, writing ascending indices.
// ---------------------------------------------------------------------------------------------------------
struct FrameTab { int4 f[PC_MAX_FRAMES]; };   // (first token, tokens, budget, output offset)

__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    if ((u << 1) == 0) u = 0;                       // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int SEL_THREADS = 512;

__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_sums, int &total) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();                                // warp_sums may still be read from the previous call
    if (lane == 31) warp_sums[w] = inc;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < SEL_THREADS / 32; ++i) {
        int s = warp_sums[i];
        if (i < w) base += s;
        tot += s;
    }
    total = tot;
    return base + inc - v;
}

__global__ void __launch_bounds__(SEL_THREADS) k_select(const float *__restrict__ scores, const __grid_constant__ FrameTab tab,
                                                       int32_t *__restrict__ sel_idx, int32_t *status) {
    __shared__ int hist[256];
    __shared__ int warp_sums[SEL_THREADS / 32];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_want;
    const int4 fr = tab.f[blockIdx.x];
    const int first = fr.x, n = fr.y, budget = fr.z, out0 = fr.w;
    if (budget <= 0 || n <= 0) return;
    const float *s = scores + first;

    uint32_t prefix = 0, mask = 0;
    int want = budget;                               // rank, among keys matching the prefix, of the threshold key
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int b = threadIdx.x; b < 256; b += SEL_THREADS) hist[b] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
            const float v = s[j];
            if (v != v) pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_SELECT_NAN);
            const uint32_t key = score_key(v);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int w = want, b = 255;
            for (; b > 0; --b) {
                if (hist[b] >= w) break;
                w -= hist[b];
            }
            sh_prefix = prefix | ((uint32_t)b << shift);
            sh_want = w;
        }
        __syncthreads();
        prefix = sh_prefix;
        want = sh_want;
        mask |= 255u << shift;
        __syncthreads();
    }
    // prefix is now the threshold key T; `want` of the keys equal to T are kept, lowest indices first
    const uint32_t T = prefix;
    int eq_seen = 0, written = 0;
    for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
        const int j = j0 + threadIdx.x;
        uint32_t key = 0;
        const bool in = j < n;
        if (in) key = score_key(s[j]);
        const int is_eq = in && key == T;
        int eq_total, keep_total;
        const int eq_rank = eq_seen + block_exclusive_scan(is_eq, warp_sums, eq_total);
        const int keep = in && (key > T || (is_eq && eq_rank < want));
        const int at = written + block_exclusive_scan(keep, warp_sums, keep_total);
        if (keep && at < budget) sel_idx[out0 + at] = first + j;
        eq_seen += eq_total;
        written += keep_total;
    }
}

template <typename T>
pc_status launch_score(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q,
                       const uint8_t *valid, float *scores, cudaStream_t stream) {
    const pc_layer_desc &D = ctx->desc;
    const int row = D.n_kv_heads * D.head_dim;
    const int n_src = src->history.n_tokens;
    const int pool_blocks = std::min<int>(PC_QPOOL_BLOCKS, n_q);
    const size_t smem = (size_t)D.n_q_heads * D.head_dim * sizeof(float);
    if (smem > 48 * 1024)
        PC_CUDA_TRY(cudaFuncSetAttribute(k_qpool<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    pc_mark(ctx, PC_MARK_SCORE0, stream);
    k_qpool<T><<<pool_blocks, 256, smem, stream>>>(static_cast<const T *>(q), q_pos, n_q, D.n_q_heads, ctx->group,
                                                   D.head_dim, ctx->rope, ctx->qpool_partial, ctx->qpool, ctx->ticket,
                                                   ctx->status);
    PC_CUDA_TRY(cudaGetLastError());
    pc_mark(ctx, PC_MARK_QPOOL, stream);
    const float scale = (float)(1.0 / ((double)D.n_q_heads * std::sqrt((double)D.head_dim)));
    const int chunks = row / Elem<T>::PER16;          // 16-byte chunks per token row
    const int warps_needed = (n_src + 1) / 2;
    const int blocks = std::max(1, std::min((warps_needed + 7) / 8, ctx->sm_count * 6));
    const T *k = static_cast<const T *>(src->history.k);
#define PC_SCORE_CASE(CPL)                                                                                          \
    case CPL:                                                                                                       \
        k_score<T, CPL><<<blocks, 256, 0, stream>>>(k, src->history.pos, valid, n_src, D.head_dim, scale, ctx->rope, \
                                                    ctx->qpool, scores, ctx->status);                              \
        break;
    if (chunks % 32) return PC_ERR_UNSUPPORTED;
    switch (chunks / 32) {
        PC_SCORE_CASE(1) PC_SCORE_CASE(2) PC_SCORE_CASE(3) PC_SCORE_CASE(4) PC_SCORE_CASE(6) PC_SCORE_CASE(8)
    default: return PC_ERR_UNSUPPORTED;
    }
#undef PC_SCORE_CASE
    PC_CUDA_TRY(cudaGetLastError());
    pc_mark(ctx, PC_MARK_SCORE, stream);
    return PC_OK;
}

}  // namespace

extern "C" pc_status pc_score(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q,
                              const int32_t *budget, const uint8_t *valid, const float *scores_override, float *scores,
                              int32_t *sel_idx, void *stream_) {
    if (!ctx || !src || !budget) return PC_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int n_frames = src->n_frames;
    if (n_frames < 0 || (n_frames > 0 && !src->frame_count)) return PC_ERR_INVALID_ARG;
    if (n_frames > PC_MAX_FRAMES) return PC_ERR_CAPACITY;
    pc_status st = pc_check_segment(&src->history, true);
    if (st != PC_OK) return st;
    const int n_src = src->history.n_tokens;
    if (n_src > ctx->desc.max_keys) return PC_ERR_CAPACITY;
    FrameTab tab;
    int64_t first = 0, out = 0;
    for (int f = 0; f < n_frames; ++f) {
        const int n = src->frame_count[f], b = budget[f];
        if (n < 0 || b < 0) return PC_ERR_INVALID_ARG;
        if (b > n) return PC_ERR_BUDGET;
        tab.f[f] = make_int4((int)first, n, b, (int)out);
        first += n;
        out += b;
    }
    if (first != n_src) return PC_ERR_INVALID_ARG;
    if (out > 0 && (!sel_idx || !pc_aligned16(sel_idx))) return PC_ERR_INVALID_ARG;
    const float *select_on = scores_override;
    if (!scores_override) {
        if (n_src > 0) {
            if (!q || !q_pos || n_q <= 0 || !scores) return PC_ERR_INVALID_ARG;
            if (!pc_aligned16(q) || !pc_aligned16(q_pos) || !pc_aligned16(scores)) return PC_ERR_INVALID_ARG;
            if (n_q > ctx->desc.max_q) return PC_ERR_CAPACITY;
            st = ctx->desc.dtype == PC_BF16
                     ? launch_score<__nv_bfloat16>(ctx, src, q, q_pos, n_q, valid, scores, stream)
                     : launch_score<float>(ctx, src, q, q_pos, n_q, valid, scores, stream);
            if (st != PC_OK) return st;
        }
        select_on = scores;
    } else if (!pc_aligned16(scores_override)) {
        return PC_ERR_INVALID_ARG;
    }
    if (n_frames > 0 && out > 0) {
        if (scores_override) pc_mark(ctx, PC_MARK_SCORE, stream);
        k_select<<<n_frames, SEL_THREADS, 0, stream>>>(select_on, tab, sel_idx, ctx->status);
        PC_CUDA_TRY(cudaGetLastError());
        pc_mark(ctx, PC_MARK_SELECT, stream);
    }
    return PC_OK;
}

// ---------------------------------------------------------------------------------------------------------
// Scoring without a context and without any allocation.
//
// Meant for hosts that cannot call cudaMalloc at the point where they need scores: a process whose device memory
// was handed to its own arena at start-up and whose policy forbids driver allocations afterwards, or a
// latency-critical thread that cannot take the device-wide synchronisation a cudaMalloc / cudaFree implies.  Such
// callers cannot create a pc_ctx (pc_create allocates), so everything a context would hold for scoring — the rotary
// table, the pooled query and its per-block partials, the completion ticket — lives in one file-scope device array
// of fixed size that every GPU loading this library carries until the process exits.
//
// In host code the array's name is only a handle; the device address is obtained once per device with
// cudaGetSymbolAddress while that device is current, and that pointer (never the symbol) is what kernels receive.
// ---------------------------------------------------------------------------------------------------------
namespace {

constexpr int STATIC_MAX_ROW = 1024;          // n_kv_heads * head_dim
constexpr int STATIC_MAX_ROPE = 32768;        // rotary table entries: sum over axes of max_pos * pairs on that axis
constexpr int STATIC_MAX_DEVICES = 64;

constexpr size_t STATIC_OFF_TICKET = 0;                                                    // unsigned, 256-byte slot
constexpr size_t STATIC_OFF_POOLED = 256;                                                  // float [STATIC_MAX_ROW]
constexpr size_t STATIC_OFF_PARTIAL = STATIC_OFF_POOLED + STATIC_MAX_ROW * sizeof(float);  // float [64][STATIC_MAX_ROW]
constexpr size_t STATIC_OFF_ROPE = STATIC_OFF_PARTIAL + (size_t)PC_QPOOL_BLOCKS * STATIC_MAX_ROW * sizeof(float);
constexpr size_t STATIC_BYTES = STATIC_OFF_ROPE + (size_t)STATIC_MAX_ROPE * sizeof(float2);   // 528,640 bytes

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

// Rotary table in fp64, stored as fp32 (cos, sin): entry (axis a, position p, column m) = p * base^(-m / n_axis[a]).
__global__ void __launch_bounds__(256) k_rope_table(float2 *__restrict__ tab, pc_rope_dev rope, double base, int total) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const int a = e >= rope.off[2] ? 2 : (e >= rope.off[1] ? 1 : 0);
    const int na = rope.n_axis[a], local = e - rope.off[a];
    const int p = local / na, m = local % na;
    const double ang = (double)p * pow(base, -(double)m / (double)na);
    tab[e] = make_float2((float)cos(ang), (float)sin(ang));
}

// Device address of the static scratch on the current device; looked up on the first call per device.
pc_status static_scratch_base(unsigned char **base) {
    static unsigned char *addr[STATIC_MAX_DEVICES] = {};
    int dev = -1;
    PC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return PC_ERR_UNSUPPORTED;
    unsigned char *p = __atomic_load_n(&addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        void *sym = nullptr;
        PC_CUDA_TRY(cudaGetSymbolAddress(&sym, g_static_scratch));
        if (!sym) return PC_ERR_CUDA;
        p = static_cast<unsigned char *>(sym);
        __atomic_store_n(&addr[dev], p, __ATOMIC_RELEASE);   // every thread resolves the same address
    }
    *base = p;
    return PC_OK;
}

template <typename T>
pc_status launch_score_static(const pc_layer_desc &D, unsigned char *base, const void *hist_k, const int32_t *hist_pos,
                              int32_t n_src, const void *q, const int32_t *q_pos, int32_t n_q, const uint8_t *valid,
                              float *scores, int32_t *status, cudaStream_t stream) {
    unsigned int *ticket = reinterpret_cast<unsigned int *>(base + STATIC_OFF_TICKET);
    float *pooled = reinterpret_cast<float *>(base + STATIC_OFF_POOLED);
    float *partial = reinterpret_cast<float *>(base + STATIC_OFF_PARTIAL);
    float2 *tab = reinterpret_cast<float2 *>(base + STATIC_OFF_ROPE);

    pc_rope_dev rope;
    int total = 0;
    for (int a = 0; a < 3; ++a) {
        rope.n_axis[a] = (D.head_dim / 2 - a + 2) / 3;
        rope.max_pos[a] = D.max_pos[a];
        rope.off[a] = total;
        total += D.max_pos[a] * rope.n_axis[a];
    }
    rope.tab = tab;
    // the array keeps whatever the last call left: the ticket must start at zero, the table is rewritten
    PC_CUDA_TRY(cudaMemsetAsync(ticket, 0, sizeof(unsigned int), stream));
    k_rope_table<<<(total + 255) / 256, 256, 0, stream>>>(tab, rope, D.rope_base, total);
    PC_CUDA_TRY(cudaGetLastError());

    const int row = D.n_kv_heads * D.head_dim;
    const int pool_blocks = std::min<int>(PC_QPOOL_BLOCKS, n_q);
    const size_t smem = (size_t)D.n_q_heads * D.head_dim * sizeof(float);
    k_qpool<T><<<pool_blocks, 256, smem, stream>>>(static_cast<const T *>(q), q_pos, n_q, D.n_q_heads,
                                                   D.n_q_heads / D.n_kv_heads, D.head_dim, rope, partial, pooled, ticket,
                                                   status);
    PC_CUDA_TRY(cudaGetLastError());
    const float scale = (float)(1.0 / ((double)D.n_q_heads * std::sqrt((double)D.head_dim)));
    const int chunks = row / Elem<T>::PER16;
    const int warps_needed = (n_src + 1) / 2;
    int sm_count = 0, dev = 0;
    PC_CUDA_TRY(cudaGetDevice(&dev));
    PC_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    const int blocks = std::max(1, std::min((warps_needed + 7) / 8, sm_count * 6));
    const T *k = static_cast<const T *>(hist_k);
#define PC_SCORE_CASE(CPL)                                                                                         \
    case CPL:                                                                                                      \
        k_score<T, CPL><<<blocks, 256, 0, stream>>>(k, hist_pos, valid, n_src, D.head_dim, scale, rope, pooled, scores, \
                                                    status);                                                      \
        break;
    switch (chunks / 32) {
        PC_SCORE_CASE(1) PC_SCORE_CASE(2) PC_SCORE_CASE(3) PC_SCORE_CASE(4) PC_SCORE_CASE(6) PC_SCORE_CASE(8)
    default: return PC_ERR_UNSUPPORTED;
    }
#undef PC_SCORE_CASE
    PC_CUDA_TRY(cudaGetLastError());
    return PC_OK;
}

}  // namespace

extern "C" pc_status pc_score_tokens_static(const pc_layer_desc *desc, const void *hist_k, const int32_t *hist_pos,
                                            int32_t n_src, const void *q, const int32_t *q_pos, int32_t n_q,
                                            const uint8_t *valid, float *scores, int32_t *status, void *stream_) {
    if (!desc || !hist_k || !hist_pos || !q || !q_pos || !scores || !status || n_src <= 0 || n_q <= 0)
        return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(hist_k) || !pc_aligned16(hist_pos) || !pc_aligned16(q) || !pc_aligned16(q_pos) ||
        !pc_aligned16(scores) || (reinterpret_cast<uintptr_t>(status) & 7u))
        return PC_ERR_INVALID_ARG;
    const pc_layer_desc &D = *desc;
    if (D.head_dim != 64 && D.head_dim != 128) return PC_ERR_UNSUPPORTED;
    if (D.dtype != PC_F32 && D.dtype != PC_BF16) return PC_ERR_UNSUPPORTED;
    if (D.n_q_heads <= 0 || D.n_kv_heads <= 0 || D.n_q_heads % D.n_kv_heads) return PC_ERR_UNSUPPORTED;
    if (!(D.rope_base > 1.0)) return PC_ERR_INVALID_ARG;
    const int row = D.n_kv_heads * D.head_dim;
    const int chunks = row / (D.dtype == PC_BF16 ? 8 : 4);
    if (chunks % 32) return PC_ERR_UNSUPPORTED;
    int64_t rope_entries = 0;
    for (int a = 0; a < 3; ++a) {
        if (D.max_pos[a] <= 0 || D.max_pos[a] > (1 << 20)) return PC_ERR_INVALID_ARG;
        rope_entries += (int64_t)D.max_pos[a] * ((D.head_dim / 2 - a + 2) / 3);
    }
    if (row > STATIC_MAX_ROW || rope_entries > STATIC_MAX_ROPE ||
        (size_t)D.n_q_heads * D.head_dim * sizeof(float) > 48 * 1024) {
        fprintf(stderr,
                "packcache: pc_score_tokens_static: shape exceeds the fixed scratch (n_kv_heads*head_dim %d > %d, or "
                "rotary table %lld > %d entries, or n_q_heads*head_dim > 12288)\n",
                row, STATIC_MAX_ROW, (long long)rope_entries, STATIC_MAX_ROPE);
        return PC_ERR_CAPACITY;
    }
    unsigned char *base = nullptr;
    pc_status st = static_scratch_base(&base);
    if (st != PC_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    return D.dtype == PC_BF16
               ? launch_score_static<__nv_bfloat16>(D, base, hist_k, hist_pos, n_src, q, q_pos, n_q, valid, scores, status, stream)
               : launch_score_static<float>(D, base, hist_k, hist_pos, n_src, q, q_pos, n_q, valid, scores, status, stream);
}
