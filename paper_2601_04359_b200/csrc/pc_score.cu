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
// Pooled query.  The rotation is the same for every head at a given token and rotary pair, so the heads of a group
// are added first and the sum is rotated once:  q~[g] = (1/n_q) sum_i R(p_i) (sum_{h in g} q_ih).
// A block owns a contiguous run of query tokens.  Its 512 threads form `slices` token slices x n_cols pair-columns
// of the [Hkv][d/2] pooled grid (a warp reads 128 contiguous bytes of each head); a thread walks its slice's tokens
// eight at a time with all loads of a batch issued before any is used.  Slices are added in slice order through
// shared memory; a second small kernel adds the per-block partials in a fixed order, so the result does not depend
// on scheduling.
// ---------------------------------------------------------------------------------------------------------
constexpr int QPOOL_THREADS = 512;
constexpr int QPOOL_BATCH = 8;

template <typename T, int GROUP /* query heads per KV head; 0 = any */>
__global__ void __launch_bounds__(QPOOL_THREADS) k_qpool(const T *__restrict__ q, const int32_t *__restrict__ q_pos, int n_q,
                                                         int n_q_heads, int group_rt, int d, pc_rope_dev rope,
                                                         float *__restrict__ partial, int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    __shared__ float2 slice_sum[QPOOL_THREADS];
    const int group = GROUP > 0 ? GROUP : group_rt;
    const int half = d / 2, n_kv = n_q_heads / group, n_cols = n_kv * half, row_len = n_kv * d;
    const size_t q_row = (size_t)n_q_heads * d;
    const int per_block = (n_q + gridDim.x - 1) / gridDim.x;
    const int first = blockIdx.x * per_block, end = min(n_q, first + per_block);
    const int slices = max(1, QPOOL_THREADS / n_cols);
    const int sl = threadIdx.x / n_cols;
    for (int col0 = 0; col0 < n_cols; col0 += QPOOL_THREADS) {        // one pass unless n_cols > 1024
        const int col = col0 + (n_cols >= QPOOL_THREADS ? threadIdx.x : threadIdx.x % n_cols);
        const bool active = sl < slices && col < n_cols;
        float acc0 = 0.f, acc1 = 0.f;
        if (active) {
            const int g = col / half, pair = col % half;
            const T *base = q + (size_t)g * group * d + 2 * pair;
            const int axis = pair % 3, amax = rope.max_pos[axis], astride = rope.n_axis[axis];
            const float2 *tab = rope.tab + rope.off[axis] + pair / 3;
            for (int i0 = first + sl; i0 < end; i0 += slices * QPOOL_BATCH) {
                int pa[QPOOL_BATCH];                                   // this pair's own coordinate of each token
                float x0[QPOOL_BATCH], x1[QPOOL_BATCH];
#pragma unroll
                for (int t = 0; t < QPOOL_BATCH; ++t) {
                    const int i = min(i0 + t * slices, end - 1);       // out-of-range slots re-read the last token, unused
                    pa[t] = __ldg(q_pos + 4 * (size_t)i + axis);
                    const T *row = base + (size_t)i * q_row;
                    x0[t] = 0.f; x1[t] = 0.f;
#pragma unroll
                    for (int u = 0; u < (GROUP > 0 ? GROUP : 1); ++u) {
                        for (int uu = u; uu < group; uu += (GROUP > 0 ? group : 1)) {
                            if constexpr (sizeof(T) == 2) {
                                const uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(row + (size_t)uu * d));
                                x0[t] += pc_bf16_lo(w); x1[t] += pc_bf16_hi(w);
                            } else {
                                const float2 w = __ldg(reinterpret_cast<const float2 *>(row + (size_t)uu * d));
                                x0[t] += w.x; x1[t] += w.y;
                            }
                        }
                    }
                }
                float2 cs[QPOOL_BATCH];
#pragma unroll
                for (int t = 0; t < QPOOL_BATCH; ++t) {
                    int p = pa[t];
                    if ((unsigned)p >= (unsigned)amax) {               // outside the table: record, clamp
                        pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_QPOOL_POS);
                        p = p < 0 ? 0 : amax - 1;
                    }
                    cs[t] = __ldg(tab + (size_t)p * astride);
                }
#pragma unroll
                for (int t = 0; t < QPOOL_BATCH; ++t)
                    if (i0 + t * slices < end) {
                        acc0 += x0[t] * cs[t].x - x1[t] * cs[t].y;
                        acc1 += x0[t] * cs[t].y + x1[t] * cs[t].x;
                    }
            }
        }
        slice_sum[threadIdx.x] = make_float2(acc0, acc1);
        __syncthreads();
        if (active && sl == 0) {
            float2 tot = make_float2(0.f, 0.f);
            const int stride = n_cols >= QPOOL_THREADS ? QPOOL_THREADS : n_cols;
            for (int k = 0; k < slices; ++k) { const float2 v = slice_sum[k * stride + threadIdx.x]; tot.x += v.x; tot.y += v.y; }
            *reinterpret_cast<float2 *>(partial + (size_t)blockIdx.x * row_len + 2 * col) = tot;
        }
        __syncthreads();
    }
}

// pooled[e] = (1/n_q) * sum over blocks of partial[b][e].  32 columns per block; 32 threads per column each add every
// 32nd partial (in block order, at most four loads, all in flight together), and the 32 sums are added in slice order.
__global__ void __launch_bounds__(1024) k_qpool_reduce(const float *__restrict__ partial, int n_partials, int row_len, float inv_n,
                                                       float *__restrict__ pooled) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    __shared__ float part[32][33];
    const int c = threadIdx.x & 31, sl = threadIdx.x >> 5, e = blockIdx.x * 32 + c;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (e < row_len) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int b = sl + 32 * i;
            if (b < n_partials) v[i] = __ldcg(partial + (size_t)b * row_len + e);
        }
    }
    part[sl][c] = (v[0] + v[1]) + (v[2] + v[3]);
    __syncthreads();
    if (sl == 0 && e < row_len) {
        float tot = 0.f;
#pragma unroll
        for (int k = 0; k < 32; ++k) tot += part[k][c];
        pooled[e] = tot * inv_n;
    }
}

// ---------------------------------------------------------------------------------------------------------
// Score.  History keys are contiguous, so a tile of 8 tokens is one run of 8 rows (16 KB at 8 KV heads x 128 bf16)
// plus 128 bytes of positions.  A producer warp streams tiles into a four-stage shared-memory ring with bulk
// asynchronous copies tracked by mbarriers; eight consumer warps take one token each.  A token's row over all KV
// heads is CPL x 32 sixteen-byte chunks; lane l reads chunks l, l+32, ...  Because 32 chunks span a multiple of d,
// all of a lane's chunks cover the same PER16/2 rotary pairs (of different heads), so the lane sums the two brackets
// over its chunks and needs PER16/2 table look-ups per token.  Chunks are processed two at a time so that every
// multiply-add is a two-lane fp32 instruction.  Blocks are persistent and take tiles round-robin.
// ---------------------------------------------------------------------------------------------------------
constexpr int SCORE_TOK = 8;                       // tokens per tile = consumer warps
constexpr int SCORE_STAGES = 4;
constexpr int SCORE_THREADS = (SCORE_TOK + 1) * 32;

template <typename T, int CPL /* chunks per lane */>
__global__ void __launch_bounds__(SCORE_THREADS) k_score(const T *__restrict__ k, const int32_t *__restrict__ k_pos,
                                                         const uint8_t *__restrict__ valid, int n_src, int d, float scale,
                                                         pc_rope_dev rope, const float *__restrict__ pooled,
                                                         float *__restrict__ scores, int32_t *status) {
    pc_grid_dep_launch();
    constexpr int PER = Elem<T>::PER16, NP = PER / 2;
    constexpr uint32_t ROW_BYTES = CPL * 32 * 16;
    constexpr uint32_t STAGE_BYTES = SCORE_TOK * ROW_BYTES + SCORE_TOK * 16;
    extern __shared__ __align__(128) uint8_t ring[];
    __shared__ __align__(8) uint64_t bars[2 * SCORE_STAGES];
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring0 = pc_smem_u32(ring), bar0 = pc_smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (SCORE_STAGES + s); };
    if (threadIdx.x == 0) {
        for (int s = 0; s < SCORE_STAGES; ++s) { pc_mbar_init(full(s), 1); pc_mbar_init(empty(s), SCORE_TOK); }
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pc_grid_dep_wait();   // the pooled query comes from the kernel before
    const int n_tiles = (n_src + SCORE_TOK - 1) / SCORE_TOK;

    if (warp == SCORE_TOK) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int it = 0;
            for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
                const int s = it % SCORE_STAGES, use = it / SCORE_STAGES;
                if (use > 0 && !pc_mbar_wait(empty(s), (use - 1) & 1, abort_flag, status, PC_WHERE_SCORE_WAIT)) break;
                const int tok0 = tile * SCORE_TOK, n_tok = min(SCORE_TOK, n_src - tok0);
                const uint32_t dst = ring0 + s * STAGE_BYTES;
                pc_mbar_expect_tx(full(s), n_tok * (ROW_BYTES + 16));
                pc_bulk_g2s(dst, reinterpret_cast<const char *>(k) + (size_t)tok0 * ROW_BYTES, n_tok * ROW_BYTES, full(s));
                pc_bulk_g2s(dst + SCORE_TOK * ROW_BYTES, k_pos + 4 * (size_t)tok0, n_tok * 16, full(s));
            }
            if (*abort_flag) {   // let copies already issued land before the block's shared memory goes away
                const uint64_t t0 = pc_global_ns();
                while (pc_global_ns() - t0 < 2000000ull) {}
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    // this lane's slice of the pooled query stays in registers, chunks paired for the two-lane multiply-adds
    constexpr int CP = CPL / 2;                                     // chunk pairs; an odd CPL leaves one single chunk
    float2 qa[CP > 0 ? CP : 1][NP], qb[CP > 0 ? CP : 1][NP];
    float qa1[NP], qb1[NP];
#pragma unroll
    for (int c = 0; c < CPL; ++c)
#pragma unroll
        for (int u = 0; u < NP; ++u) {
            const float a = pooled[(size_t)(c * 32 + lane) * PER + 2 * u], b = pooled[(size_t)(c * 32 + lane) * PER + 2 * u + 1];
            if (c < 2 * CP) {
                if (c & 1) { qa[c / 2][u].y = a; qb[c / 2][u].y = b; } else { qa[c / 2][u].x = a; qb[c / 2][u].x = b; }
            } else { qa1[u] = a; qb1[u] = b; }
        }
    // table slots of this lane's pairs: entry = tbase + coordinate(axis) * stride
    const int pair0 = ((lane * PER) % d) / 2;
    int tbase[NP], tstride[NP], taxis[NP];
#pragma unroll
    for (int u = 0; u < NP; ++u) {
        const int a = (pair0 + u) % 3;
        taxis[u] = a;
        tbase[u] = rope.off[a] + (pair0 + u) / 3;
        tstride[u] = rope.n_axis[a];
    }
    const unsigned mt = rope.max_pos[0], mh = rope.max_pos[1], mw = rope.max_pos[2];

    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
        const int s = it % SCORE_STAGES, use = it / SCORE_STAGES;
        if (!__all_sync(0xffffffffu, pc_mbar_wait(full(s), use & 1, abort_flag, status, PC_WHERE_SCORE_WAIT))) return;
        const int j = tile * SCORE_TOK + warp;
        if (j < n_src) {
            const uint32_t row = ring0 + s * STAGE_BYTES + warp * ROW_BYTES + lane * 16;
            uint4 raw[CPL];
#pragma unroll
            for (int c = 0; c < CPL; ++c) raw[c] = pc_lds128(row + c * 512);
            const uint4 pw4 = pc_lds128(ring0 + s * STAGE_BYTES + SCORE_TOK * ROW_BYTES + warp * 16);
            int pt = (int)pw4.x, ph = (int)pw4.y, pw = (int)pw4.z;
            if (!((unsigned)pt < mt && (unsigned)ph < mh && (unsigned)pw < mw)) {   // outside the tables: record, clamp
                pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_SCORE_POS);
                pt = min(max(pt, 0), (int)mt - 1); ph = min(max(ph, 0), (int)mh - 1); pw = min(max(pw, 0), (int)mw - 1);
            }
            float2 cs[NP];
#pragma unroll
            for (int u = 0; u < NP; ++u) {
                const int pa = taxis[u] == 0 ? pt : (taxis[u] == 1 ? ph : pw);
                cs[u] = __ldg(rope.tab + tbase[u] + pa * tstride[u]);
            }
            // brackets per pair:  A = sum qa ka + qb kb,  B = sum qb ka - qa kb  (B kept as two sums)
            float2 A2[NP], B2[NP], C2[NP];
            float A1[NP], B1[NP];
#pragma unroll
            for (int u = 0; u < NP; ++u) { A2[u] = B2[u] = C2[u] = make_float2(0.f, 0.f); A1[u] = B1[u] = 0.f; }
#pragma unroll
            for (int c = 0; c < CP; ++c) {
                float k0[PER], k1[PER];
                Elem<T>::unpack(raw[2 * c], k0);
                Elem<T>::unpack(raw[2 * c + 1], k1);
#pragma unroll
                for (int u = 0; u < NP; ++u) {
                    const float2 ka = make_float2(k0[2 * u], k1[2 * u]), kb = make_float2(k0[2 * u + 1], k1[2 * u + 1]);
                    pc_fma2(A2[u], qa[c][u], ka);
                    pc_fma2(A2[u], qb[c][u], kb);
                    pc_fma2(B2[u], qb[c][u], ka);
                    pc_fma2(C2[u], qa[c][u], kb);
                }
            }
            if constexpr (CPL & 1) {
                float k0[PER];
                Elem<T>::unpack(raw[CPL - 1], k0);
#pragma unroll
                for (int u = 0; u < NP; ++u) {
                    A1[u] = fmaf(qa1[u], k0[2 * u], fmaf(qb1[u], k0[2 * u + 1], A1[u]));
                    B1[u] = fmaf(qb1[u], k0[2 * u], fmaf(-qa1[u], k0[2 * u + 1], B1[u]));
                }
            }
            float sum = 0.f;
#pragma unroll
            for (int u = 0; u < NP; ++u) {
                const float A = (A2[u].x + A2[u].y) + A1[u];
                const float B = ((B2[u].x + B2[u].y) - (C2[u].x + C2[u].y)) + B1[u];
                sum = fmaf(cs[u].x, A, fmaf(cs[u].y, B, sum));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0) {
                float r = sum * scale;
                if (valid && !valid[j]) r = -INFINITY;
                scores[j] = r;
            }
        }
        __syncwarp();
        if (lane == 0) pc_mbar_arrive(empty(s));
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
constexpr int SEL_CACHE = 4096;   // keys of a frame kept in shared memory; longer frames re-read the rest from global

// Exclusive block scan of a small per-thread value; total = sum over the block.
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
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    __shared__ uint32_t keys[SEL_CACHE];
    __shared__ int hist[256];
    __shared__ int warp_sums[SEL_THREADS / 32];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_want;
    const int4 fr = tab.f[blockIdx.x];
    const int first = fr.x, n = fr.y, budget = fr.z, out0 = fr.w;
    if (budget <= 0 || n <= 0) return;
    const float *s = scores + first;
    const int lane = threadIdx.x & 31;

    for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
        const float v = s[j];
        if (v != v) pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_SELECT_NAN);
        if (j < SEL_CACHE) keys[j] = score_key(v);
    }
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    auto key_at = [&](int j) { return j < SEL_CACHE ? keys[j] : score_key(s[j]); };

    uint32_t prefix = 0, mask = 0;
    int want = budget;                               // rank, among keys matching the prefix, of the threshold key
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
            const uint32_t key = key_at(j);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane l owns digits 255 - 8l down to 248 - 8l; an inclusive scan over lanes counts keys from the top digit down
            int c[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = hist[255 - 8 * lane - i]; mine += c[i]; }
            int inc = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int v = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += v;
            }
            const int before = inc - mine;
            if (before < want && want <= inc) {      // exactly one lane: the threshold digit is among its eight
                int w = want - before, digit = 255 - 8 * lane;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (c[i] >= w) { digit = 255 - 8 * lane - i; break; }
                    w -= c[i];
                }
                sh_prefix = prefix | ((uint32_t)digit << shift);
                sh_want = w;
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        want = sh_want;
        mask |= 255u << shift;
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
    }
    // prefix is now the threshold key T: every key above it is kept, and the `want` lowest-index keys equal to it.
    // One scan per 512 keys carries both counts (keys above T in the low half, keys equal to T in the high half).
    const uint32_t T = prefix;
    int gt_seen = 0, eq_seen = 0;
    for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
        const int j = j0 + threadIdx.x;
        const bool in = j < n;
        const uint32_t key = in ? key_at(j) : 0u;
        const int is_gt = in && key > T, is_eq = in && key == T;
        int total;
        const int ex = block_exclusive_scan(is_gt | (is_eq << 16), warp_sums, total);
        const int gt_before = gt_seen + (ex & 0xFFFF), eq_before = eq_seen + (ex >> 16);
        if (is_gt || (is_eq && eq_before < want)) {
            const int at = gt_before + min(eq_before, want);
            if (at < budget) sel_idx[out0 + at] = first + j;
        }
        gt_seen += total & 0xFFFF;
        eq_seen += total >> 16;
    }
}

// Enqueue pooling and scoring on caller-given scratch (a context's, or the library's fixed array).
template <typename T>
pc_status enqueue_score(const pc_layer_desc &D, int sm_count, const pc_rope_dev &rope, float *partial, float *pooled,
                        int32_t *status, const void *hist_k, const int32_t *hist_pos, int n_src,
                        const void *q, const int32_t *q_pos, int32_t n_q, const uint8_t *valid, float *scores,
                        cudaStream_t stream, pc_ctx *marks) {
    const int row = D.n_kv_heads * D.head_dim;
    const int group = D.n_q_heads / D.n_kv_heads;
    const int pool_blocks = std::min<int>(PC_QPOOL_BLOCKS, (n_q + QPOOL_BATCH - 1) / QPOOL_BATCH);
    if (marks) pc_mark(marks, PC_MARK_SCORE0, stream);
#define PC_QPOOL_ARGS static_cast<const T *>(q), q_pos, n_q, D.n_q_heads, group, D.head_dim, rope, partial, status
    switch (group) {
    case 1: PC_LAUNCH((k_qpool<T, 1>), dim3(pool_blocks), dim3(QPOOL_THREADS), 0, stream, PC_QPOOL_ARGS); break;
    case 2: PC_LAUNCH((k_qpool<T, 2>), dim3(pool_blocks), dim3(QPOOL_THREADS), 0, stream, PC_QPOOL_ARGS); break;
    case 3: PC_LAUNCH((k_qpool<T, 3>), dim3(pool_blocks), dim3(QPOOL_THREADS), 0, stream, PC_QPOOL_ARGS); break;
    case 4: PC_LAUNCH((k_qpool<T, 4>), dim3(pool_blocks), dim3(QPOOL_THREADS), 0, stream, PC_QPOOL_ARGS); break;
    default: PC_LAUNCH((k_qpool<T, 0>), dim3(pool_blocks), dim3(QPOOL_THREADS), 0, stream, PC_QPOOL_ARGS); break;
    }
#undef PC_QPOOL_ARGS
    PC_CUDA_TRY(cudaGetLastError());
    PC_LAUNCH(k_qpool_reduce, dim3((row + 31) / 32), dim3(1024), 0, stream, partial, pool_blocks, row, 1.f / (float)n_q, pooled);
    PC_CUDA_TRY(cudaGetLastError());
    if (marks) pc_mark(marks, PC_MARK_QPOOL, stream);
    const float scale = (float)(1.0 / ((double)D.n_q_heads * std::sqrt((double)D.head_dim)));
    const int chunks = row / Elem<T>::PER16;          // 16-byte chunks per token row
    if (chunks % 32) return PC_ERR_UNSUPPORTED;
    const int n_tiles = (n_src + SCORE_TOK - 1) / SCORE_TOK;
    const T *k = static_cast<const T *>(hist_k);
#define PC_SCORE_CASE(CPL)                                                                                          \
    case CPL: {                                                                                                     \
        const int smem = SCORE_STAGES * (SCORE_TOK * CPL * 512 + SCORE_TOK * 16);                                   \
        /* resident blocks per SM of this instance (the grid is persistent), looked up once per device */          \
        static int per_sm_of[PC_MAX_DEVICES] = {};                                                                  \
        int dev_id = 0;                                                                                             \
        PC_CUDA_TRY(cudaGetDevice(&dev_id));                                                                        \
        if (dev_id < 0 || dev_id >= PC_MAX_DEVICES) return PC_ERR_UNSUPPORTED;                                      \
        if (per_sm_of[dev_id] == 0) {                                                                               \
            PC_CUDA_TRY(cudaFuncSetAttribute(k_score<T, CPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));  \
            int occ = 0;                                                                                            \
            PC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_score<T, CPL>, SCORE_THREADS, smem)); \
            per_sm_of[dev_id] = std::max(1, occ);                                                                   \
        }                                                                                                           \
        const int blocks = std::max(1, std::min(n_tiles, sm_count * per_sm_of[dev_id]));                            \
        PC_LAUNCH((k_score<T, CPL>), dim3(blocks), dim3(SCORE_THREADS), smem, stream, k, hist_pos, valid, n_src, D.head_dim, scale, rope, \
                                                                 pooled, scores, status);                          \
    } break;
    switch (chunks / 32) {
        PC_SCORE_CASE(1) PC_SCORE_CASE(2) PC_SCORE_CASE(3) PC_SCORE_CASE(4) PC_SCORE_CASE(6) PC_SCORE_CASE(8)
    default: return PC_ERR_UNSUPPORTED;
    }
#undef PC_SCORE_CASE
    PC_CUDA_TRY(cudaGetLastError());
    if (marks) pc_mark(marks, PC_MARK_SCORE, stream);
    return PC_OK;
}

template <typename T>
pc_status launch_score(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q,
                       const uint8_t *valid, float *scores, cudaStream_t stream) {
    return enqueue_score<T>(ctx->desc, ctx->sm_count, ctx->rope, ctx->qpool_partial, ctx->qpool, ctx->status,
                            src->history.k, src->history.pos, src->history.n_tokens, q, q_pos, n_q, valid, scores, stream,
                            ctx);
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
    } else if (reinterpret_cast<uintptr_t>(scores_override) & 3) {      // read element by element: any float address will do
        return PC_ERR_INVALID_ARG;
    }
    if (n_frames > 0 && out > 0) {
        if (scores_override) pc_mark(ctx, PC_MARK_SCORE, stream);
        PC_LAUNCH(k_select, dim3(n_frames), dim3(SEL_THREADS), 0, stream, select_on, tab, sel_idx, ctx->status);
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
// table, the pooled query and its per-block partials — lives in one file-scope device array
// of fixed size that every GPU loading this library carries until the process exits.
//
// In host code the array's name is only a handle; the device address is obtained once per device with
// cudaGetSymbolAddress while that device is current, and that pointer (never the symbol) is what kernels receive.
// ---------------------------------------------------------------------------------------------------------
namespace {

constexpr int STATIC_MAX_ROW = 1024;          // n_kv_heads * head_dim
constexpr int STATIC_MAX_ROPE = 32768;        // rotary table entries: sum over axes of max_pos * pairs on that axis
constexpr int STATIC_MAX_DEVICES = PC_MAX_DEVICES;

constexpr size_t STATIC_OFF_POOLED = 256;  /* first 256 bytes unused */                                                  // float [STATIC_MAX_ROW]
constexpr size_t STATIC_OFF_PARTIAL = STATIC_OFF_POOLED + STATIC_MAX_ROW * sizeof(float);  // float [PC_QPOOL_BLOCKS][STATIC_MAX_ROW]
constexpr size_t STATIC_OFF_ROPE = STATIC_OFF_PARTIAL + (size_t)PC_QPOOL_BLOCKS * STATIC_MAX_ROW * sizeof(float);
constexpr size_t STATIC_BYTES = STATIC_OFF_ROPE + (size_t)STATIC_MAX_ROPE * sizeof(float2);   // 790,784 bytes

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

// Rotary table in fp64, stored as fp32 (cos, sin): entry (axis a, position p, column m) = p * base^(-m / n_axis[a]).
__global__ void __launch_bounds__(256) k_rope_table(float2 *__restrict__ tab, pc_rope_dev rope, double base, int total) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
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
    // the array keeps whatever the last call left; the table, the partials and the pooled query are all rewritten before
    // they are read, and nothing has to start at zero
    PC_LAUNCH(k_rope_table, dim3((total + 255) / 256), dim3(256), 0, stream, tab, rope, D.rope_base, total);
    PC_CUDA_TRY(cudaGetLastError());

    int sm_count = 0, dev = 0;
    PC_CUDA_TRY(cudaGetDevice(&dev));
    PC_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    return enqueue_score<T>(D, sm_count, rope, partial, pooled, status, hist_k, hist_pos, n_src, q, q_pos, n_q,
                            valid, scores, stream, nullptr);
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
