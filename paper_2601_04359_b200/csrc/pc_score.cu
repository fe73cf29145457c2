// Token scoring and per-frame top-k selection (the "attention-relevant" retention of Sec. 3.4).
//
//   k_qprep  : one pass over Q: pooled query  q~[g][c] = sum_{h in group g} (1/n_q) sum_i (R(p_i) q_ih)[c]  (fixed-point
//              sums, deterministic) and, on request, the rotated bf16 queries the attention kernel reads
//   k_score  : s_j = 1/(Hq sqrt(d)) * sum_g q~_g . R(p_j) k_jg   — one pass over the history keys, HBM-bound
//   k_select : per frame the budget[f] best scores (ties to the lower index), ascending indices out
//
// The score of a key equals the mean scaled logit over all queries and heads because the logit is linear in the
// rotated query.  For one rotary pair (a, b) = elements (2i, 2i+1):
//   q_a (k_a cos - k_b sin) + q_b (k_a sin + k_b cos) = cos (q_a k_a + q_b k_b) + sin (q_b k_a - q_a k_b),
// and the angle is the same for every KV head, so the two brackets are summed over heads first and each pair costs
// one table look-up per token.
#include <algorithm>

#include "pc_common.cuh"
#include "pc_select.cuh"

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
// Query pass.  One read of Q serves both consumers of the rotated queries: the pooled query of the scoring pass
//   q~[g] = (1/n_q) sum_i sum_{h in g} R(p_i) q_ih
// and, for the tensor-core attention kernel, the rotated bf16 queries with log2(e)/sqrt(d) folded in (q_rot).
// A few warps share one query token: lane l of a warp reads the 16-byte chunks l, l + 32, ... of the warp's part of the
// row (all in flight at once); 32 chunks span a multiple of d, so all of a lane's chunks hold the same rotary pairs and
// the lane needs PER/2 table entries.  The rotated row also goes to a per-token slab in shared memory; after a block
// barrier the threads add, in a fixed order, the slabs' entries of each pooled element (tokens, then heads), turn the sum
// into a 64-bit fixed-point number (units of 2^-32) and add it to the global accumulator with an integer atomic:
// integer addition is associative, so the pooled query does not depend on the order in which blocks arrive.
// ---------------------------------------------------------------------------------------------------------
constexpr int QPREP_WARPS = 8;                      // warps per block when the parts of a token divide it
constexpr float FX_ONE = 4294967296.0f;             // 2^32
constexpr int FX_REPLICAS = PC_FX_REPLICAS;         // copies of the accumulator the blocks of the query pass spread over

template <typename T> __device__ __forceinline__ uint4 pack_row(const float *f);
template <> __device__ __forceinline__ uint4 pack_row<float>(const float *f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
template <> __device__ __forceinline__ uint4 pack_row<__nv_bfloat16>(const float *f) {
    return make_uint4(pc_pack_bf16(f[0], f[1]), pc_pack_bf16(f[2], f[3]), pc_pack_bf16(f[4], f[5]), pc_pack_bf16(f[6], f[7]));
}

// A query row is cut into `parts` runs of CPW x 32 chunks, one warp each (short instruction streams on many warps: the
// kernel is bound by latency, not by bytes); a block holds `tokens_per_block` tokens.
template <typename T, int CPW /* chunks per lane of one warp's part of a query row */>
__global__ void __launch_bounds__(1024) k_qprep(const T *__restrict__ q, const int32_t *__restrict__ q_pos, int n_q,
                                                int n_q_heads, int group, int d, int parts, pc_rope_dev rope,
                                                float out_scale, T *__restrict__ q_rot,
                                                unsigned long long *fx, double fx_scale, float *__restrict__ pooled,
                                                int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    constexpr int PER = Elem<T>::PER16, NP = PER / 2;
    extern __shared__ __align__(16) float slab[];                     // [tokens_per_block][Hq*d]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tokens_per_block = (blockDim.x >> 5) / parts;
    const int row_len = n_q_heads * d;
    const int tok = warp / parts, part = warp - tok * parts;
    const int i = blockIdx.x * tokens_per_block + tok;
    if (i < n_q) {
        const int4 pp = __ldg(reinterpret_cast<const int4 *>(q_pos) + i);
        const size_t at = (size_t)i * (row_len / PER) + (size_t)part * CPW * 32 + lane;     // in 16-byte chunks
        const uint4 *src = reinterpret_cast<const uint4 *>(q) + at;
        uint4 raw[CPW];
#pragma unroll
        for (int c = 0; c < CPW; ++c) raw[c] = pc_ldg_stream(src + c * 32);
        const int pair0 = ((lane * PER) % d) / 2;
        float2 cs[NP];
#pragma unroll
        for (int u = 0; u < NP; ++u) cs[u] = pc_rope_cs(rope, pair0 + u, pp.x, pp.y, pp.z, status, PC_WHERE_QPOOL_POS);
        float *mine = slab + (size_t)tok * row_len + ((size_t)part * CPW * 32 + lane) * PER;
        uint4 *dst = q_rot ? reinterpret_cast<uint4 *>(q_rot) + at : nullptr;
#pragma unroll
        for (int c = 0; c < CPW; ++c) {
            float x[PER], r[PER];
            Elem<T>::unpack(raw[c], x);
#pragma unroll
            for (int u = 0; u < NP; ++u) {
                const float2 y = pc_rotate(x[2 * u], x[2 * u + 1], cs[u]);
                r[2 * u] = y.x;
                r[2 * u + 1] = y.y;
            }
            float4 *s4 = reinterpret_cast<float4 *>(mine + (size_t)c * 32 * PER);
#pragma unroll
            for (int k = 0; k < PER / 4; ++k) s4[k] = make_float4(r[4 * k], r[4 * k + 1], r[4 * k + 2], r[4 * k + 3]);
            if (dst) {                                                  // the attention kernel's queries carry its scale
#pragma unroll
                for (int k = 0; k < PER; ++k) r[k] = __fmul_rn(r[k], out_scale);
                dst[c * 32] = pack_row<T>(r);
            }
        }
    }
    __syncthreads();
    const int n_tokens_used = min(tokens_per_block, n_q - blockIdx.x * tokens_per_block);
    const int n_out = (n_q_heads / group) * d;
    // blocks spread over FX_REPLICAS copies of the accumulator: fewer atomics queue up on each cache line
    unsigned long long *mine_fx = fx + (size_t)(blockIdx.x % FX_REPLICAS) * n_out;
    // four pooled elements per thread at a time, so that four independent sums are in flight; the order of the additions
    // of each sum is fixed (tokens ascending, heads of the group ascending)
    for (int e0 = threadIdx.x; e0 < n_out; e0 += 4 * blockDim.x) {
        const float *s[4];
        float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int e = min(e0 + k * (int)blockDim.x, n_out - 1), g = e / d, x = e - g * d;
            s[k] = slab + (size_t)g * group * d + x;
        }
        for (int w = 0; w < n_tokens_used; ++w)
            for (int h = 0; h < group; ++h) {
                const int off = w * row_len + h * d;
#pragma unroll
                for (int k = 0; k < 4; ++k) sum[k] += s[k][off];
            }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int e = e0 + k * (int)blockDim.x;
            if (e < n_out) atomicAdd(mine_fx + e, (unsigned long long)__float2ll_rn(sum[k] * FX_ONE));
        }
    }
    // The block that finishes last (a ticket in the word after the last copy; nobody waits for anybody) adds the copies,
    // writes the pooled query as fp32 and clears the accumulator and the ticket for the next call.  Nothing of this lives
    // on the host, so a captured graph replays it unchanged.
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0)
        is_last = atomicAdd(fx + (size_t)FX_REPLICAS * n_out, 1ull) == (unsigned long long)(gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int e = threadIdx.x; e < n_out; e += blockDim.x) {
        long long w = 0;
#pragma unroll
        for (int rep = 0; rep < FX_REPLICAS; ++rep) {                     // integer sums: any order gives the same bits
            w += (long long)__ldcg(fx + (size_t)rep * n_out + e);
            fx[(size_t)rep * n_out + e] = 0;
        }
        pooled[e] = (float)((double)w * fx_scale);
    }
    if (threadIdx.x == 0) fx[(size_t)FX_REPLICAS * n_out] = 0;
}

// ---------------------------------------------------------------------------------------------------------
// Score.  One warp takes two history tokens at a time: lane l loads the 16-byte chunks l, l + 32, ... of both rows
// (streaming loads, all in flight before the first is used: 2 x CPL x 512 bytes per warp) and both position records.
// 32 chunks span a multiple of d, so all of a lane's chunks cover the same PER/2 rotary pairs (of different heads): the
// lane sums the two brackets over its chunks and needs PER/2 table look-ups per token.  For a pair (a, b) the two
// brackets are two-lane products of the pair as it comes out of the unpacking, (k_a, k_b), with (q_a, q_b) and with
// (q_b, -q_a): two two-lane fp32 multiply-adds per pair, no register shuffling.  The pooled query sits in shared
// memory in that form; one 16-byte read serves both rows.
// Blocks are persistent; warps take token pairs round-robin, so the tokens in flight at any time form one contiguous
// window of the history.
// ---------------------------------------------------------------------------------------------------------
constexpr int SCORE_WARPS = 8;
constexpr int SCORE_THREADS = SCORE_WARPS * 32;

template <typename T, int CPL /* chunks per lane */>
__global__ void __launch_bounds__(SCORE_THREADS, 2) k_score(const T *__restrict__ k, const int32_t *__restrict__ k_pos,
                                                            const uint8_t *__restrict__ valid, int n_src, int d, float scale,
                                                            pc_rope_dev rope, const float *__restrict__ pooled,
                                                            float *__restrict__ scores, int32_t *status) {
    pc_grid_dep_launch();
    constexpr int PER = Elem<T>::PER16, NP = PER / 2;
    __shared__ float4 qs[CPL * NP * 32];                              // (q_a, q_b, q_b, -q_a) of (chunk, pair, lane)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gw = blockIdx.x * SCORE_WARPS + warp, n_warps = gridDim.x * SCORE_WARPS;
    const int n_pairs = (n_src + 1) >> 1;
    const uint4 *krow = reinterpret_cast<const uint4 *>(k) + lane;
    pc_grid_dep_wait();   // the pooled query comes from the kernel before

    // this warp's first two rows are requested before the pooled query is staged: both latencies overlap
    int tp = gw;
    uint4 raw0[CPL], raw1[CPL];
    int4 p0 = make_int4(0, 0, 0, 0), p1 = p0;
    auto request = [&](int pair_idx) {
        const int j0 = 2 * pair_idx, j1 = min(j0 + 1, n_src - 1);
        p0 = __ldg(reinterpret_cast<const int4 *>(k_pos) + j0);
        p1 = __ldg(reinterpret_cast<const int4 *>(k_pos) + j1);
#pragma unroll
        for (int c = 0; c < CPL; ++c) raw0[c] = pc_ldg_stream(krow + (size_t)j0 * (CPL * 32) + c * 32);
#pragma unroll
        for (int c = 0; c < CPL; ++c) raw1[c] = pc_ldg_stream(krow + (size_t)j1 * (CPL * 32) + c * 32);
    };
    if (tp < n_pairs) request(tp);

    for (int idx = threadIdx.x; idx < CPL * NP * 32; idx += SCORE_THREADS) {
        const int l = idx & 31, u = (idx >> 5) % NP, c = idx / (32 * NP);
        const float2 w = __ldcg(reinterpret_cast<const float2 *>(pooled + (size_t)(c * 32 + l) * PER + 2 * u));
        qs[idx] = make_float4(w.x, w.y, w.y, -w.x);
    }
    __syncthreads();

    // table slots of this lane's pairs: entry = tbase + coordinate(axis) * stride
    const int pair0 = ((lane * PER) % d) / 2;
    int tbase[NP], tstride[NP], taxis[NP];
#pragma unroll
    for (int u = 0; u < NP; ++u) {
        const int a = (pair0 + u) % 3;
        taxis[u] = a;
        tbase[u] = (a == 0 ? rope.off[0] : (a == 1 ? rope.off[1] : rope.off[2])) + (pair0 + u) / 3;
        tstride[u] = a == 0 ? rope.n_axis[0] : (a == 1 ? rope.n_axis[1] : rope.n_axis[2]);
    }
    const unsigned mt = rope.max_pos[0], mh = rope.max_pos[1], mw = rope.max_pos[2];
    const float4 *ql = qs + lane;

    auto table = [&](int4 p, float2 (&cs)[NP]) {
        int pt = p.x, ph = p.y, pw = p.z;
        if (!((unsigned)pt < mt && (unsigned)ph < mh && (unsigned)pw < mw)) {   // outside the tables: record, clamp
            pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_SCORE_POS);
            pt = min(max(pt, 0), (int)mt - 1); ph = min(max(ph, 0), (int)mh - 1); pw = min(max(pw, 0), (int)mw - 1);
        }
#pragma unroll
        for (int u = 0; u < NP; ++u) {
            const int pa = taxis[u] == 0 ? pt : (taxis[u] == 1 ? ph : pw);
            cs[u] = __ldg(rope.tab + tbase[u] + pa * tstride[u]);
        }
    };

    for (; tp < n_pairs; tp += n_warps) {
        float2 cs0[NP], cs1[NP];
        table(p0, cs0);
        table(p1, cs1);
        // brackets per pair:  A = sum q_a k_a + q_b k_b,  B = sum q_b k_a - q_a k_b, each as the two lanes of one register pair
        float2 A0[NP], B0[NP], A1[NP], B1[NP];
#pragma unroll
        for (int u = 0; u < NP; ++u) A0[u] = B0[u] = A1[u] = B1[u] = make_float2(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < CPL; ++c) {
            float k0[PER], k1[PER];
            Elem<T>::unpack(raw0[c], k0);
            Elem<T>::unpack(raw1[c], k1);
#pragma unroll
            for (int u = 0; u < NP; ++u) {
                const float4 qq = ql[(c * NP + u) * 32];
                const float2 qab = make_float2(qq.x, qq.y), qba = make_float2(qq.z, qq.w);
                const float2 x0 = make_float2(k0[2 * u], k0[2 * u + 1]), x1 = make_float2(k1[2 * u], k1[2 * u + 1]);
                A0[u] = __ffma2_rn(qab, x0, A0[u]);
                B0[u] = __ffma2_rn(qba, x0, B0[u]);
                A1[u] = __ffma2_rn(qab, x1, A1[u]);
                B1[u] = __ffma2_rn(qba, x1, B1[u]);
            }
        }
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int u = 0; u < NP; ++u) {
            s0 = fmaf(cs0[u].x, A0[u].x + A0[u].y, fmaf(cs0[u].y, B0[u].x + B0[u].y, s0));
            s1 = fmaf(cs1[u].x, A1[u].x + A1[u].y, fmaf(cs1[u].y, B1[u].x + B1[u].y, s1));
        }
        const int j0 = 2 * tp;
        if (tp + n_warps < n_pairs) request(tp + n_warps);           // the next two rows travel while these are reduced
        // both sums with six shuffles: after the first exchange the lower half-warp carries token 0, the upper token 1
        s0 += __shfl_xor_sync(0xffffffffu, s0, 16);
        s1 += __shfl_xor_sync(0xffffffffu, s1, 16);
        float s = lane < 16 ? s0 : s1;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if ((lane & 15) == 0) {
            const int j = j0 + (lane >> 4);
            if (j < n_src) {
                float r = s * scale;
                if (valid && !valid[j]) r = -INFINITY;
                scores[j] = r;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// Select.  One block per frame runs the block-level selection of pc_select.cuh and writes the kept tokens' indices in
// ascending order.
// ---------------------------------------------------------------------------------------------------------
constexpr int SEL_THREADS = 1024;

__global__ void __launch_bounds__(SEL_THREADS) k_select(const float *__restrict__ scores, const __grid_constant__ FrameTab tab,
                                                       int32_t *__restrict__ sel_idx, int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    __shared__ SelectShared<SEL_THREADS> sm;
    const int4 fr = tab.f[blockIdx.x];
    if (fr.z <= 0 || fr.y <= 0) return;
    const int out0 = fr.w;
    frame_select<SEL_THREADS>(scores, fr, sm, status, [&](int at, int idx) { sel_idx[out0 + at] = idx; });
}

// Enqueue the query pass and the scoring kernel on caller-given scratch (a context's, or the library's fixed array).
// fx: the fixed-point accumulator (PC_FX_REPLICAS copies of Hkv*d sums and one ticket word), all zero on entry and zero
// again when the query pass has run; pooled: Hkv*d floats, written by the query pass and read by the scoring kernel;
// q_rot / q_scale: where the rotated queries go as well and the factor folded into them.
template <typename T>
pc_status enqueue_score(const pc_layer_desc &D, int sm_count, const pc_rope_dev &rope, long long *fx, float *pooled,
                        int32_t *status, const void *hist_k, const int32_t *hist_pos, int n_src, const void *q,
                        const int32_t *q_pos, int32_t n_q, const uint8_t *valid, float *scores, void *q_rot, float q_scale,
                        cudaStream_t stream, pc_ctx *marks) {
    constexpr int PER = Elem<T>::PER16;
    const int row = D.n_kv_heads * D.head_dim;
    const int group = D.n_q_heads / D.n_kv_heads;
    const int q_row = D.n_q_heads * D.head_dim;
    const int q_chunks = q_row / PER, chunks = row / PER;            // 16-byte chunks per query row / key row
    if (chunks % 32 || q_chunks % 32 || (32 * PER) % D.head_dim) return PC_ERR_UNSUPPORTED;
    const double fx_scale = 1.0 / (4294967296.0 * (double)n_q);
    // a row's chunk rows are dealt to `parts` warps of 1-4 chunk rows each
    const int qcpl = q_chunks / 32;
    const int cpw = qcpl % 3 == 0 ? 3 : (qcpl % 4 == 0 ? 4 : (qcpl % 2 == 0 ? 2 : 1));
    const int parts = qcpl / cpw;
    if (parts > 32) return PC_ERR_UNSUPPORTED;
    int tokens_per_block = std::max(1, QPREP_WARPS / parts);
    tokens_per_block = std::max(1, std::min<int>(tokens_per_block, (int)((200u * 1024u) / ((size_t)q_row * sizeof(float)))));
    const int q_smem = tokens_per_block * q_row * (int)sizeof(float);
    const int q_blocks = (n_q + tokens_per_block - 1) / tokens_per_block;
    int dev_id = 0;
    PC_CUDA_TRY(cudaGetDevice(&dev_id));
    if (dev_id < 0 || dev_id >= PC_MAX_DEVICES) return PC_ERR_UNSUPPORTED;
    if (marks) pc_mark(marks, PC_MARK_SCORE0, stream);
#define PC_QPREP_CASE(CPW)                                                                                           \
    {                                                                                                               \
        static int smem_of[PC_MAX_DEVICES] = {};                      /* largest dynamic size allowed so far */      \
        if (q_smem + 1024 > 48 * 1024 && smem_of[dev_id] < q_smem) {   /* the block's static words count, too */    \
            PC_CUDA_TRY(cudaFuncSetAttribute(k_qprep<T, CPW>, cudaFuncAttributeMaxDynamicSharedMemorySize, q_smem)); \
            smem_of[dev_id] = q_smem;                                                                               \
        }                                                                                                           \
        PC_LAUNCH((k_qprep<T, CPW>), dim3(q_blocks), dim3(tokens_per_block * parts * 32), q_smem, stream,           \
                  static_cast<const T *>(q), q_pos, n_q, D.n_q_heads, group, D.head_dim, parts, rope, q_scale,      \
                  static_cast<T *>(q_rot), reinterpret_cast<unsigned long long *>(fx), fx_scale, pooled, status);   \
    }
    switch (cpw) {
    case 3: PC_QPREP_CASE(3) break;        // 24 query heads x 128 bf16: four warps per token
    case 4: PC_QPREP_CASE(4) break;
    case 2: PC_QPREP_CASE(2) break;
    default: PC_QPREP_CASE(1) break;
    }
#undef PC_QPREP_CASE
    PC_CUDA_TRY(cudaGetLastError());
    if (marks) pc_mark(marks, PC_MARK_QPOOL, stream);
    const float scale = (float)(1.0 / ((double)D.n_q_heads * std::sqrt((double)D.head_dim)));
    const int n_pairs = (n_src + 1) / 2;
    const T *k = static_cast<const T *>(hist_k);
#define PC_SCORE_CASE(CPL)                                                                                          \
    case CPL: {                                                                                                     \
        /* resident blocks per SM of this instance (the grid is persistent), looked up once per device */          \
        static int per_sm_of[PC_MAX_DEVICES] = {};                                                                  \
        if (per_sm_of[dev_id] == 0) {                                                                               \
            int occ = 0;                                                                                            \
            PC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_score<T, CPL>, SCORE_THREADS, 0));    \
            per_sm_of[dev_id] = std::max(1, occ);                                                                   \
        }                                                                                                           \
        const int blocks = std::max(1, std::min((n_pairs + SCORE_WARPS - 1) / SCORE_WARPS, sm_count * per_sm_of[dev_id])); \
        PC_LAUNCH((k_score<T, CPL>), dim3(blocks), dim3(SCORE_THREADS), 0, stream, k, hist_pos, valid, n_src, D.head_dim, scale, rope, \
                  pooled, scores, status);                                                                          \
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

}  // namespace

// The shapes the query pass and the scoring kernel are built for: a key row of 512, 1024, 1536, 2048, 3072 or 4096 bytes
// over all KV heads, a query row that is a multiple of 512 bytes and splits into at most 32 warps' parts.
bool pc_score_supports(const pc_layer_desc &D) {
    const int elem = D.dtype == PC_BF16 ? 2 : 4, per = 16 / elem;
    const int row = D.n_kv_heads * D.head_dim, q_row = D.n_q_heads * D.head_dim;
    if (row % (32 * per) || q_row % (32 * per) || (32 * per) % D.head_dim) return false;
    const int cpl = row / per / 32, qcpl = q_row / per / 32;
    if (cpl != 1 && cpl != 2 && cpl != 3 && cpl != 4 && cpl != 6 && cpl != 8) return false;
    const int cpw = qcpl % 3 == 0 ? 3 : (qcpl % 4 == 0 ? 4 : (qcpl % 2 == 0 ? 2 : 1));
    return qcpl / cpw <= 32;
}

pc_status pc_score_impl(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q, const int32_t *budget,
                        const uint8_t *valid, const float *scores_override, float *scores, int32_t *sel_idx, void *q_rot_out,
                        cudaStream_t stream) {
    if (!ctx || !src || !budget) return PC_ERR_INVALID_ARG;
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
            if (!pc_score_supports(ctx->desc)) return PC_ERR_UNSUPPORTED;      // before anything is enqueued
            const size_t row = (size_t)ctx->desc.n_kv_heads * ctx->desc.head_dim;
            if (ctx->qpool_dirty) {          // an earlier call stopped between the query pass and the scoring kernel
                PC_CUDA_TRY(cudaMemsetAsync(ctx->qpool_fx, 0, (PC_FX_REPLICAS * row + 1) * sizeof(long long), stream));
                ctx->qpool_dirty = 0;
            }
            ctx->qpool_dirty = 1;
            const float q_scale = pc_q_rot_scale(ctx->desc.head_dim);
            st = ctx->desc.dtype == PC_BF16
                     ? enqueue_score<__nv_bfloat16>(ctx->desc, ctx->sm_count, ctx->rope, ctx->qpool_fx, ctx->qpool, ctx->status, src->history.k,
                                                    src->history.pos, n_src, q, q_pos, n_q, valid, scores, q_rot_out, q_scale, stream, ctx)
                     : enqueue_score<float>(ctx->desc, ctx->sm_count, ctx->rope, ctx->qpool_fx, ctx->qpool, ctx->status, src->history.k,
                                            src->history.pos, n_src, q, q_pos, n_q, valid, scores, nullptr, 1.0f, stream, ctx);
            if (st != PC_OK) return st;
            ctx->qpool_dirty = 0;
            if (q_rot_out) ctx->q_rot_n = n_q;
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

extern "C" pc_status pc_score(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q,
                              const int32_t *budget, const uint8_t *valid, const float *scores_override, float *scores,
                              int32_t *sel_idx, void *stream_) {
    return pc_score_impl(ctx, src, q, q_pos, n_q, budget, valid, scores_override, scores, sel_idx, nullptr,
                         static_cast<cudaStream_t>(stream_));
}

// ---------------------------------------------------------------------------------------------------------
// Scoring without a context and without any allocation.
//
// Meant for hosts that cannot call cudaMalloc at the point where they need scores: a process whose device memory
// was handed to its own arena at start-up and whose policy forbids driver allocations afterwards, or a
// latency-critical thread that cannot take the device-wide synchronisation a cudaMalloc / cudaFree implies.  Such
// callers cannot create a pc_ctx (pc_create allocates), so everything a context would hold for scoring — the rotary
// table, the fixed-point accumulator of the pooled query and the pooled query itself — lives in one file-scope device array of fixed size
// that every GPU loading this library carries until the process exits.
//
// In host code the array's name is only a handle; the device address is obtained once per device with
// cudaGetSymbolAddress while that device is current, and that pointer (never the symbol) is what kernels receive.
// ---------------------------------------------------------------------------------------------------------
namespace {

constexpr int STATIC_MAX_ROW = 1024;          // n_kv_heads * head_dim
constexpr int STATIC_MAX_ROPE = 32768;        // rotary table entries: sum over axes of max_pos * pairs on that axis
constexpr int STATIC_MAX_QROW = 12288;        // n_q_heads * head_dim: one row of the query pass's shared-memory slab
constexpr int STATIC_MAX_DEVICES = PC_MAX_DEVICES;

constexpr size_t STATIC_OFF_FX = 256;  /* first 256 bytes unused */       // long long [PC_FX_REPLICAS * STATIC_MAX_ROW + 1 counter word]
constexpr size_t STATIC_OFF_POOLED = STATIC_OFF_FX + (size_t)PC_FX_REPLICAS * STATIC_MAX_ROW * sizeof(long long) + 256;   // float [STATIC_MAX_ROW]
constexpr size_t STATIC_OFF_ROPE = STATIC_OFF_POOLED + STATIC_MAX_ROW * sizeof(float);          // float2 [STATIC_MAX_ROPE]
constexpr size_t STATIC_BYTES = STATIC_OFF_ROPE + (size_t)STATIC_MAX_ROPE * sizeof(float2);    // 332,288 bytes

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_BYTES];

// Rotary table in fp64, stored as fp32 (cos, sin): entry (axis a, position p, column m) = p * base^(-m / n_axis[a]).
// The first `clear` 64-bit words of `fx` are set to zero as well (the accumulator of the pooled query).
__global__ void __launch_bounds__(256) k_rope_table(float2 *__restrict__ tab, pc_rope_dev rope, double base, int total,
                                                    long long *__restrict__ fx, int clear) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < clear) fx[e] = 0;
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
    long long *fx = reinterpret_cast<long long *>(base + STATIC_OFF_FX);
    float *pooled = reinterpret_cast<float *>(base + STATIC_OFF_POOLED);
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
    // the array keeps whatever the last call left: the table is rewritten before it is read, and the accumulator of the
    // pooled query, which must start at zero, is cleared by the same kernel
    const int row = D.n_kv_heads * D.head_dim;
    const int fx_words = PC_FX_REPLICAS * row + 1;
    PC_LAUNCH(k_rope_table, dim3((std::max(total, fx_words) + 255) / 256), dim3(256), 0, stream, tab, rope, D.rope_base, total, fx,
              fx_words);
    PC_CUDA_TRY(cudaGetLastError());

    int sm_count = 0, dev = 0;
    PC_CUDA_TRY(cudaGetDevice(&dev));
    PC_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    return enqueue_score<T>(D, sm_count, rope, fx, pooled, status, hist_k, hist_pos, n_src, q, q_pos, n_q, valid, scores, nullptr,
                            1.0f, stream, nullptr);
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
    const int per = D.dtype == PC_BF16 ? 8 : 4;
    if ((row / per) % 32 || (D.n_q_heads * D.head_dim / per) % 32) return PC_ERR_UNSUPPORTED;
    int64_t rope_entries = 0;
    for (int a = 0; a < 3; ++a) {
        if (D.max_pos[a] <= 0 || D.max_pos[a] > (1 << 20)) return PC_ERR_INVALID_ARG;
        rope_entries += (int64_t)D.max_pos[a] * ((D.head_dim / 2 - a + 2) / 3);
    }
    if (row > STATIC_MAX_ROW || rope_entries > STATIC_MAX_ROPE || D.n_q_heads * D.head_dim > STATIC_MAX_QROW) {
        fprintf(stderr,
                "packcache: pc_score_tokens_static: shape exceeds the fixed scratch (n_kv_heads*head_dim %d > %d, or "
                "rotary table %lld > %d entries, or n_q_heads*head_dim > %d)\n",
                row, STATIC_MAX_ROW, (long long)rope_entries, STATIC_MAX_ROPE, STATIC_MAX_QROW);
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
