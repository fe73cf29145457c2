// CUDA-core attention of the current frame's queries over anchors ++ history ++ current (Eq. 2, all keys visible).
// This is the fp32 path (tensor cores would not keep fp32 inputs within 1e-4) and a slow second opinion for bf16.
//
// Block = 128 threads = 32 query rows of one query head, four threads per row; each of the four owns a quarter of
// the head dimension (interleaved in 4-element groups so that shared-memory reads of a key row hit distinct banks).
// Keys are streamed in tiles of 32: K is rotated with the 3D rotary tables while it is copied into shared memory,
// V is copied as it is; the softmax is the usual running (max, sum) form in fp32, in the base-2 domain.
#include "pc_common.cuh"

namespace {

constexpr int AT_THREADS = 128, AT_ROWS = 32, AT_KEYS = 32;

struct SegTable {
    const void *k[PC_MAX_SEGMENTS];
    const void *v[PC_MAX_SEGMENTS];
    const int32_t *pos[PC_MAX_SEGMENTS];
    int32_t end[PC_MAX_SEGMENTS];   // running key count after each segment
    int32_t n_seg;
    int32_t n_keys;
};

template <typename T> __device__ __forceinline__ float2 load_pair(const T *p);
template <> __device__ __forceinline__ float2 load_pair<float>(const float *p) { return *reinterpret_cast<const float2 *>(p); }
template <> __device__ __forceinline__ float2 load_pair<__nv_bfloat16>(const __nv_bfloat16 *p) {
    const uint32_t w = *reinterpret_cast<const uint32_t *>(p);
    return make_float2(pc_bf16_lo(w), pc_bf16_hi(w));
}
template <typename T> __device__ __forceinline__ void store4(T *p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float *p, float a, float b, float c, float d) {
    *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16 *p, float a, float b, float c, float d) {
    *reinterpret_cast<uint2 *>(p) = make_uint2(pc_pack_bf16(a, b), pc_pack_bf16(c, d));
}

template <typename T, int D>
__global__ void __launch_bounds__(AT_THREADS) k_attend_simt(const T *__restrict__ q, const int32_t *__restrict__ q_pos,
                                                            int n_q, int n_q_heads, int n_kv_heads, SegTable seg,
                                                            pc_rope_dev rope, T *__restrict__ out,
                                                            float *__restrict__ lse, int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    constexpr int NC = D / 16;                       // 4-element groups per thread
    __shared__ __align__(16) float sk[AT_KEYS][D];
    __shared__ __align__(16) float sv[AT_KEYS][D];
    const int tid = threadIdx.x, sub = tid & 3;
    const int row = blockIdx.x * AT_ROWS + (tid >> 2);
    const int h = blockIdx.y, g = h / (n_q_heads / n_kv_heads);
    const bool live = row < n_q;
    const float scale = 1.4426950408889634f * rsqrtf((float)D);

    float qr[NC][4], o[NC][4];
#pragma unroll
    for (int c = 0; c < NC; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) { qr[c][e] = 0.f; o[c][e] = 0.f; }
    if (live) {
        const int4 pp = __ldg(reinterpret_cast<const int4 *>(q_pos) + row);
        const T *qrow = q + ((size_t)row * n_q_heads + h) * D;
#pragma unroll
        for (int c = 0; c < NC; ++c)
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int ch = 16 * c + 4 * sub + 2 * u;
                const float2 x = load_pair<T>(qrow + ch);
                const float2 cs = pc_rope_cs(rope, ch / 2, pp.x, pp.y, pp.z, status, PC_WHERE_ATTN_POS);
                qr[c][2 * u] = (x.x * cs.x - x.y * cs.y) * scale;
                qr[c][2 * u + 1] = (x.x * cs.y + x.y * cs.x) * scale;
            }
    }
    float m = -INFINITY, l = 0.f;

    for (int k0 = 0; k0 < seg.n_keys; k0 += AT_KEYS) {
        __syncthreads();
        // copy the tile: K rotated, V plain
        for (int p = tid; p < AT_KEYS * (D / 2); p += AT_THREADS) {
            const int kk = p / (D / 2), pair = p % (D / 2);
            const int key = k0 + kk;
            float2 kx = make_float2(0.f, 0.f), vx = make_float2(0.f, 0.f);
            if (key < seg.n_keys) {
                int s = 0, base = 0;
                while (s < seg.n_seg - 1 && key >= seg.end[s]) { base = seg.end[s]; ++s; }
                const size_t at = ((size_t)(key - base) * n_kv_heads + g) * D + 2 * pair;
                const int4 pp = __ldg(reinterpret_cast<const int4 *>(seg.pos[s]) + (key - base));
                const float2 x = load_pair<T>(static_cast<const T *>(seg.k[s]) + at);
                const float2 cs = pc_rope_cs(rope, pair, pp.x, pp.y, pp.z, status, PC_WHERE_ATTN_POS);
                kx = make_float2(x.x * cs.x - x.y * cs.y, x.x * cs.y + x.y * cs.x);
                vx = load_pair<T>(static_cast<const T *>(seg.v[s]) + at);
            }
            *reinterpret_cast<float2 *>(&sk[kk][2 * pair]) = kx;
            *reinterpret_cast<float2 *>(&sv[kk][2 * pair]) = vx;
        }
        __syncthreads();
        const int n_here = min(AT_KEYS, seg.n_keys - k0);
        for (int kb = 0; kb < n_here; kb += 8) {
            float x[8];
            float bm = -INFINITY;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float dot = 0.f;
                const int kk = min(kb + i, AT_KEYS - 1);
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const float4 kv = *reinterpret_cast<const float4 *>(&sk[kk][16 * c + 4 * sub]);
                    dot = fmaf(qr[c][0], kv.x, fmaf(qr[c][1], kv.y, fmaf(qr[c][2], kv.z, fmaf(qr[c][3], kv.w, dot))));
                }
                dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                x[i] = (kb + i < n_here) ? dot : -INFINITY;
                bm = fmaxf(bm, x[i]);
            }
            const float m_new = fmaxf(m, bm);
            const float corr = exp2f(m - m_new);     // exp2f(-inf) = 0 on the first block
            l *= corr;
#pragma unroll
            for (int c = 0; c < NC; ++c)
#pragma unroll
                for (int e = 0; e < 4; ++e) o[c][e] *= corr;
            m = m_new;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float p = exp2f(x[i] - m);
                l += p;
                const int kk = min(kb + i, AT_KEYS - 1);
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const float4 vv = *reinterpret_cast<const float4 *>(&sv[kk][16 * c + 4 * sub]);
                    o[c][0] = fmaf(p, vv.x, o[c][0]);
                    o[c][1] = fmaf(p, vv.y, o[c][1]);
                    o[c][2] = fmaf(p, vv.z, o[c][2]);
                    o[c][3] = fmaf(p, vv.w, o[c][3]);
                }
            }
        }
    }
    if (!live) return;
    const float inv = 1.f / l;
    T *orow = out + ((size_t)row * n_q_heads + h) * D;
#pragma unroll
    for (int c = 0; c < NC; ++c)
        store4<T>(orow + 16 * c + 4 * sub, o[c][0] * inv, o[c][1] * inv, o[c][2] * inv, o[c][3] * inv);
    if (lse && sub == 0) lse[(size_t)row * n_q_heads + h] = (m + log2f(l)) * 0.6931471805599453f;
}

}  // namespace

pc_status pc_launch_attend_simt(pc_ctx *ctx, int n_seg, const pc_segment *segs, const void *q, const int32_t *q_pos,
                                int32_t n_q, void *out, float *lse, cudaStream_t stream) {
    const pc_layer_desc &D = ctx->desc;
    SegTable t{};
    int total = 0;
    t.n_seg = n_seg;
    for (int s = 0; s < n_seg; ++s) {
        t.k[s] = segs[s].k;
        t.v[s] = segs[s].v;
        t.pos[s] = segs[s].pos;
        total += segs[s].n_tokens;
        t.end[s] = total;
    }
    t.n_keys = total;
    dim3 grid((n_q + AT_ROWS - 1) / AT_ROWS, D.n_q_heads);
    pc_mark(ctx, PC_MARK_ROPE, stream);
#define PC_AT_LAUNCH(T, DIM)                                                                                          \
    PC_LAUNCH((k_attend_simt<T, DIM>), dim3(grid), dim3(AT_THREADS), 0, stream, static_cast<const T *>(q), q_pos, n_q, D.n_q_heads,         \
                                                          D.n_kv_heads, t, ctx->rope, static_cast<T *>(out), lse,    \
                                                          ctx->status)
    if (D.dtype == PC_F32) {
        if (D.head_dim == 64) PC_AT_LAUNCH(float, 64); else PC_AT_LAUNCH(float, 128);
    } else {
        if (D.head_dim == 64) PC_AT_LAUNCH(__nv_bfloat16, 64); else PC_AT_LAUNCH(__nv_bfloat16, 128);
    }
#undef PC_AT_LAUNCH
    PC_CUDA_TRY(cudaGetLastError());
    pc_mark(ctx, PC_MARK_ATTEND, stream);
    return PC_OK;
}
