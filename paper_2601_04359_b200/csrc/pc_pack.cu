// Gather/pack of retained K/V rows into a contiguous cache (Fig. 6b) with the temporal rebase of Eq. 9.
//
// One warp moves one retained token: its K row and V row over all KV heads (16-byte vector loads and stores,
// consecutive lanes on consecutive 16-byte chunks, so every request is a full 512-byte line run) and its position
// record with t shifted by delta_t.  Rows are streamed (no L1 allocation): nothing here is read twice.
// For the fused frame step the same warp also writes the row's rotated keys (3D rotary embedding at the rebased
// position, bf16) into the attention kernel's key scratch: the row is in registers anyway, and the kernel is bound by
// memory, not by issue, so the attention call that follows needs no rotary pre-pass over the packed history.
#include "pc_common.cuh"

namespace {

constexpr int PACK_THREADS = 256;

template <int CPL /* 16-byte chunks per lane per row; 0 = generic loop */>
__global__ void __launch_bounds__(PACK_THREADS) k_pack(const char *__restrict__ src_k, const char *__restrict__ src_v,
                                                       const int32_t *__restrict__ src_pos,
                                                       const int32_t *__restrict__ sel_idx, int n_sel, int n_src,
                                                       int row_bytes, int delta_t, char *__restrict__ dst_k,
                                                       char *__restrict__ dst_v, int32_t *__restrict__ dst_pos,
                                                       int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const int r = (blockIdx.x * PACK_THREADS + threadIdx.x) >> 5;
    if (r >= n_sel) return;
    const int s = __ldg(sel_idx + r);
    if (s < 0 || s >= n_src) {                      // a bad index is recorded and the row skipped
        if (lane == 0) pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_PACK_INDEX);
        return;
    }
    const char *sk = src_k + (size_t)s * row_bytes, *sv = src_v + (size_t)s * row_bytes;
    char *dk = dst_k + (size_t)r * row_bytes, *dv = dst_v + (size_t)r * row_bytes;
    if constexpr (CPL > 0) {
        uint4 a[CPL], b[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) a[c] = pc_ldg_stream(sk + (size_t)(c * 32 + lane) * 16);
#pragma unroll
        for (int c = 0; c < CPL; ++c) b[c] = pc_ldg_stream(sv + (size_t)(c * 32 + lane) * 16);
#pragma unroll
        for (int c = 0; c < CPL; ++c) pc_stg_stream(dk + (size_t)(c * 32 + lane) * 16, a[c]);
#pragma unroll
        for (int c = 0; c < CPL; ++c) pc_stg_stream(dv + (size_t)(c * 32 + lane) * 16, b[c]);
    } else {
        for (int off = lane * 16; off < row_bytes; off += 32 * 16) {
            const uint4 a = pc_ldg_stream(sk + off), b = pc_ldg_stream(sv + off);
            pc_stg_stream(dk + off, a);
            pc_stg_stream(dv + off, b);
        }
    }
    if (lane == 0) {
        int4 p = __ldg(reinterpret_cast<const int4 *>(src_pos) + s);
        p.x -= delta_t;                              // only t moves; h, w and the tag are carried as they are
        reinterpret_cast<int4 *>(dst_pos)[r] = p;
    }
}

// The same with the rotated keys written as well (bf16 rows of CPL x 512 bytes).  Two warps per retained token: the even
// one copies the V row and the position record, the odd one copies the K row and writes its rotated form: more and
// shorter warps than one per token, since the table look-ups add a dependent load to the K side only.
template <int CPL>
__global__ void __launch_bounds__(PACK_THREADS) k_pack_rot(const char *__restrict__ src_k, const char *__restrict__ src_v,
                                                           const int32_t *__restrict__ src_pos,
                                                           const int32_t *__restrict__ sel_idx, int n_sel, int n_src,
                                                           int delta_t, char *__restrict__ dst_k, char *__restrict__ dst_v,
                                                           int32_t *__restrict__ dst_pos, char *__restrict__ rot_k,
                                                           pc_rope_dev rope, int d, int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    constexpr int row_bytes = CPL * 512;
    const int lane = threadIdx.x & 31;
    const int w = (blockIdx.x * PACK_THREADS + threadIdx.x) >> 5;
    const int r = w >> 1, k_side = w & 1;
    if (r >= n_sel) return;
    const int s = __ldg(sel_idx + r);
    if (s < 0 || s >= n_src) {                      // a bad index is recorded and the row skipped
        if (lane == 0 && k_side) pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_PACK_INDEX);
        return;
    }
    const char *src = (k_side ? src_k : src_v) + (size_t)s * row_bytes + lane * 16;
    char *dst = (k_side ? dst_k : dst_v) + (size_t)r * row_bytes + lane * 16;
    uint4 a[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) a[c] = pc_ldg_stream(src + c * 512);
    int4 p = __ldg(reinterpret_cast<const int4 *>(src_pos) + s);
    p.x -= delta_t;                                  // only t moves; h, w and the tag are carried as they are
#pragma unroll
    for (int c = 0; c < CPL; ++c) pc_stg_stream(dst + c * 512, a[c]);
    if (!k_side) {
        if (lane == 0) reinterpret_cast<int4 *>(dst_pos)[r] = p;
        return;
    }
    // 32 lanes x 8 elements span a multiple of d: all of this lane's chunks hold the same four rotary pairs
    const int pair0 = ((lane * 8) % d) / 2;
    float2 cs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) cs[u] = pc_rope_cs(rope, pair0 + u, p.x, p.y, p.z, status, PC_WHERE_ROPE_POS);
    char *rk = rot_k + (size_t)r * row_bytes + lane * 16;
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
        const uint32_t wv[4] = {a[c].x, a[c].y, a[c].z, a[c].w};
        uint32_t o[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 y = pc_rotate(pc_bf16_lo(wv[u]), pc_bf16_hi(wv[u]), cs[u]);
            o[u] = pc_pack_bf16(y.x, y.y);
        }
        *reinterpret_cast<uint4 *>(rk + c * 512) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

bool overlaps(const void *a, size_t na, const void *b, size_t nb) {
    const char *x = static_cast<const char *>(a), *y = static_cast<const char *>(b);
    return x < y + nb && y < x + na;
}

}  // namespace

// Every host-side check of a compaction, nothing enqueued: n_sel / n_src out (either may be NULL).
pc_status pc_compact_check(pc_ctx *ctx, const pc_cache *src, const int32_t *sel_idx, const int32_t *budget, const pc_cache *dst,
                           int64_t *n_sel_out, int64_t *n_src_out) {
    if (!ctx || !src || !dst || !budget) return PC_ERR_INVALID_ARG;
    if (src->n_frames < 0 || (src->n_frames > 0 && !src->frame_count)) return PC_ERR_INVALID_ARG;
    pc_status st = pc_check_segment(&src->history, true);
    if (st != PC_OK) return st;
    int64_t n_sel = 0, n_src = 0;
    for (int f = 0; f < src->n_frames; ++f) {
        if (budget[f] < 0 || src->frame_count[f] < 0) return PC_ERR_INVALID_ARG;
        if (budget[f] > src->frame_count[f]) return PC_ERR_BUDGET;
        n_sel += budget[f];
        n_src += src->frame_count[f];
    }
    if (n_src != src->history.n_tokens) return PC_ERR_INVALID_ARG;
    if (n_sel > dst->history.capacity) return PC_ERR_CAPACITY;
    if (n_sel_out) *n_sel_out = n_sel;
    if (n_src_out) *n_src_out = n_src;
    if (n_sel == 0) return PC_OK;
    if (!sel_idx || !pc_aligned16(sel_idx)) return PC_ERR_INVALID_ARG;
    const pc_segment &D = dst->history;
    if (!D.k || !D.v || !D.pos || !pc_aligned16(D.k) || !pc_aligned16(D.v) || !pc_aligned16(D.pos))
        return PC_ERR_INVALID_ARG;
    const int row_bytes = ctx->desc.n_kv_heads * ctx->desc.head_dim * ctx->elem_size;
    const size_t src_bytes = (size_t)n_src * row_bytes, dst_bytes = (size_t)n_sel * row_bytes;
    if (overlaps(src->history.k, src_bytes, D.k, dst_bytes) || overlaps(src->history.v, src_bytes, D.v, dst_bytes) ||
        overlaps(src->history.k, src_bytes, D.v, dst_bytes) || overlaps(src->history.v, src_bytes, D.k, dst_bytes) ||
        overlaps(src->history.pos, (size_t)n_src * 16, D.pos, (size_t)n_sel * 16))
        return PC_ERR_INVALID_ARG;
    return PC_OK;
}

pc_status pc_compact_impl(pc_ctx *ctx, const pc_cache *src, const int32_t *sel_idx, const int32_t *budget, int32_t delta_t,
                          pc_cache *dst, void *k_rot_dst, cudaStream_t stream) {
    int64_t n_sel = 0, n_src = 0;
    pc_status st = pc_compact_check(ctx, src, sel_idx, budget, dst, &n_sel, &n_src);
    if (st != PC_OK) return st;
    if (n_sel == 0) return PC_OK;
    const pc_segment &D = dst->history;
    pc_mark(ctx, PC_MARK_PACK0, stream);
    st = pc_launch_pack(ctx, src->history.k, src->history.v, src->history.pos, sel_idx, (int)n_sel, (int)n_src, delta_t, D.k, D.v,
                        D.pos, k_rot_dst, stream);
    if (st != PC_OK) return st;
    pc_mark(ctx, PC_MARK_PACK, stream);
    return PC_OK;
}

extern "C" pc_status pc_compact(pc_ctx *ctx, const pc_cache *src, const int32_t *sel_idx, const int32_t *budget,
                                int32_t delta_t, pc_cache *dst, void *stream_) {
    return pc_compact_impl(ctx, src, sel_idx, budget, delta_t, dst, nullptr, static_cast<cudaStream_t>(stream_));
}

// Gather n_sel rows (K, V, position records) of a source of n_src rows into a destination; arguments already checked.
pc_status pc_launch_pack(pc_ctx *ctx, const void *src_k, const void *src_v, const int32_t *src_pos, const int32_t *sel_idx,
                         int n_sel, int n_src, int delta_t, void *dst_k, void *dst_v, int32_t *dst_pos, void *k_rot_dst,
                         cudaStream_t stream) {
    const int row_bytes = ctx->desc.n_kv_heads * ctx->desc.head_dim * ctx->elem_size;
    const int blocks = (int)(((int64_t)n_sel * 32 + PACK_THREADS - 1) / PACK_THREADS);
    const char *sk = static_cast<const char *>(src_k), *sv = static_cast<const char *>(src_v);
    char *dk = static_cast<char *>(dst_k), *dv = static_cast<char *>(dst_v), *rk = static_cast<char *>(k_rot_dst);
    const int d = ctx->desc.head_dim;
    if (rk) {
        // rotated keys are written for bf16 rows whose 32 x 16-byte chunk rows span whole heads (the tensor-core shapes)
        if (ctx->desc.dtype != PC_BF16 || 256 % d) return PC_ERR_UNSUPPORTED;
        const int blocks2 = (int)(((int64_t)n_sel * 64 + PACK_THREADS - 1) / PACK_THREADS);
#define PC_PACK_ROT_ARGS sk, sv, src_pos, sel_idx, n_sel, n_src, delta_t, dk, dv, dst_pos, rk, ctx->rope, d, ctx->status
        switch (row_bytes) {
        case 512: PC_LAUNCH((k_pack_rot<1>), dim3(blocks2), dim3(PACK_THREADS), 0, stream, PC_PACK_ROT_ARGS); break;
        case 1024: PC_LAUNCH((k_pack_rot<2>), dim3(blocks2), dim3(PACK_THREADS), 0, stream, PC_PACK_ROT_ARGS); break;
        case 1536: PC_LAUNCH((k_pack_rot<3>), dim3(blocks2), dim3(PACK_THREADS), 0, stream, PC_PACK_ROT_ARGS); break;
        case 2048: PC_LAUNCH((k_pack_rot<4>), dim3(blocks2), dim3(PACK_THREADS), 0, stream, PC_PACK_ROT_ARGS); break;
        case 3072: PC_LAUNCH((k_pack_rot<6>), dim3(blocks2), dim3(PACK_THREADS), 0, stream, PC_PACK_ROT_ARGS); break;
        case 4096: PC_LAUNCH((k_pack_rot<8>), dim3(blocks2), dim3(PACK_THREADS), 0, stream, PC_PACK_ROT_ARGS); break;
        default: return PC_ERR_UNSUPPORTED;
        }
#undef PC_PACK_ROT_ARGS
    } else {
#define PC_PACK_ARGS sk, sv, src_pos, sel_idx, n_sel, n_src, row_bytes, delta_t, dk, dv, dst_pos, ctx->status
        switch (row_bytes) {
        case 512: PC_LAUNCH((k_pack<1>), dim3(blocks), dim3(PACK_THREADS), 0, stream, PC_PACK_ARGS); break;
        case 1024: PC_LAUNCH((k_pack<2>), dim3(blocks), dim3(PACK_THREADS), 0, stream, PC_PACK_ARGS); break;
        case 2048: PC_LAUNCH((k_pack<4>), dim3(blocks), dim3(PACK_THREADS), 0, stream, PC_PACK_ARGS); break;
        default: PC_LAUNCH((k_pack<0>), dim3(blocks), dim3(PACK_THREADS), 0, stream, PC_PACK_ARGS); break;
        }
#undef PC_PACK_ARGS
    }
    PC_CUDA_TRY(cudaGetLastError());
    return PC_OK;
}
