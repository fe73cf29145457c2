// Attention mass of every cached key on tcgen05 tensor cores (Sec. 3.4: retention guided by the attention a token
// receives):  mass_j = 1/(n_q Hq) * sum over query rows (i, h) of softmax_j((R q_ih).(R k_j,g(h))/sqrt(d)).
//
// The call follows an attention call on the same context and reuses what that call left behind: the rotated keys and
// the rotated, pre-scaled queries (base-2 logits) in the context's scratch, and the log-sum-exp of every query row that
// the attention kernel wrote.  With the normaliser of every row known, a key's mass is a plain column sum of
// 2^(s_ij - lse2_i), so no running maximum and no second operand are needed:
//
//   k_mass_norm    writes minus the base-2 normaliser of every query row, transposed to [head][row] and padded with
//                  -inf to whole tiles, so that one step's 128 values are one contiguous 512-byte run.
//   k_mass_tc      one CTA = two 128-key tiles of one KV head, which stay in shared memory; the query tiles of the
//                  head's group stream through a four-stage TMA ring, each stage feeding both key tiles (a CTA per
//                  single key tile reads every query tile twice as often from L2 for no gain).  The step's
//                  normalisers ride along as a bulk copy into an eight-slot ring.  S^T = K Q^T (keys on the TMEM lanes,
//                  queries on the columns) goes to one of two TMEM buffers per key tile.  Sixteen warps turn scores
//                  into sums: per key tile and column half one warp per TMEM lane quadrant, one key per thread, 64
//                  columns per step: 2^(s + (-lse2)) added up in registers.  Four such warps share each scheduler, so
//                  the waits of one hide behind the exponentials of the others; with two warps per scheduler (128
//                  columns per thread) and a per-step meeting of the warps to stage the normalisers, a third of
//                  every step was dead time.  The kernel is bound by the exponentials.
//   k_mass_reduce  adds the partial sums of the KV heads and column halves in a fixed order, divides by n_q Hq and drops the padding rows
//                  between segments.
// Every wait is bounded as in the attention kernel.
#include "pc_tc.cuh"

namespace {

using namespace pc_tc;

constexpr int MASS_THREADS = 640;          // warp 0 TMA + TMEM owner, warp 1 MMA issuer, warps 4-19 column sums
constexpr int Q_STAGES = 4;
constexpr int L_SLOTS = 8;                 // normaliser ring: deeper than query stages + score buffers, see the producer

constexpr int SM_K = 0;                                  // 2 key tiles
constexpr int SM_Q = SM_K + 2 * TILE_BYTES;              // Q_STAGES query tiles
constexpr int SM_BAR = SM_Q + Q_STAGES * TILE_BYTES;
constexpr int SM_LSE = SM_BAR + 256;                     // [L_SLOTS][128] fp32: minus the base-2 normaliser of each query row
constexpr int SM_TOTAL = SM_LSE + L_SLOTS * TILE * 4;
constexpr int SM_ALLOC = SM_TOTAL + 1024;

enum { BAR_K = 0, BAR_QFULL = 1, BAR_QEMPTY = BAR_QFULL + Q_STAGES, BAR_SFULL = BAR_QEMPTY + Q_STAGES /* [tile][buffer] */,
       BAR_SEMPTY = BAR_SFULL + 4, BAR_LFULL = BAR_SEMPTY + 4, BAR_DONE = BAR_LFULL + L_SLOTS, N_BARS = BAR_DONE + 1 };
static_assert(N_BARS * 8 + 16 <= 256, "barrier area");

struct MassParams {
    int n_q, n_q_heads, group, n_tb, n_kv_tiles, pairs;    // pairs = key-tile pairs per KV head
    const float *lse;      // [n_q][Hq] natural log
    float *norm;           // [Hq][n_tb * 128]: -log2(e) * lse, -inf past n_q
    float *part;           // [Hkv][2 column halves][n_kv_tiles * 128]
    int32_t *status;
};

__global__ void __launch_bounds__(256) k_mass_norm(const __grid_constant__ MassParams P) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int rows = P.n_tb * TILE;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * P.n_q_heads) return;
    const int row = idx / P.n_q_heads, h = idx % P.n_q_heads;         // consecutive threads read consecutive floats
    P.norm[(size_t)h * rows + row] = row < P.n_q ? -1.4426950408889634f * __ldg(P.lse + idx) : -INFINITY;
}

__global__ void __launch_bounds__(MASS_THREADS, 1)
k_mass_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
          const __grid_constant__ MassParams P) {
    pc_grid_dep_launch();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + SM_BAR + N_BARS * 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(gen + SM_BAR + N_BARS * 8 + 8);
    const uint32_t bar0 = base + SM_BAR;
    auto bar = [&](int i) { return bar0 + 8u * i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.x / P.pairs, jt0 = 2 * (blockIdx.x % P.pairs);
    const int n_t = min(2, P.n_kv_tiles - jt0);           // 1 when the tile count is odd
    const int n_steps = P.group * P.n_tb;                 // query tiles of this KV head's group

    if (threadIdx.x == 0) {
        mbar_init(bar(BAR_K), 1);
        for (int s = 0; s < Q_STAGES; ++s) {
            mbar_init(bar(BAR_QFULL + s), 1);
            mbar_init(bar(BAR_QEMPTY + s), 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar(BAR_SFULL + i), 1);
            mbar_init(bar(BAR_SEMPTY + i), 256);
        }
        for (int i = 0; i < L_SLOTS; ++i) mbar_init(bar(BAR_LFULL + i), 1);
        mbar_init(bar(BAR_DONE), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 0) {   // two score buffers of 128 columns per key tile
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    pc_grid_dep_wait();   // from here on the rotated K / Q of the attention call and the normalisers are read

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar(BAR_K), n_t * TILE_BYTES);
            for (int t = 0; t < n_t; ++t) {
                tma_load_2d(base + SM_K + t * TILE_BYTES, &map_k, g * TILE, (jt0 + t) * TILE, bar(BAR_K));
                tma_load_2d(base + SM_K + t * TILE_BYTES + HALF_BYTES, &map_k, g * TILE + 64, (jt0 + t) * TILE, bar(BAR_K));
            }
            bool alive = true;
            for (int s = 0; s < n_steps && alive; ++s) {
                const int st = s % Q_STAGES, use = s / Q_STAGES;
                if (use > 0) alive = mbar_wait(bar(BAR_QEMPTY + st), (use - 1) & 1, abort_flag, P.status, PC_WHERE_MASS_WAIT);
                if (!alive) break;
                const int tb = s / P.group, h = g * P.group + s % P.group;
                mbar_expect_tx(bar(BAR_QFULL + st), TILE_BYTES);
                tma_load_2d(base + SM_Q + st * TILE_BYTES, &map_q, h * TILE, tb * TILE, bar(BAR_QFULL + st));
                tma_load_2d(base + SM_Q + st * TILE_BYTES + HALF_BYTES, &map_q, h * TILE + 64, tb * TILE, bar(BAR_QFULL + st));
                // The step's normalisers go to slot s mod 8.  Its previous tenant, step s - 8, is out of use: this point
                // is reached after the products of step s - 4 completed, those needed the score buffers of step s - 6
                // released, and a buffer is released only after the step before it was summed up.
                const int slot = s % L_SLOTS;
                mbar_expect_tx(bar(BAR_LFULL + slot), TILE * 4);
                pc_bulk_g2s(base + SM_LSE + slot * TILE * 4, P.norm + ((size_t)h * P.n_tb + tb) * TILE, TILE * 4, bar(BAR_LFULL + slot));
            }
            if (*abort_flag) {
                // give the copies already issued a bounded chance to land before the CTA's shared memory goes away
                const uint64_t t0 = global_ns();
                while (global_ns() - t0 < 2000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (converged warp, one elected lane)
        const bool lead = elect_one();
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
        bool alive = mbar_wait(bar(BAR_K), 0, abort_flag, P.status, PC_WHERE_MASS_WAIT);
        for (int s = 0; s < n_steps && alive; ++s) {
            const int st = s % Q_STAGES, quse = s / Q_STAGES, b = s & 1, use = s >> 1;
            alive = mbar_wait(bar(BAR_QFULL + st), quse & 1, abort_flag, P.status, PC_WHERE_MASS_WAIT);
            for (int t = 0; t < n_t && alive; ++t) {
                if (use > 0) alive = mbar_wait(bar(BAR_SEMPTY + 2 * t + b), (use - 1) & 1, abort_flag, P.status, PC_WHERE_MASS_WAIT);
                if (!alive) break;
                tc_fence_after();
                const uint32_t ka = base + SM_K + t * TILE_BYTES, qa = base + SM_Q + st * TILE_BYTES;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                    if (lead) mma_ss(tm + (2 * t + b) * TILE, desc_kmajor(ka + off), desc_kmajor(qa + off), IDESC_QK, ks > 0);
                }
                if (lead) tc_commit(bar(BAR_SFULL + 2 * t + b));
            }
            if (alive && lead) tc_commit(bar(BAR_QEMPTY + st));
        }
        // nothing of ours may still be running on the tensor core when TMEM is freed
        if (lead) tc_commit(bar(BAR_DONE));
        __syncwarp();
        mbar_wait(bar(BAR_DONE), 0, abort_flag, P.status, PC_WHERE_MASS_WAIT);
    } else if (warp >= 4 && (warp - 4) >> 3 < n_t) {
        // ---------------------------------------------------------------- column sums: one key and 64 query columns per thread
        const int cw = warp - 4;
        const int t = cw >> 3, hf = (cw >> 2) & 1;        // key tile and column half of this warp
        const int quad = warp & 3;                        // TMEM lane quadrant this warp may touch
        const int r = quad * 32 + lane;                   // key row of the tile
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const float *lse_s = reinterpret_cast<const float *>(gen + SM_LSE) + hf * 64;
        float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
        bool alive = true;
        for (int s = 0; s < n_steps && alive; ++s) {
            const int b = s & 1, use = s >> 1, slot = s % L_SLOTS;
            alive = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SFULL + 2 * t + b), use & 1, abort_flag, P.status, PC_WHERE_MASS_WAIT) &&
                                                mbar_wait(bar(BAR_LFULL + slot), (s / L_SLOTS) & 1, abort_flag, P.status, PC_WHERE_MASS_WAIT));
            if (!alive) break;
            tc_fence_after();
            uint32_t sv[64];
            const uint32_t s_addr = tmem + lane_addr + (2 * t + b) * TILE + hf * 64;
            tmem_ld32(s_addr, sv);
            tmem_ld32(s_addr + 32, sv + 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(BAR_SEMPTY + 2 * t + b));     // the buffer may take the scores of step s + 2
            const float4 *nl = reinterpret_cast<const float4 *>(lse_s + slot * TILE);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const float4 m = nl[c];                   // the same address in every lane: a broadcast
                float2 x = add2(make_float2(__uint_as_float(sv[4 * c]), __uint_as_float(sv[4 * c + 1])), make_float2(m.x, m.y));
                float2 y = add2(make_float2(__uint_as_float(sv[4 * c + 2]), __uint_as_float(sv[4 * c + 3])), make_float2(m.z, m.w));
                x.x = fast_exp2(x.x); x.y = fast_exp2(x.y);
                y.x = fast_exp2(y.x); y.y = fast_exp2(y.y);
                acc0 = add2(acc0, x);
                acc1 = add2(acc1, y);
            }
        }
        if (alive) P.part[(((size_t)g * 2 + hf) * P.n_kv_tiles + jt0 + t) * TILE + r] = (acc0.x + acc0.y) + (acc1.x + acc1.y);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

struct ReduceParams {
    int n_seg, n_kv_heads, n_kv_tiles;
    int seg_first[PC_MAX_SEGMENTS + 1];     // first key of each segment in the output order; [n_seg] = all keys
    int seg_tile0[PC_MAX_SEGMENTS];         // first tile of each segment in the rotated-key scratch
    float inv_rows;                         // 1 / (n_q Hq)
};

__global__ void __launch_bounds__(256) k_mass_reduce(const __grid_constant__ ReduceParams R, const float *__restrict__ part,
                                                     float *__restrict__ mass) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= R.seg_first[R.n_seg]) return;
    int s = 0;
    while (s + 1 < R.n_seg && j >= R.seg_first[s + 1]) ++s;
    const size_t row = (size_t)R.seg_tile0[s] * TILE + (j - R.seg_first[s]);
    float sum = 0.f;
    for (int g = 0; g < 2 * R.n_kv_heads; ++g) sum += part[(size_t)g * R.n_kv_tiles * TILE + row];   // [head][column half]
    mass[j] = sum * R.inv_rows;
}

}  // namespace

extern "C" pc_status pc_attend_mass(pc_ctx *ctx, const float *lse, float *mass, int32_t n_keys, void *stream_) {
    if (!ctx || !lse || !mass) return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(lse) || !pc_aligned16(mass)) return PC_ERR_INVALID_ARG;
    const pc_layer_desc &D = ctx->desc;
    if (!pc_tensor_core_shape(ctx) || ctx->attend_impl == 1) return PC_ERR_UNSUPPORTED;
    if (ctx->last_n_q <= 0 || ctx->last_n_seg <= 0) return PC_ERR_INVALID_ARG;   // no tensor-core attention call precedes
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    MassParams P{};
    ReduceParams R{};
    int tiles = 0, keys = 0;
    for (int s = 0; s < ctx->last_n_seg; ++s) {
        R.seg_first[s] = keys;
        R.seg_tile0[s] = tiles;
        keys += ctx->last_seg_n[s];
        tiles += (ctx->last_seg_n[s] + TILE - 1) / TILE;
    }
    R.seg_first[ctx->last_n_seg] = keys;
    if (n_keys != keys) return PC_ERR_INVALID_ARG;
    if ((size_t)tiles * TILE > ctx->k_rot_rows) return PC_ERR_CAPACITY;
    R.n_seg = ctx->last_n_seg;
    R.n_kv_heads = D.n_kv_heads;
    R.n_kv_tiles = tiles;
    R.inv_rows = (float)(1.0 / ((double)ctx->last_n_q * D.n_q_heads));
    P.n_q = ctx->last_n_q;
    P.n_q_heads = D.n_q_heads;
    P.group = ctx->group;
    P.n_tb = (P.n_q + TILE - 1) / TILE;
    P.n_kv_tiles = tiles;
    P.pairs = (tiles + 1) / 2;
    P.lse = lse;
    P.part = ctx->mass_part;
    P.norm = ctx->mass_norm;
    P.status = ctx->status;

    CUtensorMap mq, mk;
    if (!make_map(&mq, ctx->q_rot, (uint64_t)P.n_q, (uint64_t)D.n_q_heads * D.head_dim) ||
        !make_map(&mk, ctx->k_rot, (uint64_t)tiles * TILE, (uint64_t)D.n_kv_heads * D.head_dim)) {
        fprintf(stderr, "packcache: cuTensorMapEncodeTiled failed\n");
        return PC_ERR_CUDA;
    }
    static bool attr_set[PC_MAX_DEVICES] = {};      // the attribute belongs to the device, not to the process
    if (ctx->device < 0 || ctx->device >= PC_MAX_DEVICES) return PC_ERR_UNSUPPORTED;
    if (!attr_set[ctx->device]) {
        PC_CUDA_TRY(cudaFuncSetAttribute(k_mass_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, SM_ALLOC));
        attr_set[ctx->device] = true;
    }
    pc_mark(ctx, PC_MARK_MASS0, stream);
    PC_LAUNCH(k_mass_norm, dim3((P.n_tb * TILE * D.n_q_heads + 255) / 256), dim3(256), 0, stream, P);
    PC_CUDA_TRY(cudaGetLastError());
    PC_LAUNCH(k_mass_tc, dim3(D.n_kv_heads * P.pairs), dim3(MASS_THREADS), SM_ALLOC, stream, mq, mk, P);
    PC_CUDA_TRY(cudaGetLastError());
    PC_LAUNCH(k_mass_reduce, dim3((keys + 255) / 256), dim3(256), 0, stream, R, static_cast<const float *>(ctx->mass_part), mass);
    PC_CUDA_TRY(cudaGetLastError());
    pc_mark(ctx, PC_MARK_MASS, stream);
    return PC_OK;
}
