// bf16 attention of one frame's queries over the compacted cache on tcgen05 tensor cores (Eq. 2, all keys visible).
//
// Launch sequence of pc_launch_attend_tc:
//   k_rope_rows   rotates K of every segment (3D rotary tables, from the stored positions) into a bf16 scratch whose
//                 segments start on 128-row boundaries, and rotates Q with log2(e)/sqrt(d) folded in.
//   k_attend_tc   persistent CTAs (one per SM) share the line of (item, key tile) steps evenly; an item = two 128-row
//                 query tiles that share a KV head (grouped-query packing).
//                 Warp 0 lane 0 drives TMA (K and V tiles, 128B swizzle, two stages each), warp 1 lane 0 issues
//                 tcgen05.mma: S_t = Q_t K^T (both operands K-major in shared memory) into TMEM, and
//                 O_t += P_t V with P_t read from TMEM and V MN-major in shared memory.  Warps 4-7 / 8-11 are the
//                 softmax groups of tile 0 / 1: tcgen05.ld the S row, running max and sum in fp32 (base 2), write
//                 bf16 P over S in TMEM (handed over in two halves of 64 keys), and rescale O in TMEM only when
//                 the running max moved by more than 2^8.
//                 While one tile's softmax runs, the tensor core works on the other tile.
//   Key ranges of one work item are launched as a thread-block cluster and merge their (max, sum, O) through
//   distributed shared memory at the end of the kernel; k_combine does the same from global partials when the
//   cluster merge is switched off.
//
// TMEM columns: S0/P0 0-127, S1/P1 128-255, O0 256-383, O1 384-511 (fp32, 128 lanes = the tile's rows).
// Every wait is bounded: a wait that runs out records PC_ERR_TIMEOUT, raises a CTA-wide abort flag that makes every
// later wait return at once, and the CTA still drains its copies, frees TMEM and exits.
#include <algorithm>

#include "pc_tc.cuh"

namespace {

using namespace pc_tc;

constexpr int TC_THREADS = 384;
constexpr int KV_STAGES = 2;
constexpr int MAX_SPLITS = 4;
constexpr float RESCALE_THRESHOLD = 8.0f;

// shared memory map (dynamic, 1024-byte aligned)
constexpr int SM_Q = 0;                                   // 2 tiles
constexpr int SM_K = SM_Q + 2 * TILE_BYTES;               // KV_STAGES tiles
constexpr int SM_V = SM_K + KV_STAGES * TILE_BYTES;       // KV_STAGES tiles
constexpr int SM_BAR = SM_V + KV_STAGES * TILE_BYTES;     // barriers etc.
constexpr int SM_ML = SM_BAR + 256;                       // (max, sum) of both tiles' rows for the cluster merge: 2 KB
constexpr int SM_TOTAL = SM_ML + 2 * TILE * 8;
constexpr int SM_ALLOC = SM_TOTAL + 1024;                 // slack for manual alignment

enum { BAR_Q = 0, BAR_QFREE = 1, BAR_KEMPTY = 2, BAR_VFULL = 5, BAR_VEMPTY = 7, BAR_SFULL = 9, BAR_PHALF = 11 /* [tile][half] */,
       BAR_DONE = 15, N_BARS = 16 };

struct TcParams {
    int n_q, n_q_heads, group, n_tb, tiles_per_g, pairs_per_g, n_splits, n_kv_tiles;
    int n_items;      // (KV head, pair of query tiles)
    int persistent;   // 1: n_cta CTAs share the line of (item, key tile) steps evenly; 0: CTA (item, s) takes one of n_splits ranges
    int n_cta;
    int part_stride;  // partial slots reserved per item (most parts any item has)
    int n_seg;
    int cluster;      // 1: the KV ranges of one item form a thread-block cluster and merge through shared memory
    uint32_t wait_us; // limit of every bounded wait in microseconds (0 = about one second)
    uint32_t extra_tx; // test hook: bytes the first barrier expects beyond what is sent, so that its wait runs out (0 = off)
    int seg_tile_end[PC_MAX_SEGMENTS];
    int seg_n[PC_MAX_SEGMENTS];
    __nv_bfloat16 *out;
    float *lse;
    float *part_o;    // [item*S + s][2] tiles of 128 x 128 fp32, 16-byte unit (c4, r) at c4*128 + r
    float *part_ml;   // [item*S + s][2][128][2]
    int32_t *status;
};

// ------------------------------------------------------------------------------------------------ rotary pre-pass
struct RopeJob {
    const __nv_bfloat16 *src;
    const int32_t *pos;
    __nv_bfloat16 *dst;
    int n_rows, chunks_per_row /* 16-byte chunks, a multiple of 32 */, first_warp;
    int rows_per_pos;      // consecutive rows that share one position record (a wide query row is cut into slices)
    float scale;
};
struct RopeJobs { RopeJob job[PC_MAX_SEGMENTS + 1]; int n_jobs, total_warps; };

// One warp per row (a query row wider than a key row is cut into key-row-wide slices, one warp each, so that all warps
// carry the same load).  32 lanes x 8 elements = 256 is a multiple of d, so all of a lane's chunks (lane, lane + 32, ...)
// hold the same four rotary pairs: four table entries per lane per row serve every chunk; the output scale (1 for keys)
// is applied after the rotation, exactly as the query pass of the scoring stage does, so both give the same bits.  All of a row's chunks are loaded before any is used.
template <int CPL /* chunks per lane */>
__device__ __forceinline__ void rope_row(const RopeJob &J, int row, int lane, const float2 (&cs)[4], float scale) {
    const uint4 *src = reinterpret_cast<const uint4 *>(J.src) + (size_t)row * (CPL * 32) + lane;
    uint4 *dst = reinterpret_cast<uint4 *>(J.dst) + (size_t)row * (CPL * 32) + lane;
    uint4 v[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) v[c] = pc_ldg_stream(src + c * 32);
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
        const uint32_t w[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
        uint32_t o[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 y = pc_rotate(pc_bf16_lo(w[u]), pc_bf16_hi(w[u]), cs[u]);
            o[u] = pc_pack_bf16(__fmul_rn(y.x, scale), __fmul_rn(y.y, scale));
        }
        dst[c * 32] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

__global__ void __launch_bounds__(256) k_rope_rows(const __grid_constant__ RopeJobs jobs, pc_rope_dev rope, int d,
                                                   int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp >= jobs.total_warps) return;
    int ji = 0;
    while (ji + 1 < jobs.n_jobs && warp >= jobs.job[ji + 1].first_warp) ++ji;
    const RopeJob &J = jobs.job[ji];
    const int row = warp - J.first_warp;
    const int4 pp = __ldg(reinterpret_cast<const int4 *>(J.pos) + row / J.rows_per_pos);
    const int pair0 = ((lane * 8) % d) / 2;
    float2 cs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) cs[u] = pc_rope_cs(rope, pair0 + u, pp.x, pp.y, pp.z, status, PC_WHERE_ROPE_POS);
    const float scale = J.scale;
    switch (J.chunks_per_row >> 5) {
    case 4: rope_row<4>(J, row, lane, cs, scale); break;        // 8 KV heads x 128
    case 12: rope_row<12>(J, row, lane, cs, scale); break;      // 24 query heads x 128
    case 1: rope_row<1>(J, row, lane, cs, scale); break;
    case 2: rope_row<2>(J, row, lane, cs, scale); break;
    case 8: rope_row<8>(J, row, lane, cs, scale); break;
    case 16: rope_row<16>(J, row, lane, cs, scale); break;
    default:
        for (int c = 0; c < (J.chunks_per_row >> 5); ++c) {
            const uint4 *src = reinterpret_cast<const uint4 *>(J.src) + (size_t)row * J.chunks_per_row + c * 32 + lane;
            uint4 *dst = reinterpret_cast<uint4 *>(J.dst) + (size_t)row * J.chunks_per_row + c * 32 + lane;
            const uint4 v = pc_ldg_stream(src);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            uint32_t o[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float2 y = pc_rotate(pc_bf16_lo(w[u]), pc_bf16_hi(w[u]), cs[u]);
                o[u] = pc_pack_bf16(__fmul_rn(y.x, scale), __fmul_rn(y.y, scale));
            }
            *dst = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// ------------------------------------------------------------------------------------------------ main kernel
__device__ __forceinline__ void kv_tile_info(const TcParams &P, int jt, int &seg, int &local, int &n_valid) {
    seg = 0;
    int start = 0;
    while (seg + 1 < P.n_seg && jt >= P.seg_tile_end[seg]) { start = P.seg_tile_end[seg]; ++seg; }
    local = jt - start;
    n_valid = min(TILE, P.seg_n[seg] - local * TILE);
}

// ---- work decomposition.  The (item, key tile) pairs of a call form one line of n_items * n_kv_tiles steps, item-major.
// A CTA takes a contiguous run of it.  Persistent form: n_cta CTAs (one per SM) share the line evenly, so a CTA's run
// usually crosses from one item into the next; set-up (barriers, tensor memory) is paid once per CTA, the next item's
// queries and first keys arrive under the current item's last steps, and all SMs finish together.  Split form: CTA
// (item, s) takes the s-th of n_splits equal ranges of one item (used when the caller fixes the number of key ranges, and
// by the cluster merge).  The part of an item one CTA works on is a "unit"; an item's units are numbered by "part".
__device__ __forceinline__ void cta_run(const TcParams &P, int c, long long &g0, long long &g1) {
    if (P.persistent) {
        const long long T = (long long)P.n_items * P.n_kv_tiles;
        g0 = T * c / P.n_cta;
        g1 = T * (c + 1) / P.n_cta;
    } else {
        const int item = c / P.n_splits, s = c % P.n_splits;
        g0 = (long long)item * P.n_kv_tiles + (long long)P.n_kv_tiles * s / P.n_splits;
        g1 = (long long)item * P.n_kv_tiles + (long long)P.n_kv_tiles * (s + 1) / P.n_splits;
    }
}
// persistent form: the CTA whose run holds step x
__device__ __forceinline__ int cta_of_step(const TcParams &P, long long x) {
    const long long T = (long long)P.n_items * P.n_kv_tiles;
    return (int)(((x + 1) * P.n_cta + T - 1) / T) - 1;
}
// number of parts of an item, and the part the unit of CTA c is
__device__ __forceinline__ void item_parts(const TcParams &P, int item, int c, int &part, int &parts) {
    if (P.persistent) {
        const int first = cta_of_step(P, (long long)item * P.n_kv_tiles);
        const int last = cta_of_step(P, (long long)item * P.n_kv_tiles + P.n_kv_tiles - 1);
        part = c - first;
        parts = last - first + 1;
    } else {
        part = c % P.n_splits;
        parts = P.n_splits;
    }
}
struct Unit { int item, jb, n_j; };   // key tiles jb .. jb + n_j - 1 of an item
__device__ __forceinline__ Unit unit_at(const TcParams &P, long long g, long long g1) {
    Unit u;
    u.item = (int)(g / P.n_kv_tiles);
    u.jb = (int)(g - (long long)u.item * P.n_kv_tiles);
    u.n_j = (int)min((long long)(P.n_kv_tiles - u.jb), g1 - g);
    return u;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
k_attend_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
            const __grid_constant__ CUtensorMap map_v0, const __grid_constant__ CUtensorMap map_v1,
            const __grid_constant__ CUtensorMap map_v2, const __grid_constant__ TcParams P) {
    pc_grid_dep_launch();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + SM_BAR + N_BARS * 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(gen + SM_BAR + N_BARS * 8 + 8);
    const uint32_t bar0 = base + SM_BAR;
    auto bar = [&](int i) { return bar0 + 8u * i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    long long G0, G1;
    cta_run(P, (int)blockIdx.x, G0, G1);           // this CTA's run of steps (never empty: the host sizes the grid so)

    if (threadIdx.x == 0) {
        mbar_init(bar(BAR_Q), 1);
        mbar_init(bar(BAR_QFREE), 1);
        mbar_init(bar(BAR_KEMPTY), 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(bar(BAR_VFULL + s), 1);
            mbar_init(bar(BAR_VEMPTY + s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar(BAR_SFULL + t), 1);
            mbar_init(bar(BAR_PHALF + 2 * t), 128);
            mbar_init(bar(BAR_PHALF + 2 * t + 1), 128);
        }
        mbar_init(bar(BAR_DONE), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {   // TMEM: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    pc_grid_dep_wait();   // barriers and TMEM are set up; from here on the rotated K / Q are read

    // Steps are counted through the whole run (gs): ring stages and barrier phases follow gs, so a unit boundary is an
    // ordinary step for the key / value pipeline.  Both query tiles always run; a unit whose head group has an odd tile
    // count loads its one tile twice and the second copy's result is dropped.
    // the softmax warps hold a whole 128-column score row per thread: registers move from warps 0-3 to warps 4-11
    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        reg_dealloc<72>();
        if (lane == 0) {
            // A unit's query tiles arrive on BAR_Q once the last QK^T of the unit before has completed (BAR_QFREE); the
            // run's first K tile rides with the first queries.  After that V(step) and K(step + 1) always travel together:
            // they are needed at the same point and their stages are released at the same point, so one full / empty
            // barrier pair serves both.  K(step + 1) may be the first tile of the next unit.
            bool alive = true;
            int gs = 0, un = 0;
            for (long long g = G0; g < G1 && alive; ++un) {
                const Unit U = unit_at(P, g, G1);
                g += U.n_j;
                const int kvh = U.item / P.pairs_per_g, pair = U.item % P.pairs_per_g;
                const int n_tiles_q = min(2, P.tiles_per_g - 2 * pair);
                if (un > 0) alive = mbar_wait(bar(BAR_QFREE), (un - 1) & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);
                if (!alive) break;
                mbar_expect_tx(bar(BAR_Q), (2 + (un == 0 ? 1 : 0)) * TILE_BYTES + (un == 0 ? P.extra_tx : 0u));
                for (int t = 0; t < 2; ++t) {
                    const int T = 2 * pair + min(t, n_tiles_q - 1), tb = T / P.group, h = kvh * P.group + T % P.group;
                    tma_load_2d(base + SM_Q + t * TILE_BYTES, &map_q, h * TILE, tb * TILE, bar(BAR_Q));
                    tma_load_2d(base + SM_Q + t * TILE_BYTES + HALF_BYTES, &map_q, h * TILE + 64, tb * TILE, bar(BAR_Q));
                }
                if (un == 0) {
                    tma_load_2d(base + SM_K, &map_k, kvh * TILE, U.jb * TILE, bar(BAR_Q));
                    tma_load_2d(base + SM_K + HALF_BYTES, &map_k, kvh * TILE + 64, U.jb * TILE, bar(BAR_Q));
                }
                for (int j = 0; j < U.n_j && alive; ++j, ++gs) {
                    const int st = gs % KV_STAGES, use = gs / KV_STAGES, kst = (gs + 1) % KV_STAGES;
                    int seg, local, n_valid;
                    kv_tile_info(P, U.jb + j, seg, local, n_valid);
                    const CUtensorMap *mv = seg == 0 ? &map_v0 : (seg == 1 ? &map_v1 : &map_v2);
                    if (use > 0) alive = mbar_wait(bar(BAR_VEMPTY + st), (use - 1) & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);
                    else if (gs == 1) alive = mbar_wait(bar(BAR_KEMPTY), 0, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);   // K(2) lands where K(0) was
                    if (!alive) break;
                    const bool in_unit = j + 1 < U.n_j, more = in_unit || g < G1;
                    mbar_expect_tx(bar(BAR_VFULL + st), (more ? 2 : 1) * TILE_BYTES);
                    tma_load_2d(base + SM_V + st * TILE_BYTES, mv, kvh * TILE, local * TILE, bar(BAR_VFULL + st));
                    tma_load_2d(base + SM_V + st * TILE_BYTES + HALF_BYTES, mv, kvh * TILE + 64, local * TILE, bar(BAR_VFULL + st));
                    if (more) {
                        // the next step's keys: the next tile of this item, or the first tile of the next item
                        const int nk = in_unit ? kvh : (U.item + 1) / P.pairs_per_g, nj = in_unit ? U.jb + j + 1 : 0;
                        tma_load_2d(base + SM_K + kst * TILE_BYTES, &map_k, nk * TILE, nj * TILE, bar(BAR_VFULL + st));
                        tma_load_2d(base + SM_K + kst * TILE_BYTES + HALF_BYTES, &map_k, nk * TILE + 64, nj * TILE, bar(BAR_VFULL + st));
                    }
                }
            }
            if (*abort_flag) {
                // give the copies already issued a bounded chance to land before the CTA's shared memory goes away
                const uint64_t t0 = global_ns();
                while (global_ns() - t0 < 2000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        // The warp stays converged (every lane takes the waits) and only the tcgen05 instructions are predicated on
        // one elected lane: issuing a multiply-add then costs about 12 cycles instead of about 60.
        reg_dealloc<72>();
        const bool lead = elect_one();
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
        auto issue_qk = [&](int t, int st) {
            const uint32_t qa = base + SM_Q + t * TILE_BYTES, ka = base + SM_K + st * TILE_BYTES;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                if (lead) mma_ss(tm + t * TILE, desc_kmajor(qa + off), desc_kmajor(ka + off), IDESC_QK, ks > 0);
            }
        };
        bool alive = mbar_wait(bar(BAR_Q), 0, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);
        int gs = 0, un = 0;
        if (alive) {
            tc_fence_after();
            for (int t = 0; t < 2; ++t) {
                issue_qk(t, 0);
                if (lead) tc_commit(bar(BAR_SFULL + t));
            }
            if (lead) tc_commit(bar(BAR_KEMPTY));
            if (unit_at(P, G0, G1).n_j == 1 && lead) tc_commit(bar(BAR_QFREE));      // that was the first unit's only QK^T
        }
        for (long long g = G0; g < G1 && alive; ++un) {
            const Unit U = unit_at(P, g, G1);
            g += U.n_j;
            const int next_n_j = g < G1 ? unit_at(P, g, G1).n_j : 0;
            for (int j = 0; j < U.n_j && alive; ++j, ++gs) {
                const int st = gs % KV_STAGES, use = gs / KV_STAGES, nst = (gs + 1) % KV_STAGES;
                alive = mbar_wait(bar(BAR_VFULL + st), use & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);      // V(step) and K(step + 1)
                const bool in_unit = j + 1 < U.n_j, more = in_unit || next_n_j > 0;
                for (int t = 0; t < 2 && alive; ++t) {
                    const uint32_t va = base + SM_V + st * TILE_BYTES;
                    // P arrives in two halves of 64 keys: the first PV steps run while the rest is exponentiated
                    for (int hf = 0; hf < 2 && alive; ++hf) {
                        alive = mbar_wait(bar(BAR_PHALF + 2 * t + hf), gs & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);
                        if (!alive) break;
                        tc_fence_after();
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {   // 16 keys per step: P columns advance by 8 (two bf16 per column)
                            const int ks = hf * 4 + k4;
                            if (lead)
                                mma_ts(tm + 256 + t * TILE, tm + t * TILE + ks * 8, desc_mnmajor(va + ks * 2048), IDESC_PV, (j > 0 || ks > 0));
                        }
                    }
                    if (!alive) break;
                    if (more) {
                        if (!in_unit && t == 0) {           // the next unit's queries must be in before its first QK^T
                            alive = mbar_wait(bar(BAR_Q), (un + 1) & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);
                            if (!alive) break;
                            tc_fence_after();
                        }
                        issue_qk(t, nst);
                    }
                    if (lead) tc_commit(bar(BAR_SFULL + t));          // S_t of the next step ready, and / or O_t of this unit final
                }
                if (alive && lead) {
                    // the QK^T just issued were the last of their unit: its query tiles may be overwritten
                    if (more && (in_unit ? j + 2 == U.n_j : next_n_j == 1)) tc_commit(bar(BAR_QFREE));
                    tc_commit(bar(BAR_VEMPTY + st));        // PV(step) and QK(step + 1) are behind this: V stage st and K stage nst are free
                }
            }
        }
        // make sure nothing of ours is still running on the tensor core before TMEM is freed
        if (lead) tc_commit(bar(BAR_DONE));
        __syncwarp();
        mbar_wait(bar(BAR_DONE), 0, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us);
    } else if (warp < 4) {
        reg_dealloc<72>();
    } else {
        // ---------------------------------------------------------------- softmax + correction + epilogue
        reg_alloc<208>();
        const int t = (warp - 4) >> 2;
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may touch
        const int r = quad * 32 + lane;                  // row of the tile
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint32_t s_addr = tmem + lane_addr + t * TILE;
        const uint32_t o_addr = tmem + lane_addr + 256 + t * TILE;
        bool alive = true;
        int gs = 0;
        for (long long g = G0; g < G1 && alive;) {
            const Unit U = unit_at(P, g, G1);
            g += U.n_j;
            const int kvh = U.item / P.pairs_per_g, pair = U.item % P.pairs_per_g;
            const int n_tiles_q = min(2, P.tiles_per_g - 2 * pair);
            float m_used = -INFINITY, l = 0.f;
            for (int j = 0; j < U.n_j && alive; ++j, ++gs) {
                int seg, local, n_valid;
                kv_tile_info(P, U.jb + j, seg, local, n_valid);
                alive = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SFULL + t), gs & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us));
                if (!alive) break;
                tc_fence_after();
                // the whole score row of this thread: one TMEM pass
                uint32_t sv[128];
                tmem_ld32(s_addr, sv);
                tmem_ld32(s_addr + 32, sv + 32);
                tmem_ld32(s_addr + 64, sv + 64);
                tmem_ld32(s_addr + 96, sv + 96);
                tmem_wait_ld();
                if (n_valid < TILE) {                        // ragged last tile of a segment: keys past its end score -inf
#pragma unroll
                    for (int i = 0; i < TILE; ++i)
                        if (i >= n_valid) sv[i] = 0xFF800000u;
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < TILE; i += 4) {
                    mx0 = fmaxf(mx0, __uint_as_float(sv[i]));
                    mx1 = fmaxf(mx1, __uint_as_float(sv[i + 1]));
                    mx2 = fmaxf(mx2, __uint_as_float(sv[i + 2]));
                    mx3 = fmaxf(mx3, __uint_as_float(sv[i + 3]));
                }
                const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                // lazy rescale: move the reference maximum only when it grew by more than the threshold
                const bool grow = mx > m_used + RESCALE_THRESHOLD;
                if (__any_sync(0xffffffffu, grow)) {
                    const float m_new = fmaxf(m_used, mx);
                    const float corr = fast_exp2(m_used - m_new);       // 0 on the first tile (m_used = -inf)
                    l *= corr;
                    if (j > 0) {
                        uint32_t v[32];
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            tmem_ld32(o_addr + c * 32, v);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * corr);
                            tmem_st32(o_addr + c * 32, v);
                        }
                    }
                    m_used = m_new;
                }
                // p = 2^(s - m) as bf16 pairs, written over the S columns; the row sum runs on two-lane adds
                const float2 neg_m = make_float2(-m_used, -m_used);
                float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float2 x = add2(make_float2(__uint_as_float(sv[c * 32 + 2 * i]), __uint_as_float(sv[c * 32 + 2 * i + 1])), neg_m);
                        float2 y = add2(make_float2(__uint_as_float(sv[c * 32 + 2 * i + 2]), __uint_as_float(sv[c * 32 + 2 * i + 3])), neg_m);
                        x.x = fast_exp2(x.x); x.y = fast_exp2(x.y);
                        y.x = fast_exp2(y.x); y.y = fast_exp2(y.y);
                        la = add2(la, x);
                        lb = add2(lb, y);
                        pk[i] = pc_pack_bf16(x.x, x.y);
                        pk[i + 1] = pc_pack_bf16(y.x, y.y);
                    }
                    tmem_st16(s_addr + c * 16, pk);
                    if (c & 1) {                               // keys 0-63, then 64-127, handed to the tensor core
                        tmem_wait_st();
                        tc_fence_before();
                        mbar_arrive(bar(BAR_PHALF + 2 * t + (c >> 1)));
                    }
                }
                l += (la.x + la.y) + (lb.x + lb.y);
            }
            // epilogue of the unit: O_t is final once the last PV has committed.  The same commit may also carry the first
            // scores of the next unit; its phase is then waited for a second time at the top of the loop, which returns at once.
            if (alive) alive = __all_sync(0xffffffffu, mbar_wait(bar(BAR_SFULL + t), gs & 1, abort_flag, P.status, PC_WHERE_ATTN_WAIT, P.wait_us));
            if (alive && t < n_tiles_q) {
                tc_fence_after();
                int part, parts;
                item_parts(P, U.item, (int)blockIdx.x, part, parts);
                const int T = 2 * pair + t, tb = T / P.group, h = kvh * P.group + T % P.group;
                const int row = tb * TILE + r;
                // the thread's whole O row leaves TMEM in one pass (four loads in flight, one wait): at a unit boundary the
                // tensor core idles until O is free again, so the read-out is on the critical path
                uint32_t v[128];
                tmem_ld32(o_addr, v);
                tmem_ld32(o_addr + 32, v + 32);
                tmem_ld32(o_addr + 64, v + 64);
                tmem_ld32(o_addr + 96, v + 96);
                tmem_wait_ld();
                if (parts == 1) {
                    const float inv = 1.f / l;
                    __nv_bfloat16 *orow = P.out + ((size_t)row * P.n_q_heads + h) * TILE;
                    if (row < P.n_q) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            uint4 w;
                            w.x = pc_pack_bf16(__uint_as_float(v[8 * i + 0]) * inv, __uint_as_float(v[8 * i + 1]) * inv);
                            w.y = pc_pack_bf16(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv);
                            w.z = pc_pack_bf16(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv);
                            w.w = pc_pack_bf16(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv);
                            *reinterpret_cast<uint4 *>(orow + i * 8) = w;
                        }
                    }
                    if (P.lse && row < P.n_q) P.lse[(size_t)row * P.n_q_heads + h] = (m_used + log2f(l)) * 0.6931471805599453f;
                } else if (P.cluster) {
                    // (split form, one unit per CTA) Stage O (un-normalised, fp32) and (max, sum) in shared memory that no
                    // multiply-add reads any more: tile 0 over both query tiles (every QK^T has completed once this tile's
                    // last PV has), tile 1 over the key stages (its own last PV is the last multiply-add of the CTA).
                    const uint32_t stage = base + (t == 0 ? SM_Q : SM_K);
#pragma unroll
                    for (int i = 0; i < 32; ++i) sts128(stage + stage_off(i, r), v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    *reinterpret_cast<float2 *>(gen + SM_ML + (t * TILE + r) * 8) = make_float2(m_used, l);
                } else {
                    // Partial tile layout: 16-byte unit (c4, r) = columns 4*c4..4*c4+3 of row r at unit c4*128 + r, so the 32 rows
                    // of a warp store 512 contiguous bytes per instruction (a row-major tile would touch 32 lines per store).
                    const size_t tile_slot = ((size_t)U.item * P.part_stride + part) * 2 + t;
                    uint4 *ptile = reinterpret_cast<uint4 *>(P.part_o) + tile_slot * (TILE * TILE / 4) + r;
#pragma unroll
                    for (int i = 0; i < 32; ++i) ptile[i * TILE] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    *reinterpret_cast<float2 *>(P.part_ml + (tile_slot * TILE + r) * 2) = make_float2(m_used, l);
                }
            }
            if (alive && g < G1) {
                // the next unit's first PV overwrites O: every read of it above must have completed (the loads have: each is
                // followed by its wait), and the tensor core must see that before the P of the next step is handed over
                tc_fence_before();
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
    if (P.cluster && P.n_splits > 1) {
        // Merge the KV ranges of this item across the cluster: CTA `rank` finishes every n_splits-th row of the two
        // tiles, reading each peer's staged O and (max, sum) through distributed shared memory.  Sixteen threads share
        // a row (two 16-byte units each), so a row's 256 output bytes leave as two 128-byte runs.
        const int item = (int)blockIdx.x / P.n_splits;
        const int kvh = item / P.pairs_per_g, pair = item % P.pairs_per_g;
        const int n_tiles_q = min(2, P.tiles_per_g - 2 * pair);
        cluster_sync_all();                        // every CTA's staging is complete and visible
        if (warp >= 4) {
            const int S = P.n_splits, my = (int)cluster_rank();
            const int id = threadIdx.x - 128, sub = id & 15, slot = id >> 4;
            uint32_t peer_base[MAX_SPLITS];
#pragma unroll
            for (int k = 0; k < MAX_SPLITS; ++k) peer_base[k] = peer_addr(base, k < S ? k : 0);
            for (int R = my + slot * S; R < 2 * TILE; R += 16 * S) {
                const int t = R >> 7, r = R & (TILE - 1);
                if (t >= n_tiles_q) break;
                const int T = 2 * pair + t, tb = T / P.group, h = kvh * P.group + T % P.group;
                const int row = tb * TILE + r;
                if (row >= P.n_q) continue;
                float mk[MAX_SPLITS], lk[MAX_SPLITS], m = -INFINITY;
#pragma unroll
                for (int k = 0; k < MAX_SPLITS; ++k)
                    if (k < S) {
                        const float2 ml = peer_ld64(peer_base[k] + SM_ML + (t * TILE + r) * 8);
                        mk[k] = ml.x; lk[k] = ml.y;
                        m = fmaxf(m, ml.x);
                    }
                float lsum = 0.f;
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
                const uint32_t stage = (t == 0 ? SM_Q : SM_K);
#pragma unroll
                for (int k = 0; k < MAX_SPLITS; ++k)
                    if (k < S) {
                        const float sc = exp2f(mk[k] - m);
                        lsum = fmaf(lk[k], sc, lsum);
                        const float4 x = peer_ld128(peer_base[k] + stage + stage_off(sub, r));
                        const float4 y = peer_ld128(peer_base[k] + stage + stage_off(sub + 16, r));
                        a.x = fmaf(x.x, sc, a.x); a.y = fmaf(x.y, sc, a.y); a.z = fmaf(x.z, sc, a.z); a.w = fmaf(x.w, sc, a.w);
                        b.x = fmaf(y.x, sc, b.x); b.y = fmaf(y.y, sc, b.y); b.z = fmaf(y.z, sc, b.z); b.w = fmaf(y.w, sc, b.w);
                    }
                const float inv = 1.f / lsum;
                __nv_bfloat16 *orow = P.out + ((size_t)row * P.n_q_heads + h) * TILE;
                *reinterpret_cast<uint2 *>(orow + 4 * sub) = make_uint2(pc_pack_bf16(a.x * inv, a.y * inv), pc_pack_bf16(a.z * inv, a.w * inv));
                *reinterpret_cast<uint2 *>(orow + 64 + 4 * sub) = make_uint2(pc_pack_bf16(b.x * inv, b.y * inv), pc_pack_bf16(b.z * inv, b.w * inv));
                if (P.lse && sub == 0) P.lse[(size_t)row * P.n_q_heads + h] = (m + log2f(lsum)) * 0.6931471805599453f;
            }
        }
        cluster_sync_all();                        // nobody leaves while a peer may still read its shared memory
    }
}

// ------------------------------------------------------------------------------------------------ combine
// Merge of the KV ranges' partials.  One block per (query tile of one head, 32-row quadrant); its eight warps take four
// 16-byte column units each, lanes are consecutive rows, so every load of the partial tiles is a 512-byte run.  Every
// load of a thread is issued before any is used.
__global__ void __launch_bounds__(256) k_combine(const TcParams P) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int lane = threadIdx.x & 31, cg = threadIdx.x >> 5;                   // cg: units 4*cg .. 4*cg+3
    const int quad = blockIdx.x & 3, tile = blockIdx.x >> 2;
    const int h = tile % P.n_q_heads, tb = tile / P.n_q_heads;
    const int g = h / P.group, T = tb * P.group + h % P.group;
    const int item = g * P.pairs_per_g + (T >> 1), t = T & 1;
    const int r = quad * 32 + lane, row = tb * TILE + r;
    if (row >= P.n_q) return;
    int part0, n_parts;
    item_parts(P, item, 0, part0, n_parts);
    if (n_parts < 2) return;                      // the one CTA that had the whole item wrote its output itself
    float2 ml[MAX_SPLITS];
    float4 o[MAX_SPLITS][4];
#pragma unroll
    for (int s = 0; s < MAX_SPLITS; ++s)
        if (s < n_parts) {
            const size_t tile_slot = ((size_t)item * P.part_stride + s) * 2 + t;
            ml[s] = __ldcg(reinterpret_cast<const float2 *>(P.part_ml) + tile_slot * TILE + r);
            const float4 *pt = reinterpret_cast<const float4 *>(P.part_o) + tile_slot * (TILE * TILE / 4) + r;
#pragma unroll
            for (int u = 0; u < 4; ++u) o[s][u] = __ldcg(pt + (cg * 4 + u) * TILE);
        }
    float m = -INFINITY;
#pragma unroll
    for (int s = 0; s < MAX_SPLITS; ++s)
        if (s < n_parts) m = fmaxf(m, ml[s].x);
    float l = 0.f;
    float4 acc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int s = 0; s < MAX_SPLITS; ++s)
        if (s < n_parts) {
            const float sc = exp2f(ml[s].x - m);
            l = fmaf(ml[s].y, sc, l);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc[u].x = fmaf(o[s][u].x, sc, acc[u].x); acc[u].y = fmaf(o[s][u].y, sc, acc[u].y);
                acc[u].z = fmaf(o[s][u].z, sc, acc[u].z); acc[u].w = fmaf(o[s][u].w, sc, acc[u].w);
            }
        }
    const float inv = 1.f / l;
    // this thread's 16 columns of its row: 32 contiguous bytes
    uint4 w0, w1;
    w0.x = pc_pack_bf16(acc[0].x * inv, acc[0].y * inv); w0.y = pc_pack_bf16(acc[0].z * inv, acc[0].w * inv);
    w0.z = pc_pack_bf16(acc[1].x * inv, acc[1].y * inv); w0.w = pc_pack_bf16(acc[1].z * inv, acc[1].w * inv);
    w1.x = pc_pack_bf16(acc[2].x * inv, acc[2].y * inv); w1.y = pc_pack_bf16(acc[2].z * inv, acc[2].w * inv);
    w1.z = pc_pack_bf16(acc[3].x * inv, acc[3].y * inv); w1.w = pc_pack_bf16(acc[3].z * inv, acc[3].w * inv);
    uint4 *orow = reinterpret_cast<uint4 *>(P.out + ((size_t)row * P.n_q_heads + h) * TILE + cg * 16);
    orow[0] = w0;
    orow[1] = w1;
    if (P.lse && cg == 0) P.lse[(size_t)row * P.n_q_heads + h] = (m + log2f(l)) * 0.6931471805599453f;
}

// ------------------------------------------------------------------------------------------------ host side
int div_up(int a, int b) { return (a + b - 1) / b; }

// number of KV ranges: fewest waves of CTAs, a fixed cost per CTA standing in for prologue and epilogue
int choose_splits(int n_items, int n_kv_tiles, int sm_count) {
    int best = 1;
    long best_cost = -1;
    for (int s = 1; s <= MAX_SPLITS && s <= n_kv_tiles; ++s) {
        const long waves = div_up(n_items * s, sm_count);
        const long cost = waves * (div_up(n_kv_tiles, s) + 3) + (s > 1 ? 2 : 0);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

}  // namespace

pc_status pc_attend_tc_scratch(const pc_layer_desc *d, int sm_count, size_t *k_rot_rows, size_t *part_o_floats,
                               size_t *part_ml_floats) {
    (void)sm_count;
    // every segment starts on a tile boundary; the query rows follow the keys in the same scratch
    *k_rot_rows = (size_t)(div_up(d->max_keys, TILE) + PC_MAX_SEGMENTS) * TILE;
    const int group = d->n_q_heads / d->n_kv_heads;
    const int n_items = d->n_kv_heads * div_up(group * div_up(d->max_q, TILE), 2);
    *part_o_floats = (size_t)n_items * MAX_SPLITS * 2 * TILE * TILE;
    *part_ml_floats = (size_t)n_items * MAX_SPLITS * 2 * TILE * 2;
    return PC_OK;
}

// what: PC_TC_ROPE_K rotates the segments' keys into the context scratch, PC_TC_ROPE_Q rotates the queries,
// PC_TC_ATTEND runs attention (and the merge) on the rotated data.
pc_status pc_launch_attend_tc(pc_ctx *ctx, int n_seg, const pc_segment *segs, const void *q, const int32_t *q_pos,
                              int32_t n_q, void *out, float *lse, cudaStream_t stream, int what) {
    const pc_layer_desc &D = ctx->desc;
    if (D.head_dim != TILE || D.dtype != PC_BF16) return PC_ERR_UNSUPPORTED;
    const int row_elems = D.n_kv_heads * D.head_dim;
    __nv_bfloat16 *k_rot = static_cast<__nv_bfloat16 *>(ctx->k_rot);

    TcParams P{};
    RopeJobs jobs{};
    const int k_chunks = row_elems / 8, q_chunks = D.n_q_heads * D.head_dim / 8;
    if (k_chunks % 32 || q_chunks % 32) return PC_ERR_UNSUPPORTED;
    int tiles = 0, warps = 0, n_jobs = 0;
    for (int s = 0; s < n_seg; ++s) {
        if ((what & PC_TC_ROPE_K) || (s == 0 && (what & PC_TC_ROPE_K0))) {
            jobs.job[n_jobs++] = RopeJob{static_cast<const __nv_bfloat16 *>(segs[s].k), segs[s].pos,
                                         k_rot + (size_t)tiles * TILE * row_elems, segs[s].n_tokens, k_chunks, warps, 1, 1.0f};
            warps += segs[s].n_tokens;
        }
        tiles += div_up(segs[s].n_tokens, TILE);
        P.seg_tile_end[s] = tiles;
        P.seg_n[s] = segs[s].n_tokens;
    }
    if ((size_t)tiles * TILE > ctx->k_rot_rows) return PC_ERR_CAPACITY;
    __nv_bfloat16 *q_rot = static_cast<__nv_bfloat16 *>(ctx->q_rot);
    if (what & PC_TC_ROPE_Q) {
        // a query row is as many slices as it holds key-row widths when that divides evenly: every warp then has the same job
        const int slices = (q_chunks % k_chunks == 0) ? q_chunks / k_chunks : 1;
        jobs.job[n_jobs++] = RopeJob{static_cast<const __nv_bfloat16 *>(q), q_pos, q_rot, n_q * slices, q_chunks / slices, warps, slices,
                                     pc_q_rot_scale(D.head_dim)};
        warps += n_q * slices;
    }
    jobs.n_jobs = n_jobs;
    jobs.total_warps = warps;
    ctx->ev_mask &= ~((1u << PC_MARK_ATT0) | (1u << PC_MARK_ROPE) | (1u << PC_MARK_ATTEND) | (1u << PC_MARK_COMBINE));
    pc_mark(ctx, PC_MARK_ATT0, stream);
    if (n_jobs > 0) {
        PC_LAUNCH(k_rope_rows, dim3(div_up(warps, 8)), dim3(256), 0, stream, jobs, ctx->rope, D.head_dim, ctx->status);
        PC_CUDA_TRY(cudaGetLastError());
        pc_mark(ctx, PC_MARK_ROPE, stream);          // no pre-pass (a fused frame step with cached anchors): no mark
    }
    if (!(what & PC_TC_ATTEND)) return PC_OK;

    P.n_q = n_q;
    P.n_q_heads = D.n_q_heads;
    P.group = ctx->group;
    P.n_tb = div_up(n_q, TILE);
    P.tiles_per_g = P.group * P.n_tb;
    P.pairs_per_g = div_up(P.tiles_per_g, 2);
    P.n_kv_tiles = tiles;
    P.n_seg = n_seg;
    const int n_items = D.n_kv_heads * P.pairs_per_g;
    P.n_items = n_items;
    P.out = static_cast<__nv_bfloat16 *>(out);
    P.lse = lse;
    P.part_o = ctx->part_o;
    P.part_ml = ctx->part_ml;
    P.status = ctx->status;
    P.wait_us = ctx->wait_limit_us;
    P.extra_tx = ctx->test_extra_tx;
    // Persistent form unless the caller fixed the number of key ranges or asked for the cluster merge: one CTA per SM, but
    // never so many that an item is cut into more than MAX_SPLITS parts (a CTA's run is at least a third of an item).
    const long long T = (long long)n_items * tiles;
    P.persistent = (ctx->kv_splits == 0 && !ctx->cluster_merge) ? 1 : 0;
    if (P.persistent) {
        P.n_cta = (int)std::min<long long>(std::min<long long>(ctx->sm_count, (long long)n_items * (MAX_SPLITS - 1)), T);
        int most = 1;
        for (int i = 0; i < n_items; ++i) {        // the kernel's own rule (cta_of_step), evaluated for every item
            const long long x0 = (long long)i * tiles, x1 = x0 + tiles - 1;
            const int first = (int)(((x0 + 1) * P.n_cta + T - 1) / T) - 1, last = (int)(((x1 + 1) * P.n_cta + T - 1) / T) - 1;
            most = std::max(most, last - first + 1);
        }
        if (most > MAX_SPLITS) P.persistent = 0;
        P.part_stride = most;
        P.n_splits = most;
    }
    if (!P.persistent) {
        P.n_splits = ctx->kv_splits > 0 ? std::min(ctx->kv_splits, tiles) : choose_splits(n_items, tiles, ctx->sm_count);
        P.n_cta = n_items * P.n_splits;
        P.part_stride = P.n_splits;
    }
    P.cluster = (!P.persistent && P.n_splits > 1 && ctx->cluster_merge) ? 1 : 0;
    if (P.part_stride > 1 && !P.cluster && (size_t)n_items * P.part_stride * 2 * TILE * TILE > ctx->part_o_floats) return PC_ERR_CAPACITY;

    CUtensorMap mq, mk, mv[PC_MAX_SEGMENTS];
    bool ok = make_map(&mq, q_rot, (uint64_t)n_q, (uint64_t)D.n_q_heads * D.head_dim) &&
              make_map(&mk, k_rot, (uint64_t)tiles * TILE, (uint64_t)row_elems);
    for (int s = 0; s < PC_MAX_SEGMENTS; ++s) {
        const pc_segment &sg = segs[s < n_seg ? s : 0];
        ok = ok && make_map(&mv[s], sg.v, (uint64_t)sg.n_tokens, (uint64_t)row_elems);
    }
    if (!ok) {
        fprintf(stderr, "packcache: cuTensorMapEncodeTiled failed\n");
        return PC_ERR_CUDA;
    }
    static bool attr_set[PC_MAX_DEVICES] = {};      // the attribute belongs to the device, not to the process
    if (ctx->device < 0 || ctx->device >= PC_MAX_DEVICES) return PC_ERR_UNSUPPORTED;
    if (!attr_set[ctx->device]) {
        PC_CUDA_TRY(cudaFuncSetAttribute(k_attend_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, SM_ALLOC));
        attr_set[ctx->device] = true;
    }
    if (P.cluster) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(P.n_cta);
        cfg.blockDim = dim3(TC_THREADS);
        cfg.dynamicSmemBytes = SM_ALLOC;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = P.n_splits;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        PC_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_attend_tc, mq, mk, mv[0], mv[1], mv[2], P));
    } else {
        PC_LAUNCH(k_attend_tc, dim3(P.n_cta), dim3(TC_THREADS), SM_ALLOC, stream, mq, mk, mv[0], mv[1], mv[2], P);
    }
    PC_CUDA_TRY(cudaGetLastError());
    pc_mark(ctx, PC_MARK_ATTEND, stream);
    if (P.part_stride > 1 && !P.cluster) {
        PC_LAUNCH(k_combine, dim3(P.n_tb * D.n_q_heads * 4), dim3(256), 0, stream, P);
        PC_CUDA_TRY(cudaGetLastError());
        pc_mark(ctx, PC_MARK_COMBINE, stream);
    }
    ctx->last_n_q = n_q;
    ctx->last_n_seg = n_seg;
    for (int s = 0; s < n_seg; ++s) ctx->last_seg_n[s] = segs[s].n_tokens;
    return PC_OK;
}
