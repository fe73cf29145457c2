// Shared declarations of the PackCache CUDA library (sm_100a).  Nothing here is used by the CPU oracle.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>

#include <cmath>

#include "packcache.h"

#define PC_CUDA_TRY(expr)                                                                     \
    do {                                                                                      \
        cudaError_t _e = (expr);                                                              \
        if (_e != cudaSuccess) {                                                              \
            fprintf(stderr, "packcache: %s failed: %s (%s:%d)\n", #expr, cudaGetErrorString(_e), \
                    __FILE__, __LINE__);                                                      \
            return PC_ERR_CUDA;                                                               \
        }                                                                                     \
    } while (0)

// "where" codes stored beside a device-side status (second status word)
enum {
    PC_WHERE_SCORE_POS = 1,
    PC_WHERE_QPOOL_POS = 2,
    PC_WHERE_SELECT_NAN = 3,
    PC_WHERE_PACK_INDEX = 4,
    PC_WHERE_ATTN_POS = 5,
    PC_WHERE_ATTN_WAIT = 6,
    PC_WHERE_ROPE_POS = 7,
    PC_WHERE_SCORE_WAIT = 8,
    PC_WHERE_MASK_COUNT = 9,
    PC_WHERE_MASS_WAIT = 10,
};

constexpr int PC_MAX_SEGMENTS = 3;
constexpr int PC_FX_REPLICAS = 8;             // copies of the pooled-query accumulator (see pc_score.cu)
constexpr int PC_MAX_DEVICES = 64;            // per-device launch state is kept in arrays of this size

// Rotary tables: for axis a (t, h, w) a [max_pos[a]][n_axis[a]] array of (cos, sin) of pos * base^(-m/n_axis[a]).
// Pair i of a head uses axis i % 3 and column m = i / 3.
struct pc_rope_dev {
    const float2 *tab;   // device, the three tables back to back
    int32_t off[3];      // offset (in float2) of each axis table
    int32_t n_axis[3];   // pairs per axis
    int32_t max_pos[3];
};

struct pc_ctx {
    pc_layer_desc desc;
    int device;
    int sm_count;
    int group;                 // Hq / Hkv
    int elem_size;             // bytes per element
    int attend_impl;           // 0 tensor-core (bf16), 1 CUDA-core
    pc_rope_dev rope;
    float2 *rope_tab;          // owned
    int32_t *status;           // device [2]: code, where
    int32_t *host_status;      // pinned [2]
    // Pooled query of the scoring pass as fixed-point sums (units of 2^-32): PC_FX_REPLICAS copies of Hkv*d 64-bit
    // integers (the blocks of the query pass spread over the copies; integer addition: the result does not depend on the
    // order of the blocks) and one ticket word.  The last block of the query pass adds the copies into `qpool` (fp32) and
    // clears the accumulator, so it is zero between calls.
    long long *qpool_fx;       // device [PC_FX_REPLICAS * Hkv*d + 1]
    float *qpool;              // device [Hkv*d]
    int qpool_dirty;           // 1: a call failed between the two kernels; the array is cleared before the next use
    // attention scratch (tensor-core path)
    void *k_rot;               // rotated keys, bf16 [rows][Hkv][d]
    size_t k_rot_rows;
    void *q_rot;               // rotated, pre-scaled queries, bf16 [max_q][Hq][d]
    int kv_splits;             // 0 = chosen per call
    int cluster_merge;         // 1 = KV ranges merge inside the kernel through cluster shared memory (default 0)
    uint32_t wait_limit_us;    // limit of every bounded device-side wait in microseconds; 0 = about one second
    uint32_t test_extra_tx;    // test hook: bytes the attention kernel's first barrier expects beyond what is sent (0 = off)
    // rotated anchor keys kept in k_rot across fused frame steps (anchors never move): the segment they were made from
    const void *anchor_rot_k;
    const int32_t *anchor_rot_pos;
    int anchor_rot_n;          // 0 = none cached
    int q_rot_n;               // rows of q_rot written by the query pass of the running fused step (0 = none)
    // key set fixed by pc_attend_prepare (its rotated keys sit in k_rot until the next prepare or pc_attend_frame)
    int prepared_n_seg;        // 0 = nothing prepared
    pc_segment prepared_seg[PC_MAX_SEGMENTS];
    // shape of the most recent tensor-core attention call, whose rotated keys and queries are still in k_rot / q_rot
    // (read by pc_attend_mass); last_n_q = 0 when there is none
    int last_n_q, last_n_seg;
    int last_seg_n[PC_MAX_SEGMENTS];
    float *mass_part;          // attention mass: partial sums per KV head and column half, [Hkv][2][k_rot_rows]
    float *mass_norm;          // attention mass: negated base-2 normalisers, [Hq][max_q rounded up to 128]
    // optional per-kernel timing (benchmarks): events at the boundaries of the kernels of each call
    int timing_on;
    unsigned ev_mask;
    unsigned ev_skip;          // marks that are not recorded (see pc_set_timing_skip)
    cudaEvent_t ev[PC_N_MARKS];
    float *part_o;             // split-KV partial outputs
    float *part_ml;            // split-KV partial (max, sum)
    size_t part_o_floats, part_ml_floats;
};

__device__ __forceinline__ void pc_flag(int32_t *status, int code, int where) {
    if (atomicCAS(status, 0, code) == 0) status[1] = where;
}

// (cos, sin) for pair i of a head at position p[0..2]; flags and clamps a position outside the table.
__device__ __forceinline__ float2 pc_rope_cs(const pc_rope_dev &r, int pair, int pt, int ph, int pw, int32_t *status,
                                             int where) {
    const int a = pair % 3, m = pair / 3;
    // the axis picks its coordinate and table by selects on fixed fields (no indexed access to the parameter block)
    int pa = a == 0 ? pt : (a == 1 ? ph : pw);
    const int mx = a == 0 ? r.max_pos[0] : (a == 1 ? r.max_pos[1] : r.max_pos[2]);
    const int off = a == 0 ? r.off[0] : (a == 1 ? r.off[1] : r.off[2]);
    const int na = a == 0 ? r.n_axis[0] : (a == 1 ? r.n_axis[1] : r.n_axis[2]);
    if (pa < 0 || pa >= mx) {
        pc_flag(status, PC_ERR_INVALID_ARG, where);
        pa = pa < 0 ? 0 : mx - 1;
    }
    return __ldg(r.tab + off + (size_t)pa * na + m);
}

// One rotary pair turned by (cos, sin), with the roundings spelt out: every kernel that rotates (query pass, key
// pre-pass, pack with rotation) produces the same bits for the same inputs.
__device__ __forceinline__ float2 pc_rotate(float x0, float x1, float2 cs) {
    return make_float2(__fmaf_rn(x0, cs.x, -__fmul_rn(x1, cs.y)), __fmaf_rn(x0, cs.y, __fmul_rn(x1, cs.x)));
}

__device__ __forceinline__ float pc_bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float pc_bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pc_pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ uint4 pc_ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void pc_stg_stream(void *p, uint4 v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

// ---- mbarrier / bulk-copy helpers (shared::cta addresses as 32-bit integers)
__device__ __forceinline__ uint32_t pc_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void pc_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void pc_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void pc_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool pc_mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t pc_global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait on an mbarrier phase, the one wait routine of every kernel of the library: gives up after limit_us
// microseconds (0 = the default of about one second), or at once when another thread of the CTA already gave up
// (abort_flag), records PC_ERR_TIMEOUT with `where` in the status word, and returns false.  The caller then skips the
// work that depended on the wait, drains what it has in flight and leaves: no trap, no unbounded spin.
__device__ __forceinline__ bool pc_mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status, int where,
                                             uint32_t limit_us = 0) {
    for (int i = 0; i < 2048; ++i)
        if (pc_mbar_try(bar, parity)) return true;
    const uint64_t t0 = pc_global_ns();
    const uint64_t limit_ns = limit_us ? (uint64_t)limit_us * 1000ull : 1000000000ull;
    for (;;) {
        if (pc_mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (pc_global_ns() - t0 > limit_ns) {
            *abort_flag = 1;
            pc_flag(status, PC_ERR_TIMEOUT, where);
            return false;
        }
    }
}
// global -> shared bulk copy (both 16-byte aligned, size a multiple of 16), completion counted on an mbarrier
__device__ __forceinline__ void pc_bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 pc_lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// d += a * b on two fp32 lanes with one instruction
__device__ __forceinline__ void pc_fma2(float2 &d, float2 a, float2 b) {
    asm("{\n\t.reg .b64 ra, rb, rc;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%0, %1};\n\t"
        "fma.rn.f32x2 rc, ra, rb, rc;\n\tmov.b64 {%0, %1}, rc;\n\t}"
        : "+f"(d.x), "+f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
}

// ---- programmatic dependent launch
// Every kernel of the library is launched with programmatic stream serialisation: it may start while the kernel before
// it in the stream is still draining.  A kernel lets its own dependents go at its very start (pc_grid_dep_launch) and
// must not touch global memory before pc_grid_dep_wait, which returns once the preceding kernel has completed and its
// writes are visible; only set-up that needs no global data (barrier initialisation, TMEM allocation) goes before it.
__device__ __forceinline__ void pc_grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pc_grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t pc_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// launch + error check in one statement (returns PC_ERR_CUDA from the calling function on failure)
#define PC_LAUNCH(kernel, grid, block, smem, stream, ...) PC_CUDA_TRY(pc_launch(kernel, grid, block, smem, stream, __VA_ARGS__))

inline void pc_mark(pc_ctx *c, int idx, cudaStream_t s) {
    if ((c->ev_skip >> idx) & 1u) {
        c->ev_mask &= ~(1u << idx);
        return;
    }
    if (c->timing_on && c->ev[idx] && cudaEventRecord(c->ev[idx], s) == cudaSuccess) c->ev_mask |= 1u << idx;
}

// Shapes the tensor-core kernels take: bf16, head_dim 128, and K / Q rows that are whole 256-element granules of the
// rotary pre-pass (a warp rotates 32 x 8 elements at a time).  Everything else runs on the CUDA-core kernel.
inline bool pc_tensor_core_shape(const pc_ctx *ctx) {
    const pc_layer_desc &d = ctx->desc;
    return d.dtype == PC_BF16 && d.head_dim == 128 && (d.n_kv_heads * d.head_dim) % 256 == 0 && (d.n_q_heads * d.head_dim) % 256 == 0;
}

// host-side helpers implemented in pc_api.cu
bool pc_aligned16(const void *p);
pc_status pc_check_segment(const pc_segment *s, bool allow_empty);

// stage launchers (each validates nothing: the pc_* entry points did)
// k_rot_dst: where the rotated copy of each packed K row goes as well (bf16 tensor-core shapes), or NULL
pc_status pc_launch_pack(pc_ctx *ctx, const void *src_k, const void *src_v, const int32_t *src_pos, const int32_t *sel_idx,
                         int n_sel, int n_src, int delta_t, void *dst_k, void *dst_v, int32_t *dst_pos, void *k_rot_dst,
                         cudaStream_t stream);
// pc_score / pc_compact with the extras of the fused frame step: q_rot_out (NULL or the context's rotated-query scratch,
// filled by the query pass that also pools), k_rot_dst (as pc_launch_pack)
bool pc_score_supports(const pc_layer_desc &D);   // the row widths the query pass and the scoring kernel take
pc_status pc_score_impl(pc_ctx *ctx, const pc_cache *src, const void *q, const int32_t *q_pos, int32_t n_q, const int32_t *budget,
                        const uint8_t *valid, const float *scores_override, float *scores, int32_t *sel_idx, void *q_rot_out,
                        cudaStream_t stream);
pc_status pc_compact_check(pc_ctx *ctx, const pc_cache *src, const int32_t *sel_idx, const int32_t *budget, const pc_cache *dst,
                           int64_t *n_sel_out, int64_t *n_src_out);   // every host-side check of pc_compact_impl, nothing enqueued
pc_status pc_compact_impl(pc_ctx *ctx, const pc_cache *src, const int32_t *sel_idx, const int32_t *budget, int32_t delta_t,
                          pc_cache *dst, void *k_rot_dst, cudaStream_t stream);
// log2(e) / sqrt(d): folded into the rotated queries of the tensor-core attention kernel (its softmax runs in base 2)
inline float pc_q_rot_scale(int head_dim) { return (float)(1.4426950408889634 / std::sqrt((double)head_dim)); }
pc_status pc_launch_attend_simt(pc_ctx *ctx, int n_seg, const pc_segment *segs, const void *q, const int32_t *q_pos,
                                int32_t n_q, void *out, float *lse, cudaStream_t stream);
// PC_TC_ROPE_K0: rotate the keys of the first segment only (the anchors of a fused frame step)
enum { PC_TC_ROPE_K = 1, PC_TC_ROPE_Q = 2, PC_TC_ATTEND = 4, PC_TC_ALL = 7, PC_TC_ROPE_K0 = 8 };
pc_status pc_launch_attend_tc(pc_ctx *ctx, int n_seg, const pc_segment *segs, const void *q, const int32_t *q_pos,
                              int32_t n_q, void *out, float *lse, cudaStream_t stream, int what);
pc_status pc_attend_tc_scratch(const pc_layer_desc *d, int sm_count, size_t *k_rot_rows, size_t *part_o_floats,
                               size_t *part_ml_floats);
