// Per-frame top-k selection as a block-level routine (used by the selection kernel and by the kernel that selects and
// packs in one launch).  Scores map to 32-bit keys whose unsigned order is the score order (-0 folded onto +0).  An
// 8-bit-digit radix descent finds the key T of the budget-th best token and how many keys beat it; a final ordered sweep
// keeps every key > T and the lowest-index (budget - beaten) keys == T, handing each kept token and its rank among the
// frame's kept tokens (ascending index order) to the caller.
#pragma once
#include "pc_common.cuh"

struct FrameTab { int4 f[PC_MAX_FRAMES]; };   // (first token, tokens, budget, output offset)

__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    if ((u << 1) == 0) u = 0;                       // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int SEL_CACHE = 4096;   // keys of a frame kept in shared memory; longer frames re-read the rest from global

template <int THREADS> struct SelectShared {
    uint32_t keys[SEL_CACHE];
    int hist[256];
    int warp_sums[THREADS / 32];
    uint32_t prefix;
    int want;
};

// Exclusive block scan of a small per-thread value; total = sum over the block.
template <int THREADS>
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
    for (int i = 0; i < THREADS / 32; ++i) {
        int s = warp_sums[i];
        if (i < w) base += s;
        tot += s;
    }
    total = tot;
    return base + inc - v;
}

// The whole block selects frame `fr` (budget > 0, n > 0); keep(rank, global index) is called once per kept token by the
// thread that owns it.  Every thread of the block must call this.
template <int THREADS, typename Keep>
__device__ __forceinline__ void frame_select(const float *__restrict__ scores, int4 fr, SelectShared<THREADS> &sm,
                                             int32_t *status, Keep keep) {
    const int first = fr.x, n = fr.y, budget = fr.z;
    const float *s = scores + first;
    const int lane = threadIdx.x & 31;

    for (int j = threadIdx.x; j < n; j += THREADS) {
        const float v = s[j];
        if (v != v) pc_flag(status, PC_ERR_INVALID_ARG, PC_WHERE_SELECT_NAN);
        if (j < SEL_CACHE) sm.keys[j] = score_key(v);
    }
    for (int i = threadIdx.x; i < 256; i += THREADS) sm.hist[i] = 0;
    __syncthreads();
    auto key_at = [&](int j) { return j < SEL_CACHE ? sm.keys[j] : score_key(s[j]); };

    uint32_t prefix = 0, mask = 0;
    int want = budget;                               // rank, among keys matching the prefix, of the threshold key
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int j = threadIdx.x; j < n; j += THREADS) {
            const uint32_t key = key_at(j);
            if ((key & mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // lane l owns digits 255 - 8l down to 248 - 8l; an inclusive scan over lanes counts keys from the top digit down
            int c[8], mine = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = sm.hist[255 - 8 * lane - i]; mine += c[i]; }
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
                sm.prefix = prefix | ((uint32_t)digit << shift);
                sm.want = w;
            }
        }
        __syncthreads();
        prefix = sm.prefix;
        want = sm.want;
        mask |= 255u << shift;
        for (int i = threadIdx.x; i < 256; i += THREADS) sm.hist[i] = 0;
        __syncthreads();
    }
    // prefix is now the threshold key T: every key above it is kept, and the `want` lowest-index keys equal to it.
    // One scan per THREADS keys carries both counts (keys above T in the low half, keys equal to T in the high half).
    const uint32_t T = prefix;
    int gt_seen = 0, eq_seen = 0;
    for (int j0 = 0; j0 < n; j0 += THREADS) {
        const int j = j0 + threadIdx.x;
        const bool in = j < n;
        const uint32_t key = in ? key_at(j) : 0u;
        const int is_gt = in && key > T, is_eq = in && key == T;
        int total;
        const int ex = block_exclusive_scan<THREADS>(is_gt | (is_eq << 16), sm.warp_sums, total);
        const int gt_before = gt_seen + (ex & 0xFFFF), eq_before = eq_seen + (ex >> 16);
        if (is_gt || (is_eq && eq_before < want)) {
            const int at = gt_before + min(eq_before, want);
            if (at < budget) keep(at, first + j);
        }
        gt_seen += total & 0xFFFF;
        eq_seen += total >> 16;
    }
}
