// Measurement support: the issue stream of the attention kernel's tensor-core multiply-adds with nothing else going on, as a
// yardstick for that kernel: how many SM cycles one tcgen05.mma (128 x 128 x 16, bf16, fp32 accumulate) takes back to back,
// and what the SM clock is meanwhile (cycles against the global timer).
#include "pc_tc.cuh"

namespace {

using namespace pc_tc;

constexpr int PROBE_SM_BAR = 6 * TILE_BYTES;                    // two query tiles, two K stages, two V stages, as in the attention kernel
constexpr int PROBE_SM_ALLOC = PROBE_SM_BAR + 256 + 1024;       // barriers etc. + slack for manual alignment

// One CTA per SM (the shared memory sees to that), one issuing warp.  A round is what the attention kernel issues per key
// tile for both query tiles: form 0 only the QK^T multiply-adds (A and B in shared memory; 16 per round), form 1 only the
// PV multiply-adds (A in tensor memory; 16 per round), form 2 both in the kernel's order (32 per round).  Two rounds are in
// flight: round i is issued once round i - 2 has completed.  Operands are pseudo-random bf16; the results are not used.
__global__ void __launch_bounds__(128, 1) k_mma_rate(int form, int rounds, long long *cycles, long long *nanos, uint32_t wait_us,
                                                      int32_t *status) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + PROBE_SM_BAR + 64);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(gen + PROBE_SM_BAR + 72);
    const uint32_t bar0 = base + PROBE_SM_BAR;
    const int warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 6 * TILE_BYTES / 4; i += 128) {          // bf16 pairs with magnitudes in [0.5, 1) and random signs
        uint32_t h = ((uint32_t)i * 2654435761u) ^ (blockIdx.x * 40503u);
        h ^= h >> 13; h *= 0x5bd1e995u; h ^= h >> 15;
        reinterpret_cast<uint32_t *>(gen)[i] = (0x3F00u | (h & 0x807Fu)) | ((0x3F00u | ((h >> 16) & 0x807Fu)) << 16);
    }
    if (threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        mbar_init(bar0 + 16, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");           // the fill above is read by the tensor core
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = *tmem_slot;
    if (warp == 1) {
        const bool lead = elect_one();
        const uint32_t q0 = base, k0 = base + 2 * TILE_BYTES, v0 = base + 4 * TILE_BYTES;
        bool alive = true;
        const uint64_t n0 = global_ns();
        const long long c0 = clock64();
        for (int it = 0; it < rounds && alive; ++it) {
            if (it >= 2) alive = mbar_wait(bar0 + 8 * (it & 1), ((it - 2) >> 1) & 1, abort_flag, status, PC_WHERE_ATTN_WAIT, wait_us);
            if (!alive) break;
            for (int t = 0; t < 2; ++t) {
                if (form != 0) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        if (lead) mma_ts(tm + 256 + t * TILE, tm + t * TILE + ks * 8, desc_mnmajor(v0 + (it & 1) * TILE_BYTES + ks * 2048), IDESC_PV, 1);
                }
                if (form != 1) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                        if (lead) mma_ss(tm + t * TILE, desc_kmajor(q0 + t * TILE_BYTES + off), desc_kmajor(k0 + (it & 1) * TILE_BYTES + off), IDESC_QK, ks > 0);
                    }
                }
            }
            if (lead) tc_commit(bar0 + 8 * (it & 1));
        }
        if (lead) tc_commit(bar0 + 16);                 // everything issued has completed once this phase does
        __syncwarp();
        mbar_wait(bar0 + 16, 0, abort_flag, status, PC_WHERE_ATTN_WAIT, wait_us);
        const long long c1 = clock64();
        const uint64_t n1 = global_ns();
        if (lead) {
            cycles[blockIdx.x] = c1 - c0;
            nanos[blockIdx.x] = (long long)(n1 - n0);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tm) : "memory");
    }
}

}  // namespace

extern "C" pc_status pc_probe_mma_rate(pc_ctx *ctx, int32_t form, int32_t rounds, int32_t n_cta, int64_t *cycles, int64_t *nanos,
                                       void *stream_) {
    if (!ctx || !cycles || !nanos || form < 0 || form > 2 || rounds < 1 || rounds > (1 << 20) || n_cta < 1 || n_cta > 4096)
        return PC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(cycles) & 7u) || (reinterpret_cast<uintptr_t>(nanos) & 7u)) return PC_ERR_INVALID_ARG;
    static bool attr_set[PC_MAX_DEVICES] = {};
    if (ctx->device < 0 || ctx->device >= PC_MAX_DEVICES) return PC_ERR_UNSUPPORTED;
    if (!attr_set[ctx->device]) {
        PC_CUDA_TRY(cudaFuncSetAttribute(k_mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, PROBE_SM_ALLOC));
        attr_set[ctx->device] = true;
    }
    PC_LAUNCH(k_mma_rate, dim3(n_cta), dim3(128), PROBE_SM_ALLOC, static_cast<cudaStream_t>(stream_), (int)form, (int)rounds,
              reinterpret_cast<long long *>(cycles), reinterpret_cast<long long *>(nanos), ctx->wait_limit_us, ctx->status);
    PC_CUDA_TRY(cudaGetLastError());
    return PC_OK;
}
