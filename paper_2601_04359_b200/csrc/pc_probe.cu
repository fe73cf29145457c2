// Measurement support: a kernel that does nothing but stream rows from HBM, as a yardstick for the HBM-bound kernels.
#include <algorithm>

#include "pc_common.cuh"

namespace {

// One warp takes two rows of `row_bytes` (a multiple of 512) at a time: every lane loads its 16-byte chunks of both rows
// with streaming loads, all in flight before the first is used, xors them and one lane stores four bytes per row: the
// memory traffic of the scoring kernel without its arithmetic.  Persistent grid, rows dealt round-robin to the warps.
__global__ void __launch_bounds__(256) k_stream_read(const uint4 *__restrict__ src, int n_rows, int chunks_per_lane,
                                                     uint32_t *__restrict__ out) {
    pc_grid_dep_launch();
    pc_grid_dep_wait();
    const int lane = threadIdx.x & 31, gw = (blockIdx.x * 256 + threadIdx.x) >> 5, n_warps = gridDim.x * 8;
    const int n_pairs = (n_rows + 1) >> 1;
    const size_t row = (size_t)chunks_per_lane * 32;
    for (int tp = gw; tp < n_pairs; tp += n_warps) {
        const int j0 = 2 * tp, j1 = min(j0 + 1, n_rows - 1);
        uint32_t x0 = 0, x1 = 0;
        if (chunks_per_lane == 4) {
            uint4 a[4], b[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) a[c] = pc_ldg_stream(src + (size_t)j0 * row + c * 32 + lane);
#pragma unroll
            for (int c = 0; c < 4; ++c) b[c] = pc_ldg_stream(src + (size_t)j1 * row + c * 32 + lane);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                x0 ^= a[c].x ^ a[c].y ^ a[c].z ^ a[c].w;
                x1 ^= b[c].x ^ b[c].y ^ b[c].z ^ b[c].w;
            }
        } else {
            for (int c = 0; c < chunks_per_lane; ++c) {
                const uint4 a = pc_ldg_stream(src + (size_t)j0 * row + c * 32 + lane), b = pc_ldg_stream(src + (size_t)j1 * row + c * 32 + lane);
                x0 ^= a.x ^ a.y ^ a.z ^ a.w;
                x1 ^= b.x ^ b.y ^ b.z ^ b.w;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            x0 ^= __shfl_xor_sync(0xffffffffu, x0, o);
            x1 ^= __shfl_xor_sync(0xffffffffu, x1, o);
        }
        if (lane == 0) {
            out[j0] = x0;
            if (j1 != j0) out[j1] = x1;
        }
    }
}

}  // namespace

extern "C" pc_status pc_probe_stream_read(const void *src, int32_t n_rows, int32_t row_bytes, uint32_t *out, void *stream_) {
    if (!src || !out || n_rows <= 0 || row_bytes <= 0 || row_bytes % 512) return PC_ERR_INVALID_ARG;
    if (!pc_aligned16(src) || (reinterpret_cast<uintptr_t>(out) & 3u)) return PC_ERR_INVALID_ARG;
    int dev = 0, sm_count = 0;
    PC_CUDA_TRY(cudaGetDevice(&dev));
    PC_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    const int n_pairs = (n_rows + 1) / 2;
    const int blocks = std::max(1, std::min((n_pairs + 7) / 8, sm_count * 4));
    PC_LAUNCH(k_stream_read, dim3(blocks), dim3(256), 0, static_cast<cudaStream_t>(stream_), static_cast<const uint4 *>(src),
              (int)n_rows, (int)(row_bytes / 512), out);
    PC_CUDA_TRY(cudaGetLastError());
    return PC_OK;
}
