// Stand-alone ordered stream compaction of the route mask (S5): warp ballot + popcount ranks,
// per-warp totals scanned in shared memory.  One block handles up to kCompactOneBlockMax
// sequences; above that, three small launches (tile counts, one-block scan, scatter).
#include "rstitch_kernels.cuh"

namespace rstitch {

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
compact_one_block_kernel(const uint8_t *mask, int B, int32_t *idx, int32_t *count, DevStat *stat)
{
    __shared__ int s_tail[66];
    tail_compact(mask, B, nullptr, nullptr, idx, count, nullptr, nullptr, stat, s_tail);
}

// Tile t covers sequences [t * kCompactTile, (t + 1) * kCompactTile).
__global__ void __launch_bounds__(kThreads)
compact_count_kernel(const uint8_t *mask, int B, int32_t *tile_counts)
{
    __shared__ int s_sum;
    if (threadIdx.x == 0) s_sum = 0;
    __syncthreads();
    const int base = blockIdx.x * kCompactTile;
    int mine = 0;
    for (int i = threadIdx.x; i < kCompactTile; i += kThreads) {
        int b = base + i;
        unsigned ball = __ballot_sync(0xffffffffu, b < B && mask[b] != 0);
        if ((threadIdx.x & 31) == 0) mine += __popc(ball);
    }
    if ((threadIdx.x & 31) == 0) atomicAdd(&s_sum, mine);
    __syncthreads();
    if (threadIdx.x == 0) tile_counts[blockIdx.x] = s_sum;
}

// Exclusive scan of the tile counts in place by one block; also writes the total.
__global__ void __launch_bounds__(kThreads)
compact_scan_kernel(int32_t *tile_counts, int n_tiles, int32_t *count)
{
    __shared__ int s_warp[kThreads / 32];
    __shared__ int s_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < n_tiles; base += kThreads) {
        int i = base + threadIdx.x;
        int v = (i < n_tiles) ? tile_counts[i] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int pre = s_carry;
        for (int w = 0; w < warp; ++w) pre += s_warp[w];
        if (i < n_tiles) tile_counts[i] = pre + incl - v;
        __syncthreads();
        if (threadIdx.x == kThreads - 1) s_carry = pre + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) *count = s_carry;
}

__global__ void __launch_bounds__(kThreads)
compact_scatter_kernel(const uint8_t *mask, int B, const int32_t *tile_offsets, int32_t *idx)
{
    __shared__ int s_warp[kThreads / 32];
    __shared__ int s_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = tile_offsets[blockIdx.x];
    __syncthreads();
    const int base = blockIdx.x * kCompactTile;
    for (int i0 = 0; i0 < kCompactTile; i0 += kThreads) {
        int b = base + i0 + threadIdx.x;
        bool routed = b < B && mask[b] != 0;
        unsigned ball = __ballot_sync(0xffffffffu, routed);
        int rank = __popc(ball & ((1u << lane) - 1u));
        if (lane == 0) s_warp[warp] = __popc(ball);
        __syncthreads();
        int pre = s_carry;
        for (int w = 0; w < warp; ++w) pre += s_warp[w];
        if (routed) idx[pre + rank] = b;
        __syncthreads();
        if (threadIdx.x == 0) {
            int c = 0;
            for (int w = 0; w < kThreads / 32; ++w) c += s_warp[w];
            s_carry += c;
        }
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_compact(const uint8_t *mask, int B, int32_t *idx, int32_t *count, DevStat *stat,
                           int32_t *block_counts, cudaStream_t stream, int *launched)
{
    if (B <= kCompactOneBlockMax || block_counts == nullptr) {
        compact_one_block_kernel<<<1, kThreads, 0, stream>>>(mask, B, idx, count, stat);
        *launched = 1;
        return cudaGetLastError();
    }
    *launched = 3;
    int n_tiles = (B + kCompactTile - 1) / kCompactTile;
    compact_count_kernel<<<n_tiles, kThreads, 0, stream>>>(mask, B, block_counts);
    compact_scan_kernel<<<1, kThreads, 0, stream>>>(block_counts, n_tiles, count);
    compact_scatter_kernel<<<n_tiles, kThreads, 0, stream>>>(mask, B, block_counts, idx);
    return cudaGetLastError();
}

}  // namespace rstitch
