// Cross-block finalisation of the head kernels as a launch of its own (S2-S6): one warp per row merges
// the row's per-slice statistics in a fixed order and writes entropy and token; the last block to
// finish applies the rule of Eq. 2, compacts and (optionally) carries Algorithm 1 on.
//
// The kernel is launched with programmatic stream serialisation behind the head kernel, and so is the
// next call's head kernel behind this one.  A head kernel streams W_head -- a weight, which no kernel
// of this library writes -- from its first instruction and only waits for the kernels before it when
// it first needs something they may have written (hidden rows, index lists, the scratch).  Back to back,
// step i + 1 therefore streams while step i's statistics are merged here on two or three SMs, and the
// other SMs do not idle through the merge, the drain of the grid and the next launch.
#include "rstitch_kernels.cuh"
#include "rstitch_ptx.cuh"

namespace rstitch {

namespace {

constexpr int kFinThreads = 128;
constexpr int kFinRows    = kFinThreads / 32;        // one warp per row
constexpr int kFinStageSeqs = 128;                   // mask bytes the deciding block keeps in shared memory

__global__ void __launch_bounds__(kFinThreads)
head_finalize_kernel(Partials P, int n_slices, int R, const int32_t *n_rows_dev, TailArgs t, unsigned *ticket)
{
    __shared__ int s_tail[66];
    __shared__ int s_last;
    // Shared memory is kept to a few hundred bytes on purpose: the head kernels leave about 1.5 KB of an
    // SM free, and with 1 KB of staging arrays here a step at 64 rows measured 5 us longer.
    __shared__ float s_ent[kFinRows];                // one block only: its rows' entropies stay on the SM
    __shared__ uint8_t s_mask[kFinStageSeqs];        // the mask, for the compaction
    ptx::grid_dep_launch_dependents();
    ptx::grid_dep_wait();                            // the head kernel has completed: its partials are visible
    int R_live = R;
    if (n_rows_dev) { int n = *n_rows_dev; R_live = n < 0 ? 0 : (n < R ? n : R); }
    const int lane = threadIdx.x & 31;
    for (int r = blockIdx.x * kFinRows + (threadIdx.x >> 5); r < R_live; r += gridDim.x * kFinRows) {
        // 256 slices at a time: one round trip to L2 per chunk with every load in flight, chunks merged in
        // ascending order (the many-row kernel leaves one partial per 256-row vocabulary tile: 594 of them)
        Stats st = tail_row_direct(P, (size_t)r * n_slices, n_slices < 256 ? n_slices : 256, lane);
        for (int c0 = 256; c0 < n_slices; c0 += 256) {
            const Stats more = tail_row_direct(P, (size_t)r * n_slices + c0, n_slices - c0 < 256 ? n_slices - c0 : 256, lane);
            stats_merge(st, more);
        }
        if (lane == 0) {
            const float H = tail_emit_row(st, r, t);
            if (r < kFinRows) s_ent[r] = H;
        }
    }
    if (gridDim.x > 1) {
        __syncthreads();             // the block's rows are written ...
        if (threadIdx.x == 0) s_last = (ptx::ticket_take(ticket) == gridDim.x - 1);   // ... and released with its ticket
        __syncthreads();
        if (!s_last) return;         // the last ticket has acquired every other block's rows
    } else {
        __syncthreads();
    }
    TailArgs ta = t;
    ta.R = R_live;
    if (n_rows_dev) ta.B = R_live < t.B ? R_live : t.B;
    // what this block can keep on the SM it does not read back from global memory: the entropies when
    // it merged every row itself, the mask whenever it fits
    tail_route(ta, s_tail, (gridDim.x == 1 && ta.R <= kFinRows) ? s_ent : nullptr,
               ta.B <= kFinStageSeqs ? s_mask : nullptr);
    if (gridDim.x > 1 && threadIdx.x == 0) *ticket = 0u;
}

}  // namespace

cudaError_t launch_dependent(const void *func, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, void **args)
{
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
    return cudaLaunchKernelExC(&cfg, func, args);
}

cudaError_t launch_head_finalize(const Partials &P, int n_slices, int R, const int32_t *n_rows_dev,
                                 const TailArgs &t, unsigned *ticket, int sm_count, cudaStream_t stream)
{
    int grid = (R + kFinRows - 1) / kFinRows;
    if (grid > sm_count) grid = sm_count;
    if (grid < 1) grid = 1;
    Partials p = P;
    TailArgs ta = t;
    void *args[] = {&p, &n_slices, &R, &n_rows_dev, &ta, &ticket};
    return launch_dependent((const void *)head_finalize_kernel, dim3((unsigned)grid), dim3(kFinThreads), 0, stream, args);
}

}  // namespace rstitch
