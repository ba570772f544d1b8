// Measurement aid, not part of the routing path: how fast this GPU streams memory that is only read.
//
// The head kernels read W_head once and write almost nothing, so the bandwidth of a copy (half reads,
// half writes) understates their ceiling.  This kernel moves a buffer through the same pipeline the
// streaming head kernel uses -- one block per SM, one thread issuing bulk copies of a contiguous slice
// into a shared-memory ring, completion on mbarriers -- and does nothing with the bytes.  Timed with
// CUDA events by the benchmark, it gives the read-only ceiling beside the copy figure.
#include "../../include/rstitch.h"
#include "rstitch_ptx.cuh"

namespace rstitch {
namespace {

constexpr int      kProbeSlots = 12;
constexpr uint32_t kProbeChunk = 16 * 1024;
constexpr int      kProbeSmem  = kProbeSlots * (int)kProbeChunk;

__global__ void __launch_bounds__(64, 1)
read_stream_kernel(const unsigned char *src, unsigned long long n_chunks, unsigned *gave_up)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) uint64_t s_full[kProbeSlots], s_empty[kProbeSlots];
    __shared__ int s_abort, s_zero;
    const unsigned long long c0 = n_chunks * blockIdx.x / gridDim.x, c1 = n_chunks * (blockIdx.x + 1) / gridDim.x;
    if (threadIdx.x == 0) {
        s_abort = 0; s_zero = 0;
        for (int s = 0; s < kProbeSlots; ++s) {
            ptx::mbar_init(ptx::smem_u32(&s_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&s_empty[s]), 1);
        }
        ptx::mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {                          // producer
        int slot = 0, round = 0;
        unsigned long long issued = 0;
        for (unsigned long long c = c0; c < c1; ++c) {
            if (!ptx::mbar_wait(ptx::smem_u32(&s_empty[slot]), (uint32_t)((round & 1) ^ 1), &s_abort)) {
                s_abort = 1;
                atomicAdd(gave_up, 1u);
                break;
            }
            const uint32_t full = ptx::smem_u32(&s_full[slot]);
            ptx::mbar_arrive_expect_tx(full, kProbeChunk);
            ptx::bulk_g2s(ptx::smem_u32(ring) + (uint32_t)slot * kProbeChunk, src + c * kProbeChunk, kProbeChunk, full);
            ++issued;
            if (++slot == kProbeSlots) { slot = 0; ++round; }
        }
        if (s_abort) {                               // no copy may still be landing when the block exits
            unsigned long long first = issued > kProbeSlots ? issued - kProbeSlots : 0;
            for (unsigned long long j = first; j < issued; ++j)
                ptx::mbar_wait(ptx::smem_u32(&s_full[j % kProbeSlots]), (uint32_t)((j / kProbeSlots) & 1), &s_zero);
        }
    } else if (threadIdx.x == 32) {                  // consumer: frees each slot as soon as it has landed
        int slot = 0, round = 0;
        for (unsigned long long c = c0; c < c1; ++c) {
            if (!ptx::mbar_wait(ptx::smem_u32(&s_full[slot]), (uint32_t)(round & 1), &s_abort)) {
                if (!s_abort) { s_abort = 1; atomicAdd(gave_up, 1u); }
                break;
            }
            ptx::mbar_arrive(ptx::smem_u32(&s_empty[slot]));
            if (++slot == kProbeSlots) { slot = 0; ++round; }
        }
    }
}

}  // namespace
}  // namespace rstitch

extern "C" int rstitch_probe_read_stream(const void *buf, size_t bytes, uint32_t *gave_up, void *cuda_stream)
{
    using namespace rstitch;
    if (!gave_up) return RSTITCH_ERR_INVALID_ARG;
    const unsigned long long n_chunks = bytes / kProbeChunk;
    if (n_chunks == 0) return RSTITCH_OK;                 // less than one chunk: nothing is read
    if (!buf || (reinterpret_cast<uintptr_t>(buf) % 16) != 0) return RSTITCH_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1 ||
        cudaFuncSetAttribute(read_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem) != cudaSuccess) {
        cudaGetLastError();
        return RSTITCH_ERR_CUDA;
    }
    const unsigned grid = n_chunks < (unsigned long long)sms ? (unsigned)n_chunks : (unsigned)sms;
    read_stream_kernel<<<grid, 64, kProbeSmem, (cudaStream_t)cuda_stream>>>((const unsigned char *)buf, n_chunks, gave_up);
    if (cudaGetLastError() != cudaSuccess) return RSTITCH_ERR_CUDA;
    return RSTITCH_OK;
}
