// Internal launch interfaces between the C ABI (rstitch_api.cu) and the kernel files.
#pragma once
#include "rstitch_tail.cuh"
#include "rstitch_sample.cuh"
#include <cuda_runtime.h>

namespace rstitch {

constexpr int    kMaxSlices   = 1024;   // upper bound on vocabulary slices (partials per row)
constexpr size_t kWsHeader    = 256;    // ticket counter lives in the first 256 bytes of the scratch

// What the head kernels read.
struct HeadArgs {
    const void    *hidden;      // bf16 [n_src, d]
    const void    *W;           // bf16 [V, d]
    int            R, d, V, n_src;
    const int32_t *row_idx;     // optional gather
    const int32_t *n_rows_dev;  // optional live row count
    SampleArgs     sample;      // sampled instead of greedy token
};

struct Scratch {
    unsigned *ticket;           // one counter, zero between launches
    void     *partials;         // partials_bytes(R, n_slices)
};

__host__ inline Scratch scratch_carve(void *ws)
{
    Scratch s;
    s.ticket   = (unsigned *)ws;
    s.partials = (char *)ws + kWsHeader;
    return s;
}

// CUDA-core streaming kernel: split-V GEMV for a handful of rows.
// *launched (optional for the streaming kernel) receives the number of kernels enqueued.
// Both head launchers enqueue the head kernel, which stops at the per-slice statistics, and
// head_finalize_kernel behind it.
cudaError_t launch_head_gemv(const HeadArgs &h, const TailArgs &t, const Scratch &s, int sm_count,
                             cudaStream_t stream, int *launched = nullptr);

// Tensor-core kernel (tcgen05 + tensor memory): any row count; the choice between the two is the
// caller's.  gather_buf (umma_gather_bytes(R, d) bytes, 256-byte aligned) is used only with row_idx.
// Encoded tensor maps by (base pointer, rows, d, box rows), least recently used replaced; owned by a
// handle and touched only on the host, by the thread that enqueues through that handle.
struct TmapCache {
    struct Entry {
        const void *base = nullptr;
        int rows = 0, d = 0, box_rows = 0;
        unsigned long long used = 0;             // 0: empty
        alignas(64) unsigned char map[128];
    } e[24];
    unsigned long long clock = 0;
};
bool        umma_shape_ok(int R, int d, int V);
size_t      umma_gather_bytes(int R, int d);
cudaError_t launch_head_umma(const HeadArgs &h, const TailArgs &t, const Scratch &s, void *gather_buf,
                             int sm_count, cudaStream_t stream, int *launched, TmapCache *cache = nullptr);

// The cross-block merge and the routing tail as a launch of its own, behind a head kernel that was
// launched without its fused tail (rstitch_finalize.cu).  Both launches carry the programmatic stream
// serialisation attribute; launch_dependent is the launch helper for such kernels.
cudaError_t launch_dependent(const void *func, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, void **args);
cudaError_t launch_head_finalize(const Partials &P, int n_slices, int R, const int32_t *n_rows_dev,
                                 const TailArgs &t, unsigned *ticket, int sm_count, cudaStream_t stream);

// Merge of the gathered vocabulary shards ([n_shards][R][5] words, shard-major) and the routing tail.
cudaError_t launch_shard_merge(const float *gathered, int n_shards, const int32_t *n_rows_dev, const TailArgs &t,
                               unsigned *ticket, cudaStream_t stream, int *launched);

// Algorithm 1's block after a routing call that has no rows of its own (one small launch), and the
// check of a caller's state structure.
bool        alg1_state_ok(const rstitch_alg1_state_t *s);
bool        make_alg1_tail(const rstitch_alg1_tail_t *t, Alg1Tail *out);   // host structure -> what the kernels carry; false: bad
cudaError_t launch_alg1_tail(const Alg1Tail &a, const int32_t *tok, const uint8_t *mask, cudaStream_t stream);

// The bounded wait running out on purpose (rstitch_selftest_wait): site id it leaves in the status word.
constexpr unsigned kSelftestSite = 0x7e57u;
cudaError_t launch_wait_selftest(DevStat *stat, long long limit_cycles, cudaStream_t stream);

// Upper bound on the partials per row of any kernel for a vocabulary of V rows.
__host__ __device__ inline size_t max_slices_for(int V)
{
    size_t tiles = ((size_t)(V > 0 ? V : 1) + 255) / 256;
    return tiles > (size_t)kMaxSlices ? tiles : (size_t)kMaxSlices;
}

// Stand-alone ordered compaction (S5).
cudaError_t launch_compact(const uint8_t *mask, int B, int32_t *idx, int32_t *count, DevStat *stat,
                           int32_t *block_counts /* scratch for B > one block's reach, or null */,
                           cudaStream_t stream, int *launched);
constexpr int kCompactOneBlockMax = 1 << 16;
constexpr int kCompactTile        = 4096;     // sequences per block in the multi-block form

}  // namespace rstitch
