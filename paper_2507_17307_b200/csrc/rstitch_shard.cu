// Vocabulary-parallel LM head, second half: merge of the per-shard softmax statistics and the routing tail.
//
// Each shard (one GPU's slice of W_head's rows) leaves five words per row: m, s, u of Eq. 1's
// single-pass form, the best token score and the global index of that token.  After the shards have
// been gathered into one buffer ([n_shards][R][5], shard-major, e.g. by an all-gather), one thread per row
// merges them in ascending shard order -- the same merge as between the thread blocks of a head kernel,
// so the lowest index still wins ties -- and writes entropy and token; the last block to finish applies
// the rule of Eq. 2 and compacts, as the head kernels' own last block does.  No block waits on another.
#include "rstitch_kernels.cuh"

namespace rstitch {
namespace {

constexpr int kMergeThreads = 256;

__global__ void __launch_bounds__(kMergeThreads)
shard_merge_kernel(const float *__restrict__ gathered, int n_shards, const int32_t *n_rows_dev, TailArgs t,
                   unsigned *ticket)
{
    __shared__ int s_tail[66];
    __shared__ int s_last;
    int R_live = t.R;
    if (n_rows_dev) { int n = *n_rows_dev; R_live = n < 0 ? 0 : (n < t.R ? n : t.R); }
    const int r = blockIdx.x * kMergeThreads + threadIdx.x;
    if (r < R_live) {
        Stats acc = stats_empty();
        for (int g = 0; g < n_shards; ++g) {
            const float *w = gathered + ((size_t)g * t.R + r) * kShardWords;
            Stats p;
            p.m = w[0]; p.s = w[1]; p.u = w[2]; p.bv = w[3]; p.bi = __float_as_int(w[4]);
            stats_merge(acc, p);
        }
        tail_emit_row(acc, r, t);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned k = atomicAdd(ticket, 1u);
        s_last = (k == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    TailArgs ta = t;
    ta.R = R_live;
    if (n_rows_dev) ta.B = R_live < t.B ? R_live : t.B;
    tail_route(ta, s_tail);
    if (threadIdx.x == 0) *ticket = 0u;
}

}  // namespace

cudaError_t launch_shard_merge(const float *gathered, int n_shards, const int32_t *n_rows_dev, const TailArgs &t,
                               unsigned *ticket, cudaStream_t stream, int *launched)
{
    *launched = 0;
    const int grid = (t.R + kMergeThreads - 1) / kMergeThreads;
    shard_merge_kernel<<<grid, kMergeThreads, 0, stream>>>(gathered, n_shards, n_rows_dev, t, ticket);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) *launched = 1;
    return e;
}

}  // namespace rstitch
