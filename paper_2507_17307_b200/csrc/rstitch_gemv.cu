// Split-V streaming LM-head kernel for a handful of rows (S1-S3 fused, then the routing tail in
// the last block).  Each block owns one contiguous slice of the vocabulary; W_head is read once
// with 128-bit loads, the logits live only in registers, and every warp keeps single-pass softmax
// statistics per row.  HBM-bound: the algorithmic traffic is V * d * 2 bytes per pass over the rows.
#include "rstitch_kernels.cuh"
#include <cuda_bf16.h>

namespace rstitch {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps   = kThreads / 32;

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// bf16 pair packed in a 32-bit word -> two floats (exact widening).
__device__ __forceinline__ float bf_lo(unsigned w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(unsigned w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float dot8(const uint4 &w, const uint4 &h, float acc)
{
    acc = fmaf(bf_lo(w.x), bf_lo(h.x), acc); acc = fmaf(bf_hi(w.x), bf_hi(h.x), acc);
    acc = fmaf(bf_lo(w.y), bf_lo(h.y), acc); acc = fmaf(bf_hi(w.y), bf_hi(h.y), acc);
    acc = fmaf(bf_lo(w.z), bf_lo(h.z), acc); acc = fmaf(bf_hi(w.z), bf_hi(h.z), acc);
    acc = fmaf(bf_lo(w.w), bf_lo(h.w), acc); acc = fmaf(bf_hi(w.w), bf_hi(h.w), acc);
    return acc;
}

template <int RT>
__global__ void __launch_bounds__(kThreads)
head_gemv_kernel(HeadArgs h, TailArgs t, Partials P, unsigned *ticket)
{
    extern __shared__ uint4 smem_hidden[];            // RT rows of d bf16
    __shared__ Stats s_warp[kWarps][RT];
    __shared__ int   s_tail[66];
    __shared__ int   s_last;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d8 = h.d >> 3;
    const int n_slices = gridDim.x, slice = blockIdx.x;
    const int v_begin = (int)(((long long)h.V * slice) / n_slices);
    const int v_end   = (int)(((long long)h.V * (slice + 1)) / n_slices);
    int R_live = h.R;
    if (h.n_rows_dev) { int n = *h.n_rows_dev; R_live = n < 0 ? 0 : (n < h.R ? n : h.R); }
    const int n_src = h.n_src > 0 ? h.n_src : h.R;
    const uint4 *W4 = (const uint4 *)h.W;
    const uint4 *H4 = (const uint4 *)h.hidden;

    for (int r0 = 0; r0 < R_live; r0 += RT) {
        __syncthreads();
        for (int i = threadIdx.x; i < RT * d8; i += kThreads) {
            int r = r0 + i / d8, c = i - (i / d8) * d8;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (r < R_live) {
                int src = h.row_idx ? h.row_idx[r] : r;
                if (src < 0 || src >= n_src) {
                    if (c == 0 && slice == 0) atomicAdd(&t.stat->bad_row_idx, 1u);
                    src = 0;
                }
                v = H4[(size_t)src * d8 + c];
            }
            smem_hidden[i] = v;
        }
        __syncthreads();

        Stats st[RT];
#pragma unroll
        for (int r = 0; r < RT; ++r) st[r] = stats_empty();

        for (int v = v_begin + warp; v < v_end; v += kWarps) {
            const uint4 *wrow = W4 + (size_t)v * d8;
            float acc[RT];
#pragma unroll
            for (int r = 0; r < RT; ++r) acc[r] = 0.f;
#pragma unroll 4
            for (int c = lane; c < d8; c += 32) {
                uint4 w = ldg_stream(wrow + c);
#pragma unroll
                for (int r = 0; r < RT; ++r) acc[r] = dot8(w, smem_hidden[r * d8 + c], acc[r]);
            }
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                float z = acc[r];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
                stats_push(st[r], z, v);
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < RT; ++r) s_warp[warp][r] = st[r];
        }
        __syncthreads();
        if (threadIdx.x < RT && r0 + threadIdx.x < R_live) {
            Stats m = s_warp[0][threadIdx.x];
            for (int w = 1; w < kWarps; ++w) stats_merge(m, s_warp[w][threadIdx.x]);
            partial_store(P, (size_t)(r0 + threadIdx.x) * n_slices + slice, m);
        }
    }

    // last block done: merge all slices and run the routing tail
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned k = atomicAdd(ticket, 1u);
        s_last = (k == (unsigned)(n_slices - 1));
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    TailArgs ta = t;
    ta.R = R_live;
    if (h.n_rows_dev) ta.B = R_live < t.B ? R_live : t.B;
    tail_finalize_rows(P, n_slices, ta);
    __syncthreads();
    tail_route(ta, s_tail);
    if (threadIdx.x == 0) {
        *ticket = 0u;
        atomicAdd(&t.stat->launches, 1u);
    }
}

template <int RT>
cudaError_t launch_rt(const HeadArgs &h, const TailArgs &t, const Scratch &s, int grid, cudaStream_t stream)
{
    size_t smem = (size_t)RT * h.d * 2;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(head_gemv_kernel<RT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
    }
    Partials P = partials_carve(s.partials, (size_t)h.R, (size_t)grid);
    head_gemv_kernel<RT><<<grid, kThreads, smem, stream>>>(h, t, P, s.ticket);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_head_gemv(const HeadArgs &h, const TailArgs &t, const Scratch &s, int sm_count,
                             cudaStream_t stream)
{
    int grid = sm_count * 4;
    int by_rows = (h.V + 7) / 8;
    if (grid > by_rows) grid = by_rows;
    if (grid > kMaxSlices) grid = kMaxSlices;
    if (grid < 1) grid = 1;
    if (h.R <= 1) return launch_rt<1>(h, t, s, grid, stream);
    if (h.R <= 2) return launch_rt<2>(h, t, s, grid, stream);
    return launch_rt<4>(h, t, s, grid, stream);
}

}  // namespace rstitch
