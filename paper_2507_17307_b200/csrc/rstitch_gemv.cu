// Split-V streaming LM-head kernel for a handful of rows (S1-S3 fused, then the routing tail in
// the last block).  HBM-bound: the algorithmic traffic is V * d * 2 bytes per pass over the rows.
//
// One persistent block per SM owns one contiguous slice of the vocabulary.  A producer thread
// streams the slice's W_head rows, which are contiguous in memory, into a shared-memory ring with
// untiled bulk copies (one copy of VR rows per slot, completion on the slot's mbarrier), so many
// kilobytes per SM are in flight with no registers tied up.  Eight consumer warps take the slots
// round-robin: 128-bit shared-memory reads, exact bf16 -> fp32 widening, fp32 FMAs against the
// hidden rows held in shared memory, a warp butterfly per logit, and single-pass softmax
// statistics per row.  The logits exist only in registers.
#include "rstitch_kernels.cuh"
#include "rstitch_ptx.cuh"

namespace rstitch {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kThreads       = (kConsumerWarps + 1) * 32;   // + the producer warp
constexpr int kMaxSlots      = 32;
constexpr int kDynSmemMax    = 220 * 1024;
constexpr int kChunkTarget   = 20 * 1024;

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

__device__ __forceinline__ void raise_abort(volatile int *flag, DevStat *stat, unsigned site)
{
    *flag = 1;
    atomicAdd(&stat->timeouts, 1u);
    atomicExch(&stat->timeout_site, site);
}

// RT hidden rows per pass, VR vocabulary rows per ring slot.
template <int RT, int VR>
__global__ void __launch_bounds__(kThreads, 1)
head_stream_kernel(HeadArgs h, TailArgs t, Partials P, int n_slots, int hid_bytes)
{
    // The merge of the slices and the routing tail run in head_finalize_kernel, launched behind this
    // kernel; it and the next call's head kernel may be scheduled as soon as every block has got here.
    ptx::grid_dep_launch_dependents();
    extern __shared__ __align__(128) unsigned char dyn_smem[];   // [hidden RT x d][ring]
    __shared__ __align__(8) uint64_t s_full[kMaxSlots];
    __shared__ __align__(8) uint64_t s_empty[kMaxSlots];
    __shared__ Stats s_warp[kConsumerWarps][RT];
    __shared__ int   s_abort;
    __shared__ int   s_zero;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d8 = h.d >> 3;
    const int n_slices = gridDim.x, slice = blockIdx.x;
    const int v_begin = (int)(((long long)h.V * slice) / n_slices);
    const int v_end   = (int)(((long long)h.V * (slice + 1)) / n_slices);
    const int n_chunks = (v_end - v_begin + VR - 1) / VR;
    const uint32_t row_bytes = (uint32_t)h.d * 2u;
    const uint32_t chunk_bytes = row_bytes * VR;
    int R_live = h.R;
    // A live row count on the device comes from the kernel before this one: wait for it.  Otherwise the
    // producer streams W_head (which no earlier kernel writes) at once, and only the consumers wait,
    // before they read the hidden rows.
    if (h.n_rows_dev) { ptx::grid_dep_wait(); int n = *h.n_rows_dev; R_live = n < 0 ? 0 : (n < h.R ? n : h.R); }
    const int n_src = h.n_src > 0 ? h.n_src : h.R;
    const uint4 *H4 = (const uint4 *)h.hidden;
    uint4 *hid4 = (uint4 *)dyn_smem;
    unsigned char *ring = dyn_smem + hid_bytes;
    const uint32_t ring_u32 = ptx::smem_u32(ring);

    if (threadIdx.x == 0) { s_abort = 0; s_zero = 0; }

    int issued = 0;                // producer thread: copies issued in the current pass
    for (int r0 = 0; r0 < R_live; r0 += RT) {
        // every pass starts the ring from scratch (the previous pass has fully drained)
        if (threadIdx.x == 0) {
            for (int s = 0; s < n_slots; ++s) {
                if (r0 > 0) {
                    ptx::mbar_inval(ptx::smem_u32(&s_full[s]));
                    ptx::mbar_inval(ptx::smem_u32(&s_empty[s]));
                }
                ptx::mbar_init(ptx::smem_u32(&s_full[s]), 1);
                ptx::mbar_init(ptx::smem_u32(&s_empty[s]), 1);
            }
            ptx::mbar_fence_init();
        }
        issued = 0;
        __syncthreads();                       // barriers ready: the producer may start at once
        // hidden rows of this pass -> shared memory (rows past the live count read as zero); only
        // the consumer warps take part, the producer is already streaming W_head
        if (warp < kConsumerWarps) ptx::grid_dep_wait();      // earlier kernels' writes (hidden rows, scratch) are visible
        if (warp < kConsumerWarps)
        for (int i = threadIdx.x; i < RT * d8; i += kConsumerWarps * 32) {
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
            hid4[i] = v;
        }

        if (warp == kConsumerWarps) {
            // ---- producer: one thread feeds the ring -------------------------------------
            if (lane == 0) {
                int slot = 0, round = 0;
                const unsigned char *src = (const unsigned char *)h.W + (size_t)v_begin * row_bytes;
                for (int i = 0; i < n_chunks; ++i) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&s_empty[slot]), (uint32_t)((round & 1) ^ 1), &s_abort)) {
                        if (!s_abort) raise_abort(&s_abort, t.stat, 0x101u);
                        break;
                    }
                    int rows = v_end - (v_begin + i * VR);
                    uint32_t bytes = rows >= VR ? chunk_bytes : (uint32_t)rows * row_bytes;
                    uint32_t full = ptx::smem_u32(&s_full[slot]);
                    ptx::mbar_arrive_expect_tx(full, bytes);
                    ptx::bulk_g2s(ring_u32 + (uint32_t)slot * chunk_bytes, src + (size_t)i * chunk_bytes, bytes, full);
                    ++issued;
                    if (++slot == n_slots) { slot = 0; ++round; }
                }
            }
            __syncwarp();
        } else {
            // ---- consumers -----------------------------------------------------------------
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");   // hidden rows staged
            Stats st = stats_empty();
            const int my_r = lane & (RT - 1);
            // Slot s always goes to warp (s mod 8), so a warp meets the rounds of a slot in order
            // and a parity wait can never be satisfied by an older phase of the same barrier.
            bool live = true;
            for (int base = 0, round = 0; live && base < n_chunks; base += n_slots, ++round)
            for (int slot = warp; slot < n_slots; slot += kConsumerWarps) {
                const int i = base + slot;
                if (i >= n_chunks) break;
                if (!ptx::mbar_wait(ptx::smem_u32(&s_full[slot]), (uint32_t)(round & 1), &s_abort)) {
                    if (lane == 0 && !s_abort) raise_abort(&s_abort, t.stat, 0x102u);
                    live = false;
                    break;
                }
                const uint4 *wb = (const uint4 *)(ring + (size_t)slot * chunk_bytes);
                float acc[VR][RT];
#pragma unroll
                for (int v = 0; v < VR; ++v)
#pragma unroll
                    for (int r = 0; r < RT; ++r) acc[v][r] = 0.f;
#pragma unroll 2
                for (int c = lane; c < d8; c += 32) {
                    uint4 hv[RT];
#pragma unroll
                    for (int r = 0; r < RT; ++r) hv[r] = hid4[r * d8 + c];
#pragma unroll
                    for (int v = 0; v < VR; ++v) {
                        uint4 w = wb[v * d8 + c];
#pragma unroll
                        for (int r = 0; r < RT; ++r) acc[v][r] = dot8(w, hv[r], acc[v][r]);
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&s_empty[slot]));   // slot is free again
#pragma unroll
                for (int v = 0; v < VR; ++v)
#pragma unroll
                    for (int r = 0; r < RT; ++r) {
                        float z = acc[v][r];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
                        acc[v][r] = z;
                    }
                // lane l keeps the statistics of row (l mod RT); lanes >= RT duplicate that work
                const int v0 = v_begin + i * VR;
                const int rows = v_end - v0;
#pragma unroll
                for (int v = 0; v < VR; ++v) {
                    if (v < rows) {
                        float z = acc[v][0];
#pragma unroll
                        for (int r = 1; r < RT; ++r) z = (my_r == r) ? acc[v][r] : z;
                        const float score = h.sample.on ? sample_score(h.sample, z, (uint32_t)(r0 + my_r),
                                                                       (uint32_t)(v0 + v)) : z;
                        stats_push(st, z, v0 + v, score);
                    }
                }
            }
            if (lane < RT) s_warp[warp][lane] = st;
        }
        __syncthreads();
        if (threadIdx.x < RT && r0 + threadIdx.x < R_live) {
            Stats m = s_warp[0][threadIdx.x];
            for (int w = 1; w < kConsumerWarps; ++w) stats_merge(m, s_warp[w][threadIdx.x]);
            partial_store(P, (size_t)(r0 + threadIdx.x) * n_slices + slice, m);
        }
        if (s_abort) break;
    }

    // after a timeout: no copy may still be landing in this block's shared memory when it exits
    if (s_abort && warp == kConsumerWarps && lane == 0) {
        int first = issued > n_slots ? issued - n_slots : 0;
        for (int j = first; j < issued; ++j)
            ptx::mbar_wait(ptx::smem_u32(&s_full[j % n_slots]), (uint32_t)((j / n_slots) & 1), &s_zero);
    }

}

struct Plan { int RT, VR, n_slots, hid_bytes; size_t smem; };

Plan make_plan(int R, int d)
{
    Plan p;
    const int row_bytes = d * 2;
    p.VR = 8;
    while (p.VR > 1 && p.VR * row_bytes > kChunkTarget) p.VR >>= 1;
    p.RT = R <= 1 ? 1 : (R <= 2 ? 2 : 4);
    for (;;) {
        p.hid_bytes = ((p.RT * row_bytes + 127) / 128) * 128;
        int ring = kDynSmemMax - p.hid_bytes;
        p.n_slots = ring > 0 ? ring / (p.VR * row_bytes) : 0;
        if (p.n_slots >= 4 || p.RT == 1) break;
        p.RT >>= 1;                          // huge d: fewer rows per pass, more passes over W
    }
    if (p.n_slots > kMaxSlots) p.n_slots = kMaxSlots;
    if (p.n_slots > kConsumerWarps) p.n_slots -= p.n_slots % kConsumerWarps;   // even load over the warps
    p.smem = (size_t)p.hid_bytes + (size_t)p.n_slots * p.VR * row_bytes;
    return p;
}

template <int RT, int VR>
cudaError_t launch_inst(const HeadArgs &h, const TailArgs &t, const Scratch &s, const Plan &p, int grid,
                        cudaStream_t stream, int sm_count)
{
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        e = cudaFuncSetAttribute(head_stream_kernel<RT, VR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kDynSmemMax);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    Partials P = partials_carve(s.partials, (size_t)h.R, (size_t)grid);
    HeadArgs hh = h;
    TailArgs tt = t;
    int n_slots = p.n_slots, hid_bytes = p.hid_bytes;
    void *args[] = {&hh, &tt, &P, &n_slots, &hid_bytes};
    e = launch_dependent((const void *)head_stream_kernel<RT, VR>, dim3((unsigned)grid), dim3(kThreads), p.smem, stream, args);
    if (e != cudaSuccess) return e;
    return launch_head_finalize(P, grid, h.R, h.n_rows_dev, t, s.ticket, sm_count, stream);
}

template <int RT>
cudaError_t launch_rt(const HeadArgs &h, const TailArgs &t, const Scratch &s, const Plan &p, int grid,
                      cudaStream_t stream, int sm_count)
{
    switch (p.VR) {
        case 8:  return launch_inst<RT, 8>(h, t, s, p, grid, stream, sm_count);
        case 4:  return launch_inst<RT, 4>(h, t, s, p, grid, stream, sm_count);
        case 2:  return launch_inst<RT, 2>(h, t, s, p, grid, stream, sm_count);
        default: return launch_inst<RT, 1>(h, t, s, p, grid, stream, sm_count);
    }
}

}  // namespace

cudaError_t launch_head_gemv(const HeadArgs &h, const TailArgs &t, const Scratch &s, int sm_count,
                             cudaStream_t stream, int *launched)
{
    if (launched) *launched = 2;
    Plan p = make_plan(h.R, h.d);
    if (p.n_slots < 1) return cudaErrorInvalidValue;
    int grid = sm_count;
    int by_rows = (h.V + p.VR - 1) / p.VR;
    if (grid > by_rows) grid = by_rows;
    if (grid > kMaxSlices) grid = kMaxSlices;
    if (grid < 1) grid = 1;
    switch (p.RT) {
        case 1:  return launch_rt<1>(h, t, s, p, grid, stream, sm_count);
        case 2:  return launch_rt<2>(h, t, s, p, grid, stream, sm_count);
        default: return launch_rt<4>(h, t, s, p, grid, stream, sm_count);
    }
}

}  // namespace rstitch
