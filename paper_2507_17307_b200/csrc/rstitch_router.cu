// R-Stitch+ router forward on the rows whose entropy exceeded the threshold (Algorithm 1: when
// H_t > tau the hidden state s_t goes through a lightweight router and
// switch = (argmax_a pi(a | s_t) == LLM)).  The appendix on the router's architecture sketches it as
// 6 FFN blocks with GELU and residual connections, a normalisation and a two-head linear layer on the
// hidden state, 0.17 M parameters; widths are not given, so they are parameters here:
//     x0 = W_in s + b_in;  x <- x + W2_l GELU(W1_l x + b1_l) + b2_l;  y = LayerNorm(x) g + beta;
//     logits = W_out y + b_out   (exact erf GELU, eps = 1e-5).
// One block per row: the d -> h projection is spread over the block's warps (coalesced fp32 weight
// rows against the bf16 hidden row held in shared memory); narrow residual blocks, the normalisation and
// the head run on one warp, wide blocks on all of them.
#include "rstitch_kernels.cuh"
#include <math_constants.h>

namespace {

constexpr int kThreads = 512;
constexpr int kMaxH = 256, kMaxFF = 1024;
constexpr int kWarpStackMax = 8192;              // h * ff up to which one warp runs the residual blocks

__device__ __forceinline__ void cp_async16(float *dst_smem, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                 ::"r"((unsigned)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}

__device__ __forceinline__ void cp_async4(float *dst_smem, const float *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                 ::"r"((unsigned)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}

// All threads of the block: n floats, global -> shared, asynchronously.
__device__ __forceinline__ const float *stage_small(float *&cursor, const float *src, int n)
{
    float *dst = cursor;
    for (int i = threadIdx.x; i < n; i += blockDim.x) cp_async4(dst + i, src + i);
    cursor += (n + 3) & ~3;
    return dst;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// sum_k a[k] v[k] over k = 0 .. len-1, visited from element `start` on (mod len): the lanes of a warp,
// each on a row of its own, then read 32 different banks whatever the row stride.  Four independent
// chains; with a power-of-two length the indices need no wrap test and the loads run ahead of the FMAs.
__device__ __forceinline__ float dot_rotated(const float *a, const float *v, int len, int start)
{
    float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
    if (len >= 16 && (len & (len - 1)) == 0) {
        // sixteen elements at a time, every load issued before the first FMA: a single warp has nothing
        // else to hide the shared-memory latency with
        const int m = len - 1;
        for (int n = 0; n < len; n += 16) {
            float av[16], vv[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const int k = (n + q + start) & m;
                av[q] = a[k];
                vv[q] = v[k];
            }
#pragma unroll
            for (int q = 0; q < 16; q += 4) {
                c0 = fmaf(av[q], vv[q], c0);
                c1 = fmaf(av[q + 1], vv[q + 1], c1);
                c2 = fmaf(av[q + 2], vv[q + 2], c2);
                c3 = fmaf(av[q + 3], vv[q + 3], c3);
            }
        }
    } else if (len >= 4 && (len & (len - 1)) == 0) {
        const int m = len - 1;
#pragma unroll 4
        for (int n = 0; n < len; n += 4) {
            const int k0 = (n + start) & m, k1 = (n + 1 + start) & m, k2 = (n + 2 + start) & m, k3 = (n + 3 + start) & m;
            c0 = fmaf(a[k0], v[k0], c0);
            c1 = fmaf(a[k1], v[k1], c1);
            c2 = fmaf(a[k2], v[k2], c2);
            c3 = fmaf(a[k3], v[k3], c3);
        }
    } else {
        int k = start % len;
        for (int n = 0; n < len; ++n) {
            c0 = fmaf(a[k], v[k], c0);
            if (++k == len) k = 0;
        }
    }
    return (c0 + c1) + (c2 + c3);
}

// The same with 16-byte loads for lengths that are multiples of four (rows 16-byte aligned): n4 chunks of
// four, visited from chunk `start` on (mod n4).  A quarter-warp's eight lanes read eight different
// 16-byte bank groups, and a chunk costs two loads, four FMAs and the wrap test: a third of the
// instructions of the scalar form, which is what a single warp is short of.
__device__ __forceinline__ float dot_rotated4(const float4 *a, const float4 *v, int n4, int start)
{
    float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
    int k = start % n4;
#pragma unroll 4
    for (int n = 0; n < n4; ++n) {
        const float4 av = a[k], vv = v[k];
        c0 = fmaf(av.x, vv.x, c0);
        c1 = fmaf(av.y, vv.y, c1);
        c2 = fmaf(av.z, vv.z, c2);
        c3 = fmaf(av.w, vv.w, c3);
        if (++k == n4) k = 0;
    }
    return (c0 + c1) + (c2 + c3);
}

// One row by one block (every thread calls; warps other than the first may leave before the end).
__device__ __forceinline__ void router_row(const rstitch_router_t &w, const unsigned short *hidden, int n_src,
                                           const int32_t *row_idx, int r, float *logits_out, uint8_t *switch_out,
                                           uint8_t *refine_mask, int stage_weights, float *sm)
{
    float *s = sm, *x = sm + w.d, *t = x + w.h;
    int src = row_idx ? row_idx[r] : r;
    const bool valid = src >= 0 && src < n_src;      // an entry outside [0, n_src) reads row 0 and decides nothing
    if (!valid) src = 0;
    const unsigned short *hrow = hidden + (size_t)src * w.d;
    for (int k = threadIdx.x; k < w.d; k += kThreads) s[k] = __uint_as_float((unsigned)hrow[k] << 16);
    float *blk = t + w.ff;                        // staged block weights
    const float *p_b_in = w.b_in, *p_b1 = w.b1, *p_b2 = w.b2, *p_ln_g = w.ln_g, *p_ln_b = w.ln_b,
                *p_W_out = w.W_out, *p_b_out = w.b_out;
    const int per_block = 2 * w.ff * w.h;
    if (stage_weights == 2) {
        // every block's matrices at once with asynchronous 16-byte copies (no registers, no waiting
        // between them): one trip to L2 that overlaps the projection below
        const int n4 = (w.ff * w.h) >> 2;
        for (int l = 0; l < w.n_blocks; ++l) {
            const float *w1 = w.W1 + (size_t)l * w.ff * w.h, *w2 = w.W2 + (size_t)l * w.h * w.ff;
            float *dst = blk + (size_t)l * per_block;
            for (int i = threadIdx.x; i < n4; i += kThreads) {
                cp_async16(dst + 4 * i, w1 + 4 * i);
                cp_async16(dst + w.ff * w.h + 4 * i, w2 + 4 * i);
            }
        }
        // and every small vector: a scalar read from global memory inside the layer loops costs a full
        // trip to L2 each time
        float *cursor = blk + (size_t)w.n_blocks * per_block;
        p_b_in = stage_small(cursor, w.b_in, w.h);
        p_b1 = stage_small(cursor, w.b1, w.n_blocks * w.ff);
        p_b2 = stage_small(cursor, w.b2, w.n_blocks * w.h);
        p_ln_g = stage_small(cursor, w.ln_g, w.h);
        p_ln_b = stage_small(cursor, w.ln_b, w.h);
        p_W_out = stage_small(cursor, w.W_out, 2 * w.h);
        p_b_out = stage_small(cursor, w.b_out, 2);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = kThreads / 32;
    // x0 = W_in s + b_in: sixteen warps, two outputs each at a time, sixteen 16-byte loads in flight
    // per lane (the projection is latency-bound: a block reads all of W_in from L2 by itself)
    const int d4 = w.d >> 2;
    const float4 *s4 = reinterpret_cast<const float4 *>(s);
    for (int i0 = warp * 2; i0 < w.h; i0 += nwarps * 2) {
        float acc[2] = {0.f, 0.f};
        const float4 *wr[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) wr[q] = reinterpret_cast<const float4 *>(w.W_in + (size_t)min(i0 + q, w.h - 1) * w.d);
#pragma unroll 8
        for (int k = lane; k < d4; k += 32) {
            const float4 sv = s4[k];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const float4 wv = __ldg(wr[q] + k);
                acc[q] = fmaf(wv.x, sv.x, fmaf(wv.y, sv.y, fmaf(wv.z, sv.z, fmaf(wv.w, sv.w, acc[q]))));
            }
        }
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const float v = warp_sum(acc[q]);
            if (lane == 0 && i0 + q < w.h) x[i0 + q] = v;            // the bias joins after the staging wait
        }
    }
    __syncthreads();
    if (stage_weights == 2) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    }
    if (threadIdx.x < w.h) x[threadIdx.x] += p_b_in[threadIdx.x];
    __syncthreads();
    // Narrow blocks (the paper's router has ~0.17 M parameters, nearly all of them in W_in): with every
    // weight already in shared memory one warp runs the whole stack, a lane per output, synchronising
    // with __syncwarp only; sixteen warps sharing these tiny products spent ~3300 cycles per block on
    // block-wide barriers and shuffle trees.
    const bool warp_stack = stage_weights == 2 && w.h * w.ff <= kWarpStackMax;
    if (warp_stack && warp != 0) return;
    const bool vec4 = ((w.h | w.ff) & 3) == 0;       // with d % 4 == 0: x, t and every staged row are 16-byte aligned
    for (int l = 0; warp_stack && l < w.n_blocks; ++l) {
        const float *w1 = blk + (size_t)l * per_block, *w2 = w1 + w.ff * w.h;
        for (int j = lane; j < w.ff; j += 32) {
            const float *row = w1 + (size_t)j * w.h;
            const float dot = vec4 ? dot_rotated4(reinterpret_cast<const float4 *>(row),
                                                  reinterpret_cast<const float4 *>(x), w.h >> 2, lane)
                                   : dot_rotated(row, x, w.h, lane);
            const float a = p_b1[(size_t)l * w.ff + j] + dot;
            t[j] = 0.5f * a * (1.0f + erff(a * 0.70710678118654752f));      // exact GELU
        }
        __syncwarp();
        for (int i = lane; i < w.h; i += 32) {                               // residual; x[i] has one reader here
            const float *row = w2 + (size_t)i * w.ff;
            const float dot = vec4 ? dot_rotated4(reinterpret_cast<const float4 *>(row),
                                                  reinterpret_cast<const float4 *>(t), w.ff >> 2, lane)
                                   : dot_rotated(row, t, w.ff, lane);
            x[i] += p_b2[(size_t)l * w.h + i] + dot;
        }
        __syncwarp();
    }
    for (int l = 0; !warp_stack && l < w.n_blocks; ++l) {           // residual FFN blocks, wide: the whole block
        const float *w1 = w.W1 + (size_t)l * w.ff * w.h, *w2 = w.W2 + (size_t)l * w.h * w.ff;
        if (stage_weights == 2) {
            w1 = blk + (size_t)l * per_block;
            w2 = w1 + w.ff * w.h;
        } else if (stage_weights == 1) {
            // both matrices of the block into shared memory with coalesced, independent loads: one trip
            // to L2 per block instead of a dependent chain of loads inside the small dot products
            float *s1 = blk, *s2 = s1 + w.ff * w.h;
#pragma unroll 8
            for (int i = threadIdx.x; i < w.ff * w.h; i += kThreads) { s1[i] = __ldg(w1 + i); s2[i] = __ldg(w2 + i); }
            __syncthreads();
            w1 = s1; w2 = s2;
        }
        // a warp takes four outputs at a time, lanes over the inner index: consecutive shared-memory
        // words (no bank conflicts), four independent dot products and butterflies in flight (a single
        // chain of dependent shuffles per output made each block cost ~8000 cycles), and lanes 0-3 apply
        // the activation to one output each
        for (int j0 = warp * 4; j0 < w.ff; j0 += nwarps * 4) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int i = lane; i < w.h; i += 32) {
                const float xi = x[i];
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] = fmaf(w1[(size_t)min(j0 + q, w.ff - 1) * w.h + i], xi, acc[q]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], o);
            }
            const float mine = lane == 0 ? acc[0] : (lane == 1 ? acc[1] : (lane == 2 ? acc[2] : acc[3]));
            if (lane < 4 && j0 + lane < w.ff) {
                const float a = mine + p_b1[(size_t)l * w.ff + j0 + lane];
                t[j0 + lane] = 0.5f * a * (1.0f + erff(a * 0.70710678118654752f));      // exact GELU
            }
        }
        __syncthreads();
        for (int i0 = warp * 4; i0 < w.h; i0 += nwarps * 4) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int j = lane; j < w.ff; j += 32) {
                const float tj = t[j];
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] = fmaf(w2[(size_t)min(i0 + q, w.h - 1) * w.ff + j], tj, acc[q]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], o);
            }
            const float mine = lane == 0 ? acc[0] : (lane == 1 ? acc[1] : (lane == 2 ? acc[2] : acc[3]));
            if (lane < 4 && i0 + lane < w.h) x[i0 + lane] += mine + p_b2[(size_t)l * w.h + i0 + lane];   // residual
        }
        __syncthreads();
    }
    if (warp == 0) {                                                // LayerNorm and the two-way head
        float sum = 0.f;
        for (int i = lane; i < w.h; i += 32) sum += x[i];
        const float mean = warp_sum(sum) / (float)w.h;
        float sq = 0.f;
        for (int i = lane; i < w.h; i += 32) { float dlt = x[i] - mean; sq = fmaf(dlt, dlt, sq); }
        const float inv = rsqrtf(warp_sum(sq) / (float)w.h + 1e-5f);
        float a0 = 0.f, a1 = 0.f;
        for (int i = lane; i < w.h; i += 32) {
            const float y = (x[i] - mean) * inv * p_ln_g[i] + p_ln_b[i];
            a0 = fmaf(p_W_out[i], y, a0);
            a1 = fmaf(p_W_out[w.h + i], y, a1);
        }
        a0 = warp_sum(a0) + p_b_out[0];
        a1 = warp_sum(a1) + p_b_out[1];
        if (lane == 0) {
            const uint8_t sw = (valid && a1 > a0) ? 1 : 0;          // a tie keeps the SLM
            logits_out[2 * r] = a0;
            logits_out[2 * r + 1] = a1;
            if (switch_out) switch_out[r] = sw;
            if (refine_mask && row_idx && valid) refine_mask[src] = sw;
        }
    }
}

// Ticket of the compacting form: the blocks of one launch count themselves here, the last one resets it.
__device__ unsigned g_router_ticket = 0;

// cmp_count == nullptr: the router alone.  Otherwise every block takes a ticket when its row is done and
// the last one compacts refine_mask [n_src] into cmp_idx / cmp_count, as rstitch_compact would.
__global__ void __launch_bounds__(kThreads, 1)
router_kernel(rstitch_router_t w, const unsigned short *hidden, int n_src, const int32_t *row_idx,
              const int32_t *n_rows_dev, int R, float *logits_out, uint8_t *switch_out, uint8_t *refine_mask,
              int stage_weights, int32_t *cmp_idx, int32_t *cmp_count, const int32_t *n_seq_dev, const int32_t *tok,
              rstitch::Alg1Tail alg1)
{
    extern __shared__ __align__(16) float sm[];   // [d] hidden row | [h] x | [ff] t | [ff h] W1 | [h ff] W2 of a block
    __shared__ int s_tail[66];
    __shared__ int s_last;
    int R_live = R;
    if (n_rows_dev) { int n = *n_rows_dev; R_live = n < 0 ? 0 : (n < R ? n : R); }
    const int r = blockIdx.x;
    if (r < R_live) router_row(w, hidden, n_src, row_idx, r, logits_out, switch_out, refine_mask, stage_weights, sm);
    if (cmp_count == nullptr) return;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&g_router_ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    int n_seq = n_src;                              // mask entries that are live in this round
    if (n_seq_dev) { int n = *n_seq_dev; n_seq = n < 0 ? 0 : (n < n_src ? n : n_src); }
    rstitch::tail_compact(refine_mask, n_seq, nullptr, nullptr, cmp_idx, cmp_count, nullptr, nullptr, nullptr, s_tail);
    // Algorithm 1, R-Stitch+ lines: the SLM's decision block runs on the mask the router has just refined
    if (alg1.on) rstitch::alg1_tail_block(alg1, tok, refine_mask, s_tail);
    if (threadIdx.x == 0) g_router_ticket = 0u;
}

}  // namespace

static int router_launch(const rstitch_router_t *w, const void *hidden, int n_src,
                         const int32_t *row_idx, const int32_t *n_rows_dev, int R,
                         float *logits_out, uint8_t *switch_out, uint8_t *refine_mask,
                         int32_t *cmp_idx, int32_t *cmp_count, void *cuda_stream,
                         const int32_t *n_seq_dev = nullptr, const int32_t *tok = nullptr,
                         const rstitch::Alg1Tail *alg1 = nullptr)
{
    if (!w || R < 0 || n_src < 0 || !logits_out) return RSTITCH_ERR_INVALID_ARG;
    if (R > 0 && n_src == 0) return RSTITCH_ERR_INVALID_ARG;           // rows to read, but none present
    if (w->d < 1 || w->h < 1 || w->ff < 1 || w->n_blocks < 0) return RSTITCH_ERR_INVALID_ARG;
    if (w->h > kMaxH || w->ff > kMaxFF || w->d > 16384) return RSTITCH_ERR_UNSUPPORTED_SHAPE;
    if (!w->W_in || !w->b_in || !w->ln_g || !w->ln_b || !w->W_out || !w->b_out) return RSTITCH_ERR_INVALID_ARG;
    if (w->n_blocks > 0 && (!w->W1 || !w->b1 || !w->W2 || !w->b2)) return RSTITCH_ERR_INVALID_ARG;
    if (R > 0 && !hidden) return RSTITCH_ERR_INVALID_ARG;
    if (refine_mask && !row_idx) return RSTITCH_ERR_INVALID_ARG;
    if (R == 0) return RSTITCH_OK;
    if (w->d % 4 != 0) return RSTITCH_ERR_UNSUPPORTED_SHAPE;
    if ((reinterpret_cast<uintptr_t>(w->W_in) & 15u) != 0) return RSTITCH_ERR_BAD_ALIGN;     // read 16 bytes at a time
    size_t smem = (size_t)(w->d + w->h + w->ff) * sizeof(float);
    const size_t one = 2 * (size_t)w->h * w->ff * sizeof(float);
    // 2: all blocks' matrices staged at once; 1: one block at a time; 0: large widths read them from L2
    int stage_weights = 0;
    const bool aligned16 = ((reinterpret_cast<uintptr_t>(w->W1) | reinterpret_cast<uintptr_t>(w->W2)) & 15u) == 0 &&
                           (w->h * w->ff) % 4 == 0 && (w->d + w->h + w->ff) % 4 == 0;
    const size_t small = (size_t)(w->h * 6 + w->n_blocks * (w->ff + w->h) + 64) * sizeof(float);
    if (aligned16 && smem + one * (size_t)w->n_blocks + small <= 200 * 1024) {
        stage_weights = 2;
        smem += one * (size_t)w->n_blocks + small;
    }
    else if (smem + one <= 200 * 1024)                  { stage_weights = 1; smem += one; }
    static size_t configured[64] = {};       // largest dynamic shared memory asked for so far, per device
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    if (smem > 48 * 1024 && smem > configured[dev]) {
        if (cudaFuncSetAttribute(router_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return RSTITCH_ERR_CUDA;
        }
        configured[dev] = smem;
    }
    router_kernel<<<R, kThreads, smem, (cudaStream_t)cuda_stream>>>(*w, (const unsigned short *)hidden, n_src, row_idx,
                                                                    n_rows_dev, R, logits_out, switch_out, refine_mask,
                                                                    stage_weights, cmp_idx, cmp_count, n_seq_dev, tok,
                                                                    alg1 ? *alg1 : rstitch::Alg1Tail{});
    if (cudaGetLastError() != cudaSuccess) return RSTITCH_ERR_CUDA;
    return RSTITCH_OK;
}

extern "C" int rstitch_router_forward(const rstitch_router_t *w, const void *hidden, int n_src,
                                      const int32_t *row_idx, const int32_t *n_rows_dev, int R,
                                      float *logits_out, uint8_t *switch_out, uint8_t *refine_mask,
                                      void *cuda_stream)
{
    return router_launch(w, hidden, n_src, row_idx, n_rows_dev, R, logits_out, switch_out, refine_mask, nullptr,
                         nullptr, cuda_stream);
}

extern "C" int rstitch_router_route(const rstitch_router_t *w, const void *hidden, int n_src,
                                    const int32_t *row_idx, const int32_t *n_rows_dev, int R,
                                    float *logits_out, uint8_t *switch_out, uint8_t *route_mask,
                                    int32_t *llm_idx, int32_t *llm_count, void *cuda_stream)
{
    if (!row_idx || !route_mask || !llm_count || (n_src > 0 && !llm_idx)) return RSTITCH_ERR_INVALID_ARG;
    if (n_src > 65536) return RSTITCH_ERR_UNSUPPORTED_SHAPE;             // one block compacts the mask
    if (R == 0) return rstitch_compact(route_mask, n_src, llm_idx, llm_count, cuda_stream);
    return router_launch(w, hidden, n_src, row_idx, n_rows_dev, R, logits_out, switch_out, route_mask, llm_idx,
                         llm_count, cuda_stream);
}

extern "C" int rstitch_router_route_alg1(const rstitch_router_t *w, const void *hidden, int n_src,
                                         const int32_t *n_seq_dev, const int32_t *row_idx, const int32_t *n_rows_dev,
                                         int R, float *logits_out, uint8_t *switch_out, uint8_t *route_mask,
                                         int32_t *llm_idx, int32_t *llm_count, const int32_t *tok,
                                         const rstitch_alg1_tail_t *alg1_tail, void *cuda_stream)
{
    if (!row_idx || !route_mask || !llm_count || (n_src > 0 && !llm_idx) || !alg1_tail || !tok)
        return RSTITCH_ERR_INVALID_ARG;
    if (n_src > 65536) return RSTITCH_ERR_UNSUPPORTED_SHAPE;             // one block compacts the mask
    rstitch::Alg1Tail alg1;
    if (!rstitch::make_alg1_tail(alg1_tail, &alg1) || alg1.model != 0) return RSTITCH_ERR_INVALID_ARG;
    if (R == 0 || n_src == 0) {
        // no row can have crossed the threshold: the compaction of the mask as it stands, then the block
        int st = rstitch_compact(route_mask, n_src, llm_idx, llm_count, cuda_stream);
        if (st != RSTITCH_OK) return st;
        if (rstitch::launch_alg1_tail(alg1, tok, route_mask, (cudaStream_t)cuda_stream) != cudaSuccess) {
            cudaGetLastError();
            return RSTITCH_ERR_CUDA;
        }
        return RSTITCH_OK;
    }
    return router_launch(w, hidden, n_src, row_idx, n_rows_dev, R, logits_out, switch_out, route_mask, llm_idx,
                         llm_count, cuda_stream, n_seq_dev, tok, &alg1);
}
