// R-Stitch+ router forward on the rows whose entropy exceeded the threshold (Algorithm 1: when
// H_t > tau the hidden state s_t goes through a lightweight router and
// switch = (argmax_a pi(a | s_t) == LLM)).  The appendix on the router's architecture sketches it as
// 6 FFN blocks with GELU and residual connections, a normalisation and a two-head linear layer on the
// hidden state, 0.17 M parameters; widths are not given, so they are parameters here:
//     x0 = W_in s + b_in;  x <- x + W2_l GELU(W1_l x + b1_l) + b2_l;  y = LayerNorm(x) g + beta;
//     logits = W_out y + b_out   (exact erf GELU, eps = 1e-5).
// One block per row: the d -> h projection is spread over the block's warps (coalesced fp32 weight
// rows against the bf16 hidden row held in shared memory), the small blocks run on one warp.
#include "../../include/rstitch.h"
#include <cuda_runtime.h>
#include <math_constants.h>

namespace {

constexpr int kThreads = 256;
constexpr int kMaxH = 256, kMaxFF = 1024;

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kThreads)
router_kernel(rstitch_router_t w, const unsigned short *hidden, int n_src, const int32_t *row_idx,
              const int32_t *n_rows_dev, int R, float *logits_out, uint8_t *switch_out, uint8_t *refine_mask)
{
    extern __shared__ float sm[];                 // [d] hidden row | [h] x | [ff] t
    float *s = sm, *x = sm + w.d, *t = x + w.h;
    int R_live = R;
    if (n_rows_dev) { int n = *n_rows_dev; R_live = n < 0 ? 0 : (n < R ? n : R); }
    const int r = blockIdx.x;
    if (r >= R_live) return;
    int src = row_idx ? row_idx[r] : r;
    if (src < 0 || src >= n_src) src = 0;
    const unsigned short *hrow = hidden + (size_t)src * w.d;
    for (int k = threadIdx.x; k < w.d; k += kThreads) s[k] = __uint_as_float((unsigned)hrow[k] << 16);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = kThreads / 32;
    for (int i = warp; i < w.h; i += nwarps) {                       // x0 = W_in s + b_in
        const float *wr = w.W_in + (size_t)i * w.d;
        float acc = 0.f;
        for (int k = lane; k < w.d; k += 32) acc = fmaf(wr[k], s[k], acc);
        acc = warp_sum(acc);
        if (lane == 0) x[i] = acc + w.b_in[i];
    }
    __syncthreads();
    for (int l = 0; l < w.n_blocks; ++l) {                          // residual FFN blocks
        const float *w1 = w.W1 + (size_t)l * w.ff * w.h, *w2 = w.W2 + (size_t)l * w.h * w.ff;
        for (int j = threadIdx.x; j < w.ff; j += kThreads) {
            float acc = w.b1[(size_t)l * w.ff + j];
            for (int i = 0; i < w.h; ++i) acc = fmaf(w1[(size_t)j * w.h + i], x[i], acc);
            t[j] = 0.5f * acc * (1.0f + erff(acc * 0.70710678118654752f));     // exact GELU
        }
        __syncthreads();
        float add = 0.f;
        if (threadIdx.x < w.h) {
            add = w.b2[(size_t)l * w.h + threadIdx.x];
            for (int j = 0; j < w.ff; ++j) add = fmaf(w2[(size_t)threadIdx.x * w.ff + j], t[j], add);
        }
        __syncthreads();
        if (threadIdx.x < w.h) x[threadIdx.x] += add;
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
            const float y = (x[i] - mean) * inv * w.ln_g[i] + w.ln_b[i];
            a0 = fmaf(w.W_out[i], y, a0);
            a1 = fmaf(w.W_out[w.h + i], y, a1);
        }
        a0 = warp_sum(a0) + w.b_out[0];
        a1 = warp_sum(a1) + w.b_out[1];
        if (lane == 0) {
            const uint8_t sw = a1 > a0 ? 1 : 0;                     // a tie keeps the SLM
            logits_out[2 * r] = a0;
            logits_out[2 * r + 1] = a1;
            if (switch_out) switch_out[r] = sw;
            if (refine_mask && row_idx) refine_mask[src] = sw;
        }
    }
}

}  // namespace

extern "C" int rstitch_router_forward(const rstitch_router_t *w, const void *hidden, int n_src,
                                      const int32_t *row_idx, const int32_t *n_rows_dev, int R,
                                      float *logits_out, uint8_t *switch_out, uint8_t *refine_mask,
                                      void *cuda_stream)
{
    if (!w || R < 0 || n_src < 0 || !logits_out) return RSTITCH_ERR_INVALID_ARG;
    if (w->d < 1 || w->h < 1 || w->ff < 1 || w->n_blocks < 0) return RSTITCH_ERR_INVALID_ARG;
    if (w->h > kMaxH || w->ff > kMaxFF || w->d > 16384) return RSTITCH_ERR_UNSUPPORTED_SHAPE;
    if (!w->W_in || !w->b_in || !w->ln_g || !w->ln_b || !w->W_out || !w->b_out) return RSTITCH_ERR_INVALID_ARG;
    if (w->n_blocks > 0 && (!w->W1 || !w->b1 || !w->W2 || !w->b2)) return RSTITCH_ERR_INVALID_ARG;
    if (R > 0 && !hidden) return RSTITCH_ERR_INVALID_ARG;
    if (refine_mask && !row_idx) return RSTITCH_ERR_INVALID_ARG;
    if (R == 0) return RSTITCH_OK;
    const size_t smem = (size_t)(w->d + w->h + w->ff) * sizeof(float);
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(router_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return RSTITCH_ERR_CUDA;
        }
    }
    router_kernel<<<R, kThreads, smem, (cudaStream_t)cuda_stream>>>(*w, (const unsigned short *)hidden, n_src, row_idx,
                                                                    n_rows_dev, R, logits_out, switch_out, refine_mask);
    if (cudaGetLastError() != cudaSuccess) return RSTITCH_ERR_CUDA;
    return RSTITCH_OK;
}
