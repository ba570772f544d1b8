// The steps of Algorithm 1 either side of the routing decision, batched: per-sequence state kept on
// the device (active model, the two KV-cache sizes, sequence length, generated tokens) and two small
// kernels per model and iteration.
//   plan:   which sequences run on this model now, how many tokens each must process (prefill of
//           the missing span, or one decode token), the row offsets of that batch, the KV-size
//           update, and the latency estimate of Eq. 5 accumulated per sequence;
//   commit: the decision block after the entropy test -- discard and roll back on an SLM hand-off,
//           hand back from the LLM on low entropy, append the token, stop on EOS.
// Integer work on B elements; one block, warp ballots and prefix sums for the ordered run list.
#include "../../include/rstitch.h"
#include <cuda_runtime.h>

#include <cmath>

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
alg1_init_kernel(rstitch_alg1_state_t s, int B, const int32_t *prompt_len)
{
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
        s.active[b] = 0; s.kv_slm[b] = 0; s.kv_llm[b] = 0;
        s.seq_len[b] = prompt_len[b];
        s.n_out[b] = 0; s.done[b] = 0; s.iters[b] = 0;
        s.kept[b] = 0; s.kept[B + b] = 0; s.steps[b] = 0; s.steps[B + b] = 0;
        s.lat_ms[b] = 0.0;
    }
}

// One block.  Sequences are taken in chunks of blockDim.x; inside a chunk a ballot gives each selected
// sequence its rank within the warp, warp totals are scanned in shared memory and a carry links the
// chunks, so run_idx comes out ascending and row_off is the exclusive scan of n_inf in that order.
__global__ void __launch_bounds__(kThreads)
alg1_plan_kernel(rstitch_alg1_state_t s, int B, int model, int t_max, rstitch_latency_model_t lat,
                 int32_t *run_idx, int32_t *run_count, int32_t *n_inf_out, int32_t *n_kv_out, int32_t *row_off)
{
    __shared__ int w_cnt[kThreads / 32], w_rows[kThreads / 32], carry[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    int32_t *kv = model == 0 ? s.kv_slm : s.kv_llm;
    if (threadIdx.x == 0) { carry[0] = 0; carry[1] = 0; }
    __syncthreads();
    for (int base = 0; base < B; base += blockDim.x) {
        const int b = base + threadIdx.x;
        bool run = false;
        int n_inf = 0, n_kv = 0;
        if (b < B) run = !s.done[b] && s.iters[b] < t_max && s.active[b] == model;   // "for t = 1 .. T_max"
        if (run) {
            const int L = kv[b], len = s.seq_len[b];
            n_kv = L;
            if (L < len) { n_inf = len - L; kv[b] = len + 1; }         // prefill of the missing span
            else         { n_inf = 1;       kv[b] = L + 1; }           // decode
            const double ni = (double)n_inf, nk = (double)n_kv;
            s.lat_ms[b] += lat.a * ni * nk + lat.b * ni * ni + lat.c * ni + lat.d;     // Eq. 5
            s.steps[model * B + b] += 1;
            s.iters[b] += 1;
        }
        const unsigned ball = __ballot_sync(0xffffffffu, run);
        const int rank = __popc(ball & ((1u << lane) - 1u));
        int incl = n_inf;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) { w_cnt[warp] = __popc(ball); w_rows[warp] = incl; }
        __syncthreads();
        int pre_cnt = carry[0], pre_rows = carry[1];
        for (int w = 0; w < warp; ++w) { pre_cnt += w_cnt[w]; pre_rows += w_rows[w]; }
        if (run) {
            const int j = pre_cnt + rank;
            run_idx[j] = b;
            n_inf_out[j] = n_inf;
            n_kv_out[j] = n_kv;
            row_off[j] = pre_rows + incl - n_inf;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int c = 0, r = 0;
            for (int w = 0; w < nwarps; ++w) { c += w_cnt[w]; r += w_rows[w]; }
            carry[0] += c; carry[1] += r;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) { *run_count = carry[0]; row_off[carry[0]] = carry[1]; }
}

__global__ void __launch_bounds__(kThreads)
alg1_commit_kernel(rstitch_alg1_state_t s, int B, int model, const int32_t *run_idx, const int32_t *run_count,
                   const int32_t *row_off, const int32_t *tok, const uint8_t *mask, int32_t eos_id)
{
    const int n = *run_count;
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
        const int b = run_idx[j];
        if (b < 0 || b >= B) continue;
        const int row = row_off ? row_off[j + 1] - 1 : j;      // a prefill yields its token at the end of the span
        const int32_t yt = tok[row];
        if (mask[j]) {                                         // H_t > tau
            if (model == 0) {                                  // SLM -> LLM: discard, roll the cache back
                s.kv_slm[b] -= 1;
                s.active[b] = 1;
                continue;
            }                                                  // on the LLM: keep decoding with it
        } else if (model == 1) {
            s.active[b] = 0;                                   // LLM -> SLM
        }
        const int k = s.n_out[b];
        if (k < s.y_cap) s.y[(size_t)b * s.y_cap + k] = yt;    // append y_t
        s.n_out[b] = k + 1;
        s.seq_len[b] += 1;
        s.kept[model * B + b] += 1;
        if (yt == eos_id) s.done[b] = 1;
    }
}

bool state_ok(const rstitch_alg1_state_t *s)
{
    return s && s->active && s->kv_slm && s->kv_llm && s->seq_len && s->n_out && s->done && s->iters && s->kept &&
           s->steps && s->lat_ms && s->y && s->y_cap > 0;
}

}  // namespace

extern "C" {

int rstitch_alg1_init(const rstitch_alg1_state_t *s, int B, const int32_t *prompt_len, void *cuda_stream)
{
    if (B < 0 || !state_ok(s) || (B > 0 && !prompt_len)) return RSTITCH_ERR_INVALID_ARG;
    if (B == 0) return RSTITCH_OK;
    int grid = (B + kThreads - 1) / kThreads;
    if (grid > 1024) grid = 1024;
    alg1_init_kernel<<<grid, kThreads, 0, (cudaStream_t)cuda_stream>>>(*s, B, prompt_len);
    if (cudaGetLastError() != cudaSuccess) return RSTITCH_ERR_CUDA;
    return RSTITCH_OK;
}

int rstitch_alg1_plan(const rstitch_alg1_state_t *s, int B, int model, int t_max,
                      const rstitch_latency_model_t *latency, int32_t *run_idx, int32_t *run_count,
                      int32_t *n_inf, int32_t *n_kv, int32_t *row_off, void *cuda_stream)
{
    if (B < 0 || !state_ok(s) || (model != 0 && model != 1) || t_max < 0 || !latency || !run_count || !row_off)
        return RSTITCH_ERR_INVALID_ARG;
    if (B > 0 && (!run_idx || !n_inf || !n_kv)) return RSTITCH_ERR_INVALID_ARG;
    if (!std::isfinite(latency->a) || !std::isfinite(latency->b) || !std::isfinite(latency->c) ||
        !std::isfinite(latency->d))
        return RSTITCH_ERR_INVALID_ARG;
    alg1_plan_kernel<<<1, kThreads, 0, (cudaStream_t)cuda_stream>>>(*s, B, model, t_max, *latency, run_idx,
                                                                   run_count, n_inf, n_kv, row_off);
    if (cudaGetLastError() != cudaSuccess) return RSTITCH_ERR_CUDA;
    return RSTITCH_OK;
}

int rstitch_alg1_commit(const rstitch_alg1_state_t *s, int B, int model, const int32_t *run_idx,
                        const int32_t *run_count, const int32_t *row_off, const int32_t *tok,
                        const uint8_t *route_mask, int32_t eos_id, void *cuda_stream)
{
    if (B < 0 || !state_ok(s) || (model != 0 && model != 1) || !run_count) return RSTITCH_ERR_INVALID_ARG;
    if (B > 0 && (!run_idx || !tok || !route_mask)) return RSTITCH_ERR_INVALID_ARG;
    if (B == 0) return RSTITCH_OK;
    int grid = (B + kThreads - 1) / kThreads;
    if (grid > 1024) grid = 1024;
    alg1_commit_kernel<<<grid, kThreads, 0, (cudaStream_t)cuda_stream>>>(*s, B, model, run_idx, run_count, row_off,
                                                                        tok, route_mask, eos_id);
    if (cudaGetLastError() != cudaSuccess) return RSTITCH_ERR_CUDA;
    return RSTITCH_OK;
}

}  // extern "C"
