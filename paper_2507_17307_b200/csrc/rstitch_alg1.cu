// The steps of Algorithm 1 either side of the routing decision, batched: per-sequence state kept on
// the device (active model, the two KV-cache sizes, sequence length, generated tokens) and two small
// kernels per model and iteration.
//   plan:   which sequences run on this model now, how many tokens each must process (prefill of
//           the missing span, or one decode token), the row offsets of that batch, the KV-size
//           update, and the latency estimate of Eq. 5 accumulated per sequence;
//   commit: the decision block after the entropy test -- discard and roll back on an SLM hand-off,
//           hand back from the LLM on low entropy, append the token, stop on EOS.
// Integer work on B elements; one block, warp ballots and prefix sums for the ordered run list.
#include "rstitch_alg1.cuh"
#include "rstitch_kernels.cuh"

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

// One block: see alg1_plan_block.
__global__ void __launch_bounds__(kThreads)
alg1_plan_kernel(rstitch_alg1_state_t s, int B, int model, int t_max, rstitch_latency_model_t lat,
                 int32_t *run_idx, int32_t *run_count, int32_t *n_inf_out, int32_t *n_kv_out, int32_t *row_off)
{
    __shared__ int smem[34];
    rstitch::alg1_plan_block(s, B, model, t_max, lat, run_idx, run_count, n_inf_out, n_kv_out, row_off, smem);
}

__global__ void __launch_bounds__(kThreads)
alg1_commit_kernel(rstitch_alg1_state_t s, int B, int model, const int32_t *run_idx, const int32_t *run_count,
                   const int32_t *row_off, const int32_t *tok, const uint8_t *mask, int32_t eos_id)
{
    rstitch::alg1_commit_entries(s, B, model, run_idx, *run_count, row_off, tok, mask, eos_id,
                                 (int)(blockIdx.x * blockDim.x + threadIdx.x), (int)(gridDim.x * blockDim.x));
}

// The block a routing call would have run after its own tail, for a call that has no rows to evaluate.
__global__ void __launch_bounds__(kThreads)
alg1_tail_kernel(rstitch::Alg1Tail a, const int32_t *tok, const uint8_t *mask)
{
    __shared__ int smem[34];
    rstitch::alg1_tail_block(a, tok, mask, smem);
}

bool state_ok(const rstitch_alg1_state_t *s)
{
    return s && s->active && s->kv_slm && s->kv_llm && s->seq_len && s->n_out && s->done && s->iters && s->kept &&
           s->steps && s->lat_ms && s->y && s->y_cap > 0;
}

}  // namespace

namespace rstitch {

bool alg1_state_ok(const rstitch_alg1_state_t *s) { return state_ok(s); }

cudaError_t launch_alg1_tail(const Alg1Tail &a, const int32_t *tok, const uint8_t *mask, cudaStream_t stream)
{
    alg1_tail_kernel<<<1, kThreads, 0, stream>>>(a, tok, mask);
    return cudaGetLastError();
}

}  // namespace rstitch

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
