// Device-side steps of Algorithm 1 either side of the routing decision, written for one thread block so
// that they can run as kernels of their own (rstitch_alg1.cu) or at the end of a routing call, in the
// block that has just produced the tokens and the mask (rstitch_tail.cuh).
#pragma once
#include "../../include/rstitch.h"
#include <cuda_runtime.h>

namespace rstitch {

// What a routing call needs to carry Algorithm 1 on from its own decision (device copy of
// rstitch_alg1_tail_t).  on = 0: nothing to do.
struct Alg1Tail {
    int on;
    rstitch_alg1_state_t s;
    int n_seq, model;
    const int32_t *run_idx, *run_count, *row_off;
    int32_t eos_id;
    int plan_next, t_max;
    rstitch_latency_model_t lat[2];
    int32_t *nx_idx[2], *nx_cnt[2], *nx_ninf[2], *nx_nkv[2], *nx_off[2];
};

// Algorithm 1 from "if H_t > tau" to the EOS test for run entries first, first + stride, ... of one model's
// batch: entry j is sequence run_idx[j], its token sits in the last row of its span.
__device__ inline void alg1_commit_entries(const rstitch_alg1_state_t &s, int B, int model, const int32_t *run_idx,
                                           int n, const int32_t *row_off, const int32_t *tok, const uint8_t *mask,
                                           int32_t eos_id, int first, int stride)
{
    for (int j = first; j < n; j += stride) {
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

// The prefill-or-decode test for one model, by one whole block (at most 512 threads; every thread calls).
// Sequences are taken in chunks of blockDim.x; inside a chunk a ballot gives each selected sequence its rank
// within the warp, warp totals are scanned in shared memory and a carry links the chunks, so run_idx comes
// out ascending and row_off is the exclusive scan of n_inf in that order.  smem: 34 ints.
__device__ inline void alg1_plan_block(const rstitch_alg1_state_t &s, int B, int model, int t_max,
                                       const rstitch_latency_model_t &lat, int32_t *run_idx, int32_t *run_count,
                                       int32_t *n_inf_out, int32_t *n_kv_out, int32_t *row_off, int *smem)
{
    int *w_cnt = smem, *w_rows = smem + 16, *carry = smem + 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    int32_t *kv = model == 0 ? s.kv_slm : s.kv_llm;
    __syncthreads();
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
    __syncthreads();
}

// After a routing call's own tail: this model's decision block, then (plan_next) the next round's
// planning for both models.  Every thread of the block calls; tok and mask are the call's outputs.
__device__ inline void alg1_tail_block(const Alg1Tail &a, const int32_t *tok, const uint8_t *mask, int *smem)
{
    __syncthreads();                     // the block's own tok / mask stores are visible to all its threads
    const int n = *a.run_count;
    alg1_commit_entries(a.s, a.n_seq, a.model, a.run_idx, n, a.row_off, tok, mask, a.eos_id, (int)threadIdx.x,
                        (int)blockDim.x);
    if (!a.plan_next) return;
    for (int m = 0; m < 2; ++m)          // all commits of this round are done: plan the next one
        alg1_plan_block(a.s, a.n_seq, m, a.t_max, a.lat[m], a.nx_idx[m], a.nx_cnt[m], a.nx_ninf[m], a.nx_nkv[m],
                        a.nx_off[m], smem);
}

}  // namespace rstitch
