// Cross-block merge of the head kernels' partial statistics and the routing tail (S2-S6).  The merge is
// one warp per row (head_finalize_kernel); the tail is run by ONE thread block: the block of that kernel
// (or of the shard-merge kernel) that drew the last ticket, or the single block of the stand-alone
// compaction kernel.  No block ever waits on another, so nothing here can hang.
#pragma once
#include "rstitch_stats.cuh"
#include "rstitch_ptx.cuh"
#include "rstitch_alg1.cuh"
#include <stdint.h>

namespace rstitch {

// Device status word; mirrors rstitch_devstat_t field by field.
struct DevStat {
    unsigned nan_rows, bad_row_idx, bad_span, timeouts, timeout_site, launches, r0, r1;
};

// Per-(row, slice) partial statistics in scratch memory, structure of arrays, [R][n_slices].
struct Partials {
    float *m, *s, *u, *bv;
    int   *bi;
};

__host__ __device__ inline size_t partials_bytes(size_t R, size_t n_slices)
{
    size_t one = ((R * n_slices * 4 + 255) / 256) * 256;
    return 5 * one;
}

__host__ __device__ inline Partials partials_carve(void *base, size_t R, size_t n_slices)
{
    size_t one = ((R * n_slices * 4 + 255) / 256) * 256;
    char *p = (char *)base;
    Partials q;
    q.m  = (float *)(p);
    q.s  = (float *)(p + one);
    q.u  = (float *)(p + 2 * one);
    q.bv = (float *)(p + 3 * one);
    q.bi = (int *)(p + 4 * one);
    return q;
}

__device__ __forceinline__ void partial_store(const Partials &P, size_t at, const Stats &t)
{
    P.m[at] = t.m; P.s[at] = t.s; P.u[at] = t.u; P.bv[at] = t.bv; P.bi[at] = t.bi;
}

__device__ __forceinline__ Stats partial_load(const Partials &P, size_t at)
{
    Stats t;                     // written by other blocks of this launch: bypass L1
    t.m = __ldcg(P.m + at); t.s = __ldcg(P.s + at); t.u = __ldcg(P.u + at);
    t.bv = __ldcg(P.bv + at); t.bi = __ldcg(P.bi + at);
    return t;
}

struct TailArgs {
    int R, B;                    // rows evaluated, sequences decided (already clamped to the live count)
    int V;
    float tau;                   // nats
    const int32_t *row_seq;      // optional [R]
    const int32_t *seq_len, *kv_len;   // optional [B]
    int32_t *tok_out;            // [R]
    float   *ent_out;            // [R]
    uint8_t *route_mask;         // [B]
    int32_t *llm_idx, *llm_count;
    int32_t *llm_span, *llm_row_off;   // optional
    DevStat *stat;
    // Vocabulary-shard mode: when shard_stats is set the head covers only entries [v_base, v_base + V) of
    // the vocabulary; each row's merged statistics go out as five words (m, s, u, best score, global
    // index of the best entry) and nothing is decided: shard_merge_kernel does that on the gathered shards.
    float   *shard_stats;        // [R][5] or nullptr
    int      v_base;
    Alg1Tail alg1;               // optional: Algorithm 1's decision block (and the next round's plans) after S6
    // Host-buffer calls: after everything else the deciding block copies the call's outputs (one contiguous
    // piece of device memory, a multiple of 16 bytes) to pinned host memory mapped into the device's address
    // space, which saves the device-to-host copy command and its latency.  nullptr: no copy.
    const uint4 *mirror_src;
    uint4       *mirror_dst;
    uint32_t     mirror_vec;     // number of 16-byte words
};

constexpr int kShardWords = 5;

// Writes ent_out / tok_out of one row from its merged statistics; returns the entropy.
__device__ __forceinline__ float tail_emit_row(const Stats &t, int r, const TailArgs &a)
{
    if (a.shard_stats) {
        float *o = a.shard_stats + (size_t)r * kShardWords;
        const bool found = !(t.bi == INT_MAX || t.bi < 0 || t.bi >= a.V);
        o[0] = t.m; o[1] = t.s; o[2] = t.u; o[3] = t.bv;
        o[4] = __int_as_float(found ? t.bi + a.v_base : INT_MAX);
        return 0.f;
    }
    float H = logf(t.s) - t.u / t.s;
    if (H < 0.f) H = 0.f;                      // rounding below zero; NaN stays NaN
    a.ent_out[r] = H;
    a.tok_out[r] = (t.bi == INT_MAX || t.bi < 0 || t.bi >= a.V) ? 0 : t.bi;
    if (H != H) atomicAdd(&a.stat->nan_rows, 1u);
    return H;
}

// One row's n_slices <= 256 partials merged by one warp: every partial of the row is pulled into
// registers with all loads in flight at once (a single round trip to L2), then merged without a
// dependent chain: the row maximum M and the greedy token first, then one exponential per partial for
// the sums.  Every lane returns the merged statistics.
__device__ __forceinline__ Stats tail_row_direct(const Partials &P, size_t base, int n_slices, int lane)
{
    float m[8], s[8], u[8], bv[8];
    int bi[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int c = lane + 32 * k;
        const bool in = c < n_slices;
        const size_t at = base + (in ? c : 0);
        m[k]  = in ? __ldcg(P.m + at)  : -CUDART_INF_F;
        s[k]  = in ? __ldcg(P.s + at)  : 0.f;
        u[k]  = in ? __ldcg(P.u + at)  : 0.f;
        bv[k] = in ? __ldcg(P.bv + at) : -CUDART_INF_F;
        bi[k] = in ? __ldcg(P.bi + at) : INT_MAX;
    }
    float M = -CUDART_INF_F, best = -CUDART_INF_F;
    int besti = INT_MAX;
#pragma unroll
    for (int k = 0; k < 8; ++k) { M = fmaxf(M, m[k]); argmax_take(best, besti, bv[k], bi[k]); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float obv = __shfl_xor_sync(0xffffffffu, best, o);
        int obi = __shfl_xor_sync(0xffffffffu, besti, o);
        argmax_take(best, besti, obv, obi);
    }
    float ss = 0.f, uu = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k)
        if (m[k] != -CUDART_INF_F) {
            const float dm = m[k] - M, e = exp_approx(dm);
            ss = fmaf(e, s[k], ss);
            uu = fmaf(e, fmaf(dm, s[k], u[k]), uu);
        }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ss += __shfl_xor_sync(0xffffffffu, ss, o);
        uu += __shfl_xor_sync(0xffffffffu, uu, o);
    }
    Stats t;
    t.m = M; t.s = ss; t.u = uu; t.bv = best; t.bi = besti;
    return t;
}

// Eq. 2 / Algorithm 1: mask = H > tau (strict); a NaN entropy routes to the LLM.
__device__ __forceinline__ uint8_t rule(float H, float tau)
{
    return (H != H || H > tau) ? 1 : 0;
}

// S4: per-sequence mask from the per-row entropies: ent is a.ent_out (global memory, written before the
// block's last barrier) or the block's own copy of it in shared memory.  With mask_stage (shared memory,
// a.B bytes) the mask is also kept there for the compaction, which then reads nothing back from global.
__device__ inline void tail_mask(const TailArgs &a, const float *ent, uint8_t *mask_stage)
{
    if (a.row_seq == nullptr) {
        for (int b = threadIdx.x; b < a.B; b += blockDim.x) {
            const uint8_t m = (b < a.R) ? rule(ent[b], a.tau) : 0;
            a.route_mask[b] = m;
            if (mask_stage) mask_stage[b] = m;
        }
    } else {
        uint8_t *mk = mask_stage ? mask_stage : a.route_mask;
        for (int b = threadIdx.x; b < a.B; b += blockDim.x) mk[b] = 0;
        __syncthreads();
        for (int r = threadIdx.x; r < a.R; r += blockDim.x) {
            int sq = a.row_seq[r];
            bool last = (r == a.R - 1) || (a.row_seq[r + 1] != sq);
            if (last && sq >= 0 && sq < a.B) mk[sq] = rule(ent[r], a.tau);
        }
        if (mask_stage) {
            __syncthreads();
            for (int b = threadIdx.x; b < a.B; b += blockDim.x) a.route_mask[b] = mask_stage[b];
        }
    }
    __syncthreads();
}

// S5 + S6 by one block: chunks of blockDim.x sequences; inside a chunk a warp ballot gives each
// routed sequence its rank in the warp, per-warp totals are scanned in shared memory, and a
// running carry links the chunks, so llm_idx comes out ascending.  Spans get the same treatment
// with an inclusive warp scan.  smem: at least 2 * 32 + 2 ints.
__device__ inline void tail_compact(const uint8_t *mask, int B, const int32_t *seq_len,
                                    const int32_t *kv_len, int32_t *llm_idx, int32_t *llm_count,
                                    int32_t *llm_span, int32_t *llm_row_off, DevStat *stat,
                                    int *smem /* >= 66 ints */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    int *w_cnt = smem, *w_rows = smem + 32, *carry = smem + 64;     // carry[0] = count, carry[1] = rows
    if (threadIdx.x == 0) { carry[0] = 0; carry[1] = 0; }
    __syncthreads();
    const bool spans = (seq_len != nullptr);
    for (int base = 0; base < B; base += blockDim.x) {
        int b = base + threadIdx.x;
        bool routed = (b < B) && (mask[b] != 0);
        unsigned ball = __ballot_sync(0xffffffffu, routed);
        int rank = __popc(ball & ((1u << lane) - 1u));
        int span = 0, incl = 0;
        if (spans) {
            if (routed) {
                span = seq_len[b] - kv_len[b];
                if (span < 1) atomicAdd(&stat->bad_span, 1u);
            }
            incl = span;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
        }
        if (lane == 31) { w_cnt[warp] = __popc(ball); w_rows[warp] = incl; }
        __syncthreads();
        int pre_cnt = carry[0], pre_rows = carry[1];
        for (int w = 0; w < warp; ++w) { pre_cnt += w_cnt[w]; pre_rows += w_rows[w]; }
        if (routed) {
            int j = pre_cnt + rank;
            llm_idx[j] = b;
            if (spans) { llm_span[j] = span; llm_row_off[j] = pre_rows + incl - span; }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int c = 0, rws = 0;
            for (int w = 0; w < nwarps; ++w) { c += w_cnt[w]; rws += w_rows[w]; }
            carry[0] += c; carry[1] += rws;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        *llm_count = carry[0];
        if (spans) llm_row_off[carry[0]] = carry[1];
    }
}

// S4-S6 for at most 32 sequences decided row by row: one warp, ballots and shuffles, no block barrier.
// The entropies were written by this block before its last barrier.
__device__ inline void tail_route_warp(const TailArgs &a, const float *ent)
{
    if (threadIdx.x >= 32) return;
    const int b = threadIdx.x;
    const bool in = b < a.B;
    const bool routed = in && b < a.R && rule(ent[b], a.tau) != 0;
    if (in) a.route_mask[b] = routed ? 1 : 0;
    const unsigned ball = __ballot_sync(0xffffffffu, routed);
    const int rank = __popc(ball & ((1u << b) - 1u));
    const bool spans = (a.seq_len != nullptr);
    int span = 0, incl = 0;
    if (spans) {
        if (routed) {
            span = a.seq_len[b] - a.kv_len[b];
            if (span < 1) atomicAdd(&a.stat->bad_span, 1u);
        }
        incl = span;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (b >= o) incl += v;
        }
    }
    if (routed) {
        a.llm_idx[rank] = b;
        if (spans) { a.llm_span[rank] = span; a.llm_row_off[rank] = incl - span; }
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    if (b == 0) {
        *a.llm_count = __popc(ball);
        if (spans) a.llm_row_off[__popc(ball)] = total;
    }
}

// ent_stage / mask_stage (optional, shared memory): the block's own copy of the a.R entropies it has just
// written, and room for a.B mask bytes; without them both are read back from global memory.
__device__ inline void tail_route(const TailArgs &a, int *smem, const float *ent_stage = nullptr,
                                  uint8_t *mask_stage = nullptr)
{
    if (a.shard_stats) return;                       // a vocabulary shard decides nothing
    const float *ent = ent_stage ? ent_stage : a.ent_out;
    if (a.B <= 32 && a.row_seq == nullptr) {
        tail_route_warp(a, ent);
    } else {
        tail_mask(a, ent, mask_stage);
        tail_compact(mask_stage ? mask_stage : a.route_mask, a.B, a.seq_len, a.kv_len, a.llm_idx, a.llm_count,
                     a.llm_span, a.llm_row_off, a.stat, smem);
    }
    if (a.alg1.on) alg1_tail_block(a.alg1, a.tok_out, a.route_mask, smem);
    if (a.mirror_dst) {
        __syncthreads();             // the block's own output stores; other blocks' came before the ticket
        for (uint32_t i = threadIdx.x; i < a.mirror_vec; i += blockDim.x) a.mirror_dst[i] = __ldcg(a.mirror_src + i);
    }
}

}  // namespace rstitch
