// Cross-CTA finalisation of the head kernels and the routing tail (S2-S6), run by ONE thread
// block: the block that drew the last ticket of a head kernel, or the single block of the
// stand-alone compaction kernel.  No block ever waits on another, so nothing here can hang.
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

// Writes ent_out / tok_out of one row from its merged statistics.
__device__ __forceinline__ void tail_emit_row(const Stats &t, int r, const TailArgs &a)
{
    if (a.shard_stats) {
        float *o = a.shard_stats + (size_t)r * kShardWords;
        const bool found = !(t.bi == INT_MAX || t.bi < 0 || t.bi >= a.V);
        o[0] = t.m; o[1] = t.s; o[2] = t.u; o[3] = t.bv;
        o[4] = __int_as_float(found ? t.bi + a.v_base : INT_MAX);
        return;
    }
    float H = logf(t.s) - t.u / t.s;
    if (H < 0.f) H = 0.f;                      // rounding below zero; NaN stays NaN
    a.ent_out[r] = H;
    a.tok_out[r] = (t.bi == INT_MAX || t.bi < 0 || t.bi >= a.V) ? 0 : t.bi;
    if (H != H) atomicAdd(&a.stat->nan_rows, 1u);
}

// Merge of slices part, part + parts, ... of one row by one thread, loads issued four at a time.
__device__ __forceinline__ Stats tail_merge_strided(const Partials &P, size_t row_base, int n_slices,
                                                    int part, int parts)
{
    Stats t = stats_empty();
    int c = part;
    for (; c + 3 * parts < n_slices; c += 4 * parts) {
        Stats p0 = partial_load(P, row_base + c);
        Stats p1 = partial_load(P, row_base + c + parts);
        Stats p2 = partial_load(P, row_base + c + 2 * parts);
        Stats p3 = partial_load(P, row_base + c + 3 * parts);
        stats_merge(p0, p1);
        stats_merge(p2, p3);
        stats_merge(p0, p2);
        stats_merge(t, p0);
    }
    for (; c < n_slices; c += parts) {
        Stats p = partial_load(P, row_base + c);
        stats_merge(t, p);
    }
    return t;
}

// Merge the n_slices partials of every row in a fixed order and write ent_out / tok_out.  A row is
// shared by `parts` adjacent lanes (a power of two, as many as the block can spare for the row
// count), each taking a strided subset of the slices; a butterfly over the group finishes the row.
__device__ inline void tail_finalize_rows(const Partials &P, int n_slices, const TailArgs &a)
{
    int parts = 32;
    while (parts > 1 && a.R * parts > (int)blockDim.x) parts >>= 1;
    const int rows_per_pass = (int)blockDim.x / parts;
    const int part = threadIdx.x & (parts - 1);
    const int sub = threadIdx.x / parts;
    const bool in_pass = sub < rows_per_pass;          // blockDim.x need not be a multiple of parts
    for (int r0 = 0; r0 < a.R; r0 += rows_per_pass) {
        const int r = r0 + sub;
        const bool act = in_pass && r < a.R;
        Stats t = act ? tail_merge_strided(P, (size_t)r * n_slices, n_slices, part, parts) : stats_empty();
        for (int o = parts >> 1; o > 0; o >>= 1) {     // whole warp takes part: same trip count everywhere
            Stats p = stats_shfl_xor(t, o);
            stats_merge(t, p);
        }
        if (act && part == 0) tail_emit_row(t, r, a);
    }
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
            const float dm = m[k] - M, e = __expf(dm);
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

// Finalisation for a handful of rows and at most 256 slices: one warp per row.
__device__ inline void tail_finalize_rows_direct(const Partials &P, int n_slices, const TailArgs &a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int r = warp; r < a.R; r += nwarps) {
        const Stats t = tail_row_direct(P, (size_t)r * n_slices, n_slices, lane);
        if (lane == 0) tail_emit_row(t, r, a);
    }
}

// The same finalisation for many rows (tensor-core kernel, up to 128 rows x ~150 slices), where
// fetching the partials straight from L2 is a chain of dependent round trips.  The partials of a
// group of rows are first brought into shared memory with five bulk copies (one per statistics
// array; the rows of a group are contiguous in each), then merged from there without a dependent
// chain: pass 1 takes the row maximum M and the greedy token, pass 2 sums e^{m_i - M} s_i and
// e^{m_i - M} (u_i + (m_i - M) s_i), one exponential per partial.
//   stage / stage_bytes: free shared memory (16-byte aligned); bar: an initialised mbarrier
//   (count 1) whose completed phases so far number bar_phase.
// Returns false if a bounded wait ran out (the caller records it).
__device__ inline bool tail_finalize_rows_staged(const Partials &P, int n_slices, const TailArgs &a,
                                                 unsigned char *stage, uint32_t stage_bytes, uint64_t *bar,
                                                 uint32_t bar_phase, volatile int *abort_flag)
{
    int parts = 32;
    while (parts > 1 && a.R * parts > (int)blockDim.x) parts >>= 1;
    const int part = threadIdx.x & (parts - 1);
    const int sub = threadIdx.x / parts;
    const uint32_t row_bytes = (uint32_t)n_slices * 4u;
    int group = stage_bytes > 80u ? (int)((stage_bytes - 80u) / 5u / row_bytes) & ~3 : 0;   // rows per group
    if (group > (int)blockDim.x / parts) group = ((int)blockDim.x / parts) & ~3;
    if (group < 4) {                                                     // no room to stage: read from L2
        tail_finalize_rows(P, n_slices, a);
        return true;
    }
    const uint32_t region = (((uint32_t)group * row_bytes + 15u) & ~15u);
    const float *sm_m = (const float *)(stage);
    const float *sm_s = (const float *)(stage + region);
    const float *sm_u = (const float *)(stage + 2 * region);
    const float *sm_bv = (const float *)(stage + 3 * region);
    const int   *sm_bi = (const int *)(stage + 4 * region);
    const uint32_t bar_u32 = ptx::smem_u32(bar);
    bool ok = true;
    for (int g0 = 0; g0 < a.R; g0 += group, ++bar_phase) {
        const int rows = (a.R - g0) < group ? (a.R - g0) : group;
        if (threadIdx.x == 0) {
            const uint32_t bytes = (((uint32_t)rows * row_bytes + 15u) & ~15u);
            const size_t off = (size_t)g0 * n_slices;
            ptx::fence_proxy_async_all();       // the partials were written with ordinary stores
            ptx::mbar_arrive_expect_tx(bar_u32, 5u * bytes);
            ptx::bulk_g2s(ptx::smem_u32(sm_m), P.m + off, bytes, bar_u32);
            ptx::bulk_g2s(ptx::smem_u32(sm_s), P.s + off, bytes, bar_u32);
            ptx::bulk_g2s(ptx::smem_u32(sm_u), P.u + off, bytes, bar_u32);
            ptx::bulk_g2s(ptx::smem_u32(sm_bv), P.bv + off, bytes, bar_u32);
            ptx::bulk_g2s(ptx::smem_u32(sm_bi), P.bi + off, bytes, bar_u32);
        }
        if (!ptx::mbar_wait(bar_u32, bar_phase & 1u, abort_flag)) ok = false;
        const int r = g0 + sub;
        const bool act = ok && sub < rows;
        const int base = sub * n_slices;
        float M = -CUDART_INF_F, bv = -CUDART_INF_F;
        int bi = INT_MAX;
        if (act)
            for (int c = part; c < n_slices; c += parts) {
                M = fmaxf(M, sm_m[base + c]);
                argmax_take(bv, bi, sm_bv[base + c], sm_bi[base + c]);
            }
        for (int o = parts >> 1; o > 0; o >>= 1) {
            M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
            float obv = __shfl_xor_sync(0xffffffffu, bv, o);
            int obi = __shfl_xor_sync(0xffffffffu, bi, o);
            argmax_take(bv, bi, obv, obi);
        }
        float ss = 0.f, uu = 0.f;
        if (act)
            for (int c = part; c < n_slices; c += parts) {
                const float mi = sm_m[base + c];
                if (mi != -CUDART_INF_F) {
                    const float dm = mi - M, e = __expf(dm), si = sm_s[base + c];
                    ss = fmaf(e, si, ss);
                    uu = fmaf(e, fmaf(dm, si, sm_u[base + c]), uu);
                }
            }
        for (int o = parts >> 1; o > 0; o >>= 1) {
            ss += __shfl_xor_sync(0xffffffffu, ss, o);
            uu += __shfl_xor_sync(0xffffffffu, uu, o);
        }
        if (act && part == 0) {
            Stats t;
            t.m = M; t.s = ss; t.u = uu; t.bv = bv; t.bi = bi;
            tail_emit_row(t, r, a);
        }
        __syncthreads();                        // the stage is reused by the next group
    }
    return ok;
}

// Eq. 2 / Algorithm 1: mask = H > tau (strict); a NaN entropy routes to the LLM.
__device__ __forceinline__ uint8_t rule(float H, float tau)
{
    return (H != H || H > tau) ? 1 : 0;
}

// S4: per-sequence mask from per-row entropies already in global memory (written by this block).
__device__ inline void tail_mask(const TailArgs &a)
{
    if (a.row_seq == nullptr) {
        for (int b = threadIdx.x; b < a.B; b += blockDim.x)
            a.route_mask[b] = (b < a.R) ? rule(a.ent_out[b], a.tau) : 0;
    } else {
        for (int b = threadIdx.x; b < a.B; b += blockDim.x) a.route_mask[b] = 0;
        __syncthreads();
        for (int r = threadIdx.x; r < a.R; r += blockDim.x) {
            int sq = a.row_seq[r];
            bool last = (r == a.R - 1) || (a.row_seq[r + 1] != sq);
            if (last && sq >= 0 && sq < a.B) a.route_mask[sq] = rule(a.ent_out[r], a.tau);
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
__device__ inline void tail_route_warp(const TailArgs &a)
{
    if (threadIdx.x >= 32) return;
    const int b = threadIdx.x;
    const bool in = b < a.B;
    const bool routed = in && b < a.R && rule(a.ent_out[b], a.tau) != 0;
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

__device__ inline void tail_route(const TailArgs &a, int *smem)
{
    if (a.shard_stats) return;                       // a vocabulary shard decides nothing
    if (a.B <= 32 && a.row_seq == nullptr) {
        tail_route_warp(a);
    } else {
        tail_mask(a);
        tail_compact(a.route_mask, a.B, a.seq_len, a.kv_len, a.llm_idx, a.llm_count, a.llm_span,
                     a.llm_row_off, a.stat, smem);
    }
    if (a.alg1.on) alg1_tail_block(a.alg1, a.tok_out, a.route_mask, smem);
    if (a.mirror_dst) {
        __syncthreads();             // the block's own output stores; other blocks' came before the ticket
        for (uint32_t i = threadIdx.x; i < a.mirror_vec; i += blockDim.x) a.mirror_dst[i] = __ldcg(a.mirror_src + i);
    }
}

}  // namespace rstitch
