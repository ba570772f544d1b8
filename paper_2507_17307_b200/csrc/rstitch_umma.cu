// Tensor-core LM-head kernel (S1-S3 fused): hidden rows on the M side of tcgen05.mma, vocabulary
// on the N side, fp32 accumulators in tensor memory, and an epilogue that turns each accumulator
// tile into single-pass softmax statistics and the greedy token without the logits ever leaving
// the SM.
//
// head_umma_kernel (at most 128 rows: one M tile).  Block = 10 warps, one block per SM:
//   warp 0  producer: one thread issues tensor-map (TMA) copies of the hidden tile and an N x 64 W_head
//           tile (128-byte swizzle) into a shared-memory ring of up to eight stages, two k-steps at a time;
//   warp 1  one thread issues the tcgen05.mma instructions (M = 128 or 64, N <= 256, K = 16) and commits
//           them to the ring's "empty" barriers and to the accumulator's "full" barrier; the warp
//           also owns the tensor-memory allocation (512 columns = two 256-column accumulators);
//   warps 2-9  epilogue: thread = one hidden row (one TMEM lane); it reads its row of the accumulator
//           32 columns at a time and folds the logits into (m, s, u, argmax); warps 2-5 take the first
//           half of a tile's columns, warps 6-9 the second.
// The two accumulators alternate, so the epilogue of one tile runs under the MMAs of the next.
// Each block owns one contiguous, balanced range of the vocabulary, cut into tiles of at most 256 rows,
// and keeps one running statistic per row; W_head is read from HBM exactly once and the kernel is
// HBM-bound.
//
// head_umma2_kernel (more rows): work items are (256-row vocabulary tile, pair of 128-row M tiles) dealt
// round-robin with the pairs of one vocabulary tile adjacent, so that they run at the same time on
// neighbouring SMs and W_head comes from HBM once and from L2 for the others; see the comment there.
#include "rstitch_kernels.cuh"
#include "rstitch_ptx.cuh"

#include <cuda.h>
#include <cstring>

namespace rstitch {

namespace {

constexpr int kProducers = 1;                        // copy-issuing warps of the many-row kernels.  One thread issues ~7
                                                     // tensor-map copies per microsecond and separate warps issue in
                                                     // parallel (a probe reached 19/us with four), but these kernels need at
                                                     // most ~6/us and measured the same with 1, 2 and 3; their dealing code
                                                     // stays general
// k-steps whose copies the one-M-tile kernel issues together.  Measured on the 3584 x 152064 head with 16
// rows: 1 -> 197 us, 2 -> 181 us, 4 -> 200 us (a group needs that many free stages at once; with eight
// stages a group of four leaves too little in flight).
constexpr int kIssueGroup = 2;
constexpr int kEpiWarps  = 8;
constexpr int kThreads   = 64 + kEpiWarps * 32;      // head_umma_kernel: producer, MMA, 8 epilogue warps
constexpr int kMaxStages = 8;
constexpr int kTileM     = 128;
constexpr int kTileNMax  = 256;
constexpr int kTileK     = 64;                       // bf16 elements = one 128-byte swizzle row
constexpr int kABytes    = kTileM * kTileK * 2;      // 16 KB
constexpr int kBBytes    = kTileNMax * kTileK * 2;   // 32 KB
constexpr int kRingBytes = 224 * 1024;                     // cut into as many stages as fit
constexpr int kDynSmem   = kRingBytes + 1024;              // + slack to align the ring to 1024 B
constexpr int kTmemCols  = 512;

struct Item { int v0, N; };

// The W tile head_umma_kernel's block takes at its j-th iteration; identical in every role of the block.
// Each block owns a balanced contiguous vocabulary range in units of 16 rows, cut into n_tiles tiles.
struct Schedule {
    int u_begin, nu, n_tiles;
    int n_items;

    // tiles_per_block: the same for every block (from the largest range), so that no block's
    // tile exceeds the tile size the shared-memory stages were laid out for
    __device__ void init(int V, int grid, int cta, int tiles_per_block)
    {
        long long units = (V + 15) / 16;
        u_begin = (int)(units * cta / grid);
        int u_end = (int)(units * (cta + 1) / grid);
        nu = u_end - u_begin;
        n_tiles = tiles_per_block;
        n_items = n_tiles;
    }
    __device__ Item item(int j) const
    {
        Item it;
        int a = u_begin + (int)((long long)nu * j / n_tiles);
        int b = u_begin + (int)((long long)nu * (j + 1) / n_tiles);
        it.v0 = a * 16; it.N = (b - a) * 16;
        return it;
    }
};

__device__ __forceinline__ void raise_abort(volatile int *flag, DevStat *stat, unsigned site)
{
    *flag = 1;
    atomicAdd(&stat->timeouts, 1u);
    atomicExch(&stat->timeout_site, site);
}

// Fold 32 logits (columns c0 .. c0+31 of the tile, vocabulary index vbase + column) into the row's
// statistics: one rescale of the running sums per chunk, then one ex2 per logit.  Four independent
// partial maxima / sums keep the dependent chains short: an epilogue warp has a scheduler to itself,
// so instruction-level parallelism is all the latency hiding there is.
__device__ __forceinline__ void fold_chunk_full(Stats &st, const float (&z)[32], int vbase, const SampleArgs &sa,
                                                uint32_t row)
{
    float c0 = fmaxf(z[0], z[4]), c1 = fmaxf(z[1], z[5]), c2 = fmaxf(z[2], z[6]), c3 = fmaxf(z[3], z[7]);
#pragma unroll
    for (int i = 8; i < 32; i += 4) {
        c0 = fmaxf(c0, z[i]); c1 = fmaxf(c1, z[i + 1]); c2 = fmaxf(c2, z[i + 2]); c3 = fmaxf(c3, z[i + 3]);
    }
    const float cmax = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));          // fmaxf skips NaN operands
    const float m_new = fmaxf(st.m, cmax);
    if (st.m == -CUDART_INF_F) { st.s = 0.f; st.u = 0.f; }
    else {
        float dm = st.m - m_new;
        float a = exp_approx(dm);
        st.u = a * (st.u + dm * st.s);
        st.s = a * st.s;
    }
    st.m = m_new;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f, u0 = 0.f, u1 = 0.f, u2 = 0.f, u3 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        float d0 = z[i] - m_new, d1 = z[i + 1] - m_new, d2 = z[i + 2] - m_new, d3 = z[i + 3] - m_new;
        float e0 = exp_approx(d0), e1 = exp_approx(d1), e2 = exp_approx(d2), e3 = exp_approx(d3);   // NaN logit -> NaN sums
        s0 += e0; s1 += e1; s2 += e2; s3 += e3;
        u0 = fmaf(e0, d0, u0); u1 = fmaf(e1, d1, u1); u2 = fmaf(e2, d2, u2); u3 = fmaf(e3, d3, u3);
    }
    st.s += (s0 + s1) + (s2 + s3);
    st.u += (u0 + u1) + (u2 + u3);
    if (sa.on) {                              // sampled token: the same for every lane of the warp
        // vbase is a multiple of 4, so each generator call serves four consecutive columns
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
            uint32_t o[4];
            philox4x32_10((uint32_t)(vbase + i) >> 2, row, sa.d0, sa.d1, sa.k0, sa.k1, o);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float sc = fmaf(z[i + q], sa.inv_t, gumbel_from_bits(o[q]));
                if (z[i + q] == z[i + q] && sc > st.bv) { st.bv = sc; st.bi = vbase + i + q; }
            }
        }
        return;
    }
    if (cmax > st.bv) {                       // strictly larger: an earlier chunk keeps a tie
        int idx = 31;
#pragma unroll
        for (int i = 30; i >= 0; --i) idx = (z[i] == cmax) ? i : idx;     // lowest column holding the maximum
        st.bv = cmax;
        st.bi = vbase + idx;
    }
}

// The same for a chunk with fewer than 32 real vocabulary entries (tile tails).
__device__ __forceinline__ void fold_chunk_tail(Stats &st, const float (&z)[32], int n_valid, int vbase,
                                                const SampleArgs &sa, uint32_t row)
{
    float cmax = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (i < n_valid) cmax = fmaxf(cmax, z[i]);
    const float m_new = fmaxf(st.m, cmax);
    if (st.m == -CUDART_INF_F) { st.s = 0.f; st.u = 0.f; }
    else {
        float dm = st.m - m_new;
        float a = exp_approx(dm);
        st.u = a * (st.u + dm * st.s);
        st.s = a * st.s;
    }
    st.m = m_new;
    float s = 0.f, u = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        if (i < n_valid) {
            float dz = z[i] - m_new;
            float e = exp_approx(dz);
            s += e;
            u = fmaf(e, dz, u);
            const float sc = sa.on ? sample_score(sa, z[i], row, (uint32_t)(vbase + i)) : z[i];
            if (z[i] == z[i] && sc > st.bv) { st.bv = sc; st.bi = vbase + i; }   // ascending index: first maximum wins
        }
    }
    st.s += s;
    st.u += u;
}

__device__ __forceinline__ void fold_chunk(Stats &st, const float (&z)[32], int n_valid, int vbase,
                                           const SampleArgs &sa, uint32_t row)
{
    if (n_valid >= 32) fold_chunk_full(st, z, vbase, sa, row);     // n_valid is the same in every lane
    else               fold_chunk_tail(st, z, n_valid, vbase, sa, row);
}

// Tensor maps over W_head with boxes of 16, 32, 64, 128 and 256 rows: a tile of N rows (a multiple
// of 16) is fetched with one copy per set bit of N / 16, largest first.  Few large copies matter:
// a copy of a few KB costs the TMA unit about as much time as one of 16 KB.
struct WMaps { CUtensorMap box[5]; };

// Launch geometry computed on the host.
struct UmmaPlan {
    int nM, n_slices;
    int a_rows;            // hidden rows fetched per k-step (the MMA still reads 128)
    int n_stages, a_bytes, stage_bytes;
    int tiles_per_block;   // one M tile only
    int m64;               // one M tile only: at most 64 rows, issue M = 64 instructions
};

__global__ void __launch_bounds__(kThreads, 1)
head_umma_kernel(const __grid_constant__ CUtensorMap tm_hidden, const __grid_constant__ WMaps tm_w,
                 HeadArgs h, TailArgs t, Partials P, UmmaPlan plan)
{
    // The kernels after this one in the stream (head_finalize_kernel, then the next call's head kernel) may be
    // scheduled as soon as every block has got here; they wait for this kernel's completion themselves
    // before they touch what it writes.
    ptx::grid_dep_launch_dependents();
    extern __shared__ unsigned char dyn_smem_raw[];
    __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages];
    const int n_slices = plan.n_slices, n_stages = plan.n_stages;
    __shared__ __align__(8) uint64_t s_acc_full[2], s_acc_empty[2], s_done;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort, s_zero;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring = (ptx::smem_u32(dyn_smem_raw) + 1023u) & ~1023u;
    const int nK = (h.d + kTileK - 1) / kTileK;
    // The live row count, when it sits on the device, is the output of an earlier kernel, and so may the
    // hidden rows be; W_head is not.  Every role therefore waits for the kernels before this one by itself,
    // as late as it can: the producer only after a first ring of W_head has been asked for, the others
    // when they first need the count.
    auto rows_live = [&]() -> int {
        if (!h.n_rows_dev) return h.R;
        ptx::grid_dep_wait();
        const int n = *h.n_rows_dev;
        return n < 0 ? 0 : (n < h.R ? n : h.R);
    };

    Schedule sch;
    sch.init(h.V, gridDim.x, blockIdx.x, plan.tiles_per_block);

    if (threadIdx.x == 0) {
        s_abort = 0; s_zero = 0;
        for (int s = 0; s < n_stages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&s_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&s_empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&s_acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&s_acc_empty[b]), kEpiWarps);   // one arrival per epilogue warp
        }
        ptx::mbar_init(ptx::smem_u32(&s_done), 1);
        ptx::mbar_fence_init();
        ptx::prefetch_tmap(&tm_hidden);
        ptx::prefetch_tmap(&tm_w.box[4]);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&s_tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    if (warp == 0) {
        // ---- producer --------------------------------------------------------------------
        constexpr int pid = 0;
        if (lane == 0) {
            int stage = 0, round = 0, issued = 0;
            bool live = true;
            // The hidden rows may be the output of the kernel before this one, W_head is not.  Until the first
            // pass over the ring is complete only the W parts of the stages are fetched, and the hidden
            // tiles owed to those stages are remembered; then the producer waits for the earlier kernels,
            // pays the debt and goes on with whole stages.  A ring of W_head is in flight meanwhile.
            bool waited = false, no_rows = false;
            uint32_t owed_full[kMaxStages], owed_dst[kMaxStages];
            int owed_x[kMaxStages], n_owed = 0;
            auto settle = [&]() {
                ptx::grid_dep_wait();
                for (int q = 0; q < n_owed; ++q) ptx::tma_g2s_2d(owed_dst[q], &tm_hidden, owed_x[q], 0, owed_full[q]);
                n_owed = 0;
                waited = true;
                // no live row after all (a count on the device): the stages asked for so far complete, nobody
                // consumes them, and the producer only sees them land before it leaves
                if (h.n_rows_dev && *h.n_rows_dev <= 0) { no_rows = true; live = false; }
            };
            for (int j = 0; live && j < sch.n_items; ++j) {
                const Item it = sch.item(j);
                const uint32_t bytes = (uint32_t)((plan.a_rows + it.N) * kTileK * 2);
                // The k-steps are issued in groups: a copy brings 128 bytes of each of its rows, so the
                // copies of kIssueGroup consecutive k-steps, issued back to back box by box, ask DRAM for
                // kIssueGroup * 128 contiguous bytes of a row at a time instead of 128.
                for (int ks = 0; live && ks < nK; ks += kIssueGroup) {
                    int ng = nK - ks < kIssueGroup ? nK - ks : kIssueGroup;
                    if (ng > n_stages) ng = n_stages;
                    if (!waited && issued + ng > n_stages) settle();     // the ring has been round once
                    if (!live) break;
                    uint32_t full[kIssueGroup], a_dst[kIssueGroup];
                    for (int g = 0; g < ng; ++g) {
                        int sg = stage + g, rd = round;
                        if (sg >= n_stages) { sg -= n_stages; ++rd; }
                        if (!ptx::mbar_wait(ptx::smem_u32(&s_empty[sg]), (uint32_t)((rd & 1) ^ 1), &s_abort)) {
                            if (!s_abort) raise_abort(&s_abort, t.stat, 0x201u);
                            live = false;
                            ng = g;                  // the stages armed so far still get their copies
                            break;
                        }
                        full[g] = ptx::smem_u32(&s_full[sg]);
                        a_dst[g] = ring + (uint32_t)(sg * plan.stage_bytes);
                        ptx::mbar_arrive_expect_tx(full[g], bytes);
                    }
                    // only the first a_rows rows of the hidden tile are fetched; the MMA reads all 128,
                    // and what the stale rows produce lands in accumulator rows nobody looks at
                    for (int g = 0; g < ng; ++g) {
                        if (waited) {
                            ptx::tma_g2s_2d(a_dst[g], &tm_hidden, (ks + g) * kTileK, 0, full[g]);
                        } else {
                            owed_full[n_owed] = full[g]; owed_dst[n_owed] = a_dst[g]; owed_x[n_owed] = (ks + g) * kTileK;
                            ++n_owed;
                        }
                    }
                    int r = 0;
#pragma unroll
                    for (int b = 4; b >= 0; --b) {
                        const int rows = 16 << b;
                        if (it.N - r >= rows) {
                            for (int g = 0; g < ng; ++g)
                                ptx::tma_g2s_2d(a_dst[g] + (uint32_t)plan.a_bytes + (uint32_t)r * 128u, &tm_w.box[b],
                                                (ks + g) * kTileK, it.v0 + r, full[g]);
                            r += rows;
                        }
                    }
                    issued += ng;
                    stage += ng;
                    if (stage >= n_stages) { stage -= n_stages; ++round; }
                    if (ng < kIssueGroup && ks + ng < nK) ks += ng - kIssueGroup;   // fewer stages than a group
                }
            }
            if (!waited) settle();                   // fewer k-steps than stages: every armed stage gets its hidden tile
            if ((s_abort || no_rows) && pid == 0) {
                // no copy may still be landing in this block's shared memory when it exits
                int first = issued > n_stages ? issued - n_stages : 0;
                for (int q = first; q < issued; ++q)
                    ptx::mbar_wait(ptx::smem_u32(&s_full[q % n_stages]), (uint32_t)((q / n_stages) & 1), &s_zero);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---- MMA issuer ------------------------------------------------------------------
        if (lane == 0) {
            int stage = 0, round = 0;
            bool live = true;
            if (rows_live() == 0) sch.n_items = 0;       // no live rows (device-side count): nothing to multiply
            for (int j = 0; live && j < sch.n_items; ++j) {
                const Item it = sch.item(j);
                const int buf = j & 1, use = j >> 1;
                if (!ptx::mbar_wait(ptx::smem_u32(&s_acc_empty[buf]), (uint32_t)((use & 1) ^ 1), &s_abort)) {
                    if (!s_abort) raise_abort(&s_abort, t.stat, 0x202u);
                    break;
                }
                ptx::tc_fence_after_sync();
                // with at most 64 rows an M = 64 instruction does half the tensor work and reads half the
                // hidden tile; its 64 accumulator rows sit in lanes 0-15 of each 32-lane quarter
                const uint32_t idesc = ptx::umma_idesc_bf16(plan.m64 ? 64 : kTileM, it.N);
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * kTileNMax;
                for (int ks = 0; ks < nK; ++ks) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&s_full[stage]), (uint32_t)(round & 1), &s_abort)) {
                        if (!s_abort) raise_abort(&s_abort, t.stat, 0x203u);
                        live = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_src = ring + (uint32_t)(stage * plan.stage_bytes);
                    const uint64_t a_desc = ptx::smem_desc_sw128(a_src);
                    const uint64_t b_desc = ptx::smem_desc_sw128(a_src + (uint32_t)plan.a_bytes);
#pragma unroll
                    for (int kk = 0; kk < kTileK / 16; ++kk)     // 32 bytes along K per instruction
                        ptx::umma_bf16(d_tmem, a_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc,
                                       (uint32_t)((ks | kk) != 0));
                    ptx::umma_commit(ptx::smem_u32(&s_empty[stage]));      // frees the stage when the MMAs are done
                    if (++stage == n_stages) { stage = 0; ++round; }
                }
                if (live) ptx::umma_commit(ptx::smem_u32(&s_acc_full[buf]));   // accumulator complete
            }
            if (sch.n_items > 0) {
                // everything issued has finished before the tensor memory is released (a commit with
                // no MMA before it would never arrive)
                ptx::umma_commit(ptx::smem_u32(&s_done));
                ptx::mbar_wait(ptx::smem_u32(&s_done), 0u, &s_zero);
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue: warps 2-5 fold the first half of a tile's 32-column chunks, warps 6-9 the rest ----
        const int quarter = warp & 3;                        // the TMEM lanes this warp may read
        const int half = (warp - 2) >> 2;
        const int R_live = rows_live();
        if (R_live == 0) sch.n_items = 0;
        // M = 128: accumulator row i is lane i.  M = 64: row i is lane 32 (i / 16) + i % 16.
        const int rows_per_quarter = plan.m64 ? 16 : 32;
        const int row = quarter * rows_per_quarter + lane;
        const bool lane_has_row = lane < rows_per_quarter && row < R_live;
        const bool warp_has_rows = quarter * rows_per_quarter < R_live;
        Stats st = stats_empty();
        for (int j = 0; j < sch.n_items; ++j) {
            const Item it = sch.item(j);
            const int buf = j & 1, use = j >> 1;
            if (!ptx::mbar_wait(ptx::smem_u32(&s_acc_full[buf]), (uint32_t)(use & 1), &s_abort)) {
                if (lane == 0 && !s_abort) raise_abort(&s_abort, t.stat, 0x204u);
                break;
            }
            ptx::tc_fence_after_sync();
            if (warp_has_rows) {
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * kTileNMax;
                const int n_chunks = (it.N + 31) >> 5;
                const int c_split = ((n_chunks + 1) >> 1) << 5;
                const int c_begin = half ? c_split : 0, c_end = half ? it.N : (c_split < it.N ? c_split : it.N);
                for (int c0 = c_begin; c0 < c_end; c0 += 32) {
                    float z[32];
                    ptx::tmem_ld_32x32(taddr + (uint32_t)c0, z);
                    int n_valid = it.N - c0;
                    if (h.V - (it.v0 + c0) < n_valid) n_valid = h.V - (it.v0 + c0);
                    if (n_valid > 32) n_valid = 32;
                    if (lane_has_row && n_valid > 0)
                        fold_chunk(st, z, n_valid, it.v0 + c0, h.sample, (uint32_t)row);
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&s_acc_empty[buf]));
        }
        // Every accumulator has been drained, so every copy has landed and the ring is idle: the second
        // half's statistics cross to the first half through it, which writes the block's partial.
        float *xch = reinterpret_cast<float *>(dyn_smem_raw + (ring - ptx::smem_u32(dyn_smem_raw)));
        const int slot = (quarter * 32 + lane) * 5;
        if (half == 1) {
            xch[slot] = st.m; xch[slot + 1] = st.s; xch[slot + 2] = st.u; xch[slot + 3] = st.bv;
            xch[slot + 4] = __int_as_float(st.bi);
        }
        asm volatile("bar.sync 1, %0;" :: "n"(kEpiWarps * 32) : "memory");
        ptx::grid_dep_wait();                        // the scratch may still be read by the call before this one
        if (half == 0 && lane_has_row) {
            Stats o;
            o.m = xch[slot]; o.s = xch[slot + 1]; o.u = xch[slot + 2]; o.bv = xch[slot + 3];
            o.bi = __float_as_int(xch[slot + 4]);
            stats_merge(st, o);
            partial_store(P, (size_t)row * n_slices + blockIdx.x, st);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
    // head_finalize_kernel, launched behind this kernel, merges the blocks' partials and decides
}

// ---- several M tiles, two per W tile ------------------------------------------------------------
// With more than 128 rows one block works on TWO M tiles against the same W tile, so each 32 KB W stage
// is used twice: per k-step 64 KB of copies feed eight MMAs instead of 96 KB.  The 512 tensor-memory
// columns hold the two accumulators, so there is no second buffer: eight epilogue warps (four per
// accumulator) drain them while the tensor pipe waits, a few percent of an item.  Work items are
// (vocabulary tile, pair of M tiles), dealt round-robin with the pairs of one vocabulary tile adjacent
// (W_head from HBM once, then from L2).  Timing variants showed the k-step time to be the sum of the
// copy bytes and the operand bytes over ~200 KB/us: shared-memory bandwidth, not HBM, L2 latency
// (an L2 prefetch changed nothing) or instruction issue, bounds this kernel at about 0.8 of the
// library GEMM's rate when the M tiles are full.
constexpr int kThreads2    = 320 + (kProducers - 1) * 32;  // producer, MMA, 8 epilogue warps, extra producers
constexpr int kStages2     = 3;
constexpr int kStage2Bytes = 2 * kABytes + kBBytes;        // 64 KB
constexpr int kDynSmem2    = kStages2 * kStage2Bytes + 1024;

struct Item2 { int v0, N, m0, two; };

// An M tile that holds at most 64 of the R rows (the last, partly filled one).
__device__ __forceinline__ bool tile_is_small(int tile, int R)
{
    const int rows = R - tile * kTileM;
    return rows > 0 && rows <= 64;
}

__device__ __forceinline__ Item2 item2(int q, int nMG, int nM, int V)
{
    Item2 it;
    int vt = q / nMG;
    int mg = q - vt * nMG;
    it.m0 = 2 * mg;
    it.two = (it.m0 + 1 < nM) ? 1 : 0;
    it.v0 = vt * kTileNMax;
    int left = V - it.v0;
    it.N = left >= kTileNMax ? kTileNMax : ((left + 15) / 16) * 16;
    return it;
}

// Work of one block of head_umma2_kernel.  Items q = 0 .. total-1 are dealt round-robin: block c takes
// c, c + grid, ...  The last, partly filled round would leave most blocks idle for a whole item, so when
// its items split into at most `grid` single-M-tile pieces they are dealt as such, one piece per block
// (a piece costs ~0.6 of a two-tile item: its own hidden tile plus the whole W tile).
struct Sched2 {
    int nM, nMG, grid, cta;
    int n_items;                 // whole items of this block
    int piece_q, piece_mt;       // this block's piece of the last round (piece_q < 0: none)
};

__device__ __forceinline__ int tiles_of_item2(int q, int nMG, int nM)
{
    const int mg = q % nMG;
    return (2 * mg + 1 < nM) ? 2 : 1;
}

__device__ __forceinline__ Sched2 sched2_make(int nM, int V, int grid, int cta, bool any_rows)
{
    Sched2 s;
    s.nM = nM; s.nMG = (nM + 1) / 2; s.grid = grid; s.cta = cta;
    s.piece_q = -1; s.piece_mt = 0;
    const int total = ((V + kTileNMax - 1) / kTileNMax) * s.nMG;
    const int full = (total / grid) * grid;              // items of the completely filled rounds
    int pieces = 0;
    for (int q = full; q < total; ++q) pieces += tiles_of_item2(q, s.nMG, nM);
    if (!any_rows) { s.n_items = 0; return s; }
    if (pieces > grid || pieces == 0) {                  // nothing to split, or too many pieces: plain deal
        s.n_items = cta < total ? (total - cta + grid - 1) / grid : 0;
        return s;
    }
    s.n_items = full / grid;
    int k = 0;
    for (int q = full; q < total; ++q) {
        const int n = tiles_of_item2(q, s.nMG, nM);
        if (cta >= k && cta < k + n) { s.piece_q = q; s.piece_mt = cta - k; }
        k += n;
    }
    return s;
}

__device__ __forceinline__ int sched2_count(const Sched2 &s) { return s.n_items + (s.piece_q >= 0 ? 1 : 0); }

__device__ __forceinline__ Item2 sched2_item(const Sched2 &s, int j, int V)
{
    if (j < s.n_items) return item2(s.cta + j * s.grid, s.nMG, s.nM, V);
    Item2 it = item2(s.piece_q, s.nMG, s.nM, V);
    it.m0 += s.piece_mt;                                 // one M tile of the pair, in the first accumulator
    it.two = 0;
    return it;
}

__global__ void __launch_bounds__(kThreads2, 1)
head_umma2_kernel(const __grid_constant__ CUtensorMap tm_hidden, const __grid_constant__ WMaps tm_w,
                  HeadArgs h, TailArgs t, Partials P, int nM, int n_slices)
{
    extern __shared__ unsigned char dyn_smem_raw[];
    __shared__ __align__(8) uint64_t s_full[kStages2], s_empty[kStages2];
    __shared__ __align__(8) uint64_t s_acc_full, s_acc_empty, s_done;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort, s_zero;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring = (ptx::smem_u32(dyn_smem_raw) + 1023u) & ~1023u;
    const int nK = (h.d + kTileK - 1) / kTileK;
    ptx::grid_dep_launch_dependents();
    ptx::grid_dep_wait();          // hidden rows, the live count and the scratch may come from the kernels before
    int R_live = h.R;
    if (h.n_rows_dev) { int n = *h.n_rows_dev; R_live = n < 0 ? 0 : (n < h.R ? n : h.R); }
    const Sched2 sch = sched2_make(nM, h.V, (int)gridDim.x, (int)blockIdx.x, R_live > 0);
    const int n_items = sched2_count(sch);

    if (threadIdx.x == 0) {
        s_abort = 0; s_zero = 0;
        for (int s = 0; s < kStages2; ++s) {
            ptx::mbar_init(ptx::smem_u32(&s_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&s_empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&s_acc_full), 1);
        ptx::mbar_init(ptx::smem_u32(&s_acc_empty), 8);        // one arrival per epilogue warp
        ptx::mbar_init(ptx::smem_u32(&s_done), 1);
        ptx::mbar_fence_init();
        ptx::prefetch_tmap(&tm_hidden);
        ptx::prefetch_tmap(&tm_w.box[4]);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&s_tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = s_tmem_base;

    if (warp == 0 || warp >= 10) {
        // ---- producers: the copies of a stage are dealt round-robin to kProducers threads ------
        const int pid = warp == 0 ? 0 : warp - 9;
        if (lane == 0) {
            int stage = 0, round = 0, issued = 0;
            bool live = true;
            for (int j = 0; live && j < n_items; ++j) {
                const Item2 it = sched2_item(sch, j, h.V);
                for (int ks = 0; ks < nK; ++ks) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&s_empty[stage]), (uint32_t)((round & 1) ^ 1), &s_abort)) {
                        if (!s_abort) raise_abort(&s_abort, t.stat, 0x211u);
                        live = false;
                        break;
                    }
                    const uint32_t full = ptx::smem_u32(&s_full[stage]);
                    const uint32_t a_dst = ring + (uint32_t)(stage * kStage2Bytes);
                    const uint32_t b_dst = a_dst + 2u * kABytes;
                    if (pid == 0) {
                        ptx::mbar_arrive_expect_tx(full, (uint32_t)((it.two ? 2 : 1) * kABytes + it.N * kTileK * 2));
                        ptx::tma_g2s_2d(a_dst, &tm_hidden, ks * kTileK, it.m0 * kTileM, full);
                    }
                    if (it.two && pid == 1 % kProducers)
                        ptx::tma_g2s_2d(a_dst + kABytes, &tm_hidden, ks * kTileK, (it.m0 + 1) * kTileM, full);
                    int r = 0, op = 2;
#pragma unroll
                    for (int b = 4; b >= 0; --b) {
                        const int rows = 16 << b;
                        if (it.N - r >= rows) {
                            if (op % kProducers == pid)
                                ptx::tma_g2s_2d(b_dst + (uint32_t)r * 128u, &tm_w.box[b], ks * kTileK, it.v0 + r, full);
                            r += rows;
                            ++op;
                        }
                    }
                    ++issued;
                    if (++stage == kStages2) { stage = 0; ++round; }
                }
            }
            if (s_abort && pid == 0) {
                int first = issued > kStages2 ? issued - kStages2 : 0;
                for (int q = first; q < issued; ++q)
                    ptx::mbar_wait(ptx::smem_u32(&s_full[q % kStages2]), (uint32_t)((q / kStages2) & 1), &s_zero);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---- MMA issuer ------------------------------------------------------------------
        if (lane == 0) {
            int stage = 0, round = 0;
            bool live = true;
            for (int j = 0; live && j < n_items; ++j) {
                const Item2 it = sched2_item(sch, j, h.V);
                if (!ptx::mbar_wait(ptx::smem_u32(&s_acc_empty), (uint32_t)((j & 1) ^ 1), &s_abort)) {
                    if (!s_abort) raise_abort(&s_abort, t.stat, 0x212u);
                    break;
                }
                ptx::tc_fence_after_sync();
                // an M tile with at most 64 rows (the last one) takes M = 64 instructions
                const uint32_t idesc0 = ptx::umma_idesc_bf16(tile_is_small(it.m0, h.R) ? 64 : kTileM, it.N);
                const uint32_t idesc1 = ptx::umma_idesc_bf16(tile_is_small(it.m0 + 1, h.R) ? 64 : kTileM, it.N);
                for (int ks = 0; ks < nK; ++ks) {
                    if (!ptx::mbar_wait(ptx::smem_u32(&s_full[stage]), (uint32_t)(round & 1), &s_abort)) {
                        if (!s_abort) raise_abort(&s_abort, t.stat, 0x213u);
                        live = false;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_src = ring + (uint32_t)(stage * kStage2Bytes);
                    const uint64_t a0_desc = ptx::smem_desc_sw128(a_src);
                    const uint64_t a1_desc = ptx::smem_desc_sw128(a_src + kABytes);
                    const uint64_t b_desc = ptx::smem_desc_sw128(a_src + 2u * kABytes);
#pragma unroll
                    for (int kk = 0; kk < kTileK / 16; ++kk)
                        ptx::umma_bf16(tmem_base, a0_desc + (uint64_t)(kk * 2), b_desc + (uint64_t)(kk * 2), idesc0,
                                       (uint32_t)((ks | kk) != 0));
                    if (it.two) {
#pragma unroll
                        for (int kk = 0; kk < kTileK / 16; ++kk)
                            ptx::umma_bf16(tmem_base + kTileNMax, a1_desc + (uint64_t)(kk * 2),
                                           b_desc + (uint64_t)(kk * 2), idesc1, (uint32_t)((ks | kk) != 0));
                    }
                    ptx::umma_commit(ptx::smem_u32(&s_empty[stage]));
                    if (++stage == kStages2) { stage = 0; ++round; }
                }
                if (live) ptx::umma_commit(ptx::smem_u32(&s_acc_full));
            }
            if (n_items > 0) {
                // everything issued has finished before the tensor memory is released
                ptx::umma_commit(ptx::smem_u32(&s_done));
                ptx::mbar_wait(ptx::smem_u32(&s_done), 0u, &s_zero);
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue: warps 2-5 drain the first accumulator, warps 6-9 the second ---------
        const int mt = (warp - 2) >> 2;
        const int quarter = warp & 3;
        for (int j = 0; j < n_items; ++j) {
            const Item2 it = sched2_item(sch, j, h.V);
            const int rows_per_quarter = tile_is_small(it.m0 + mt, h.R) ? 16 : 32;     // M = 64: 16 rows per quarter
            const int row0 = (it.m0 + mt) * kTileM + quarter * rows_per_quarter;
            const int row = row0 + lane;
            const bool lane_has_row = lane < rows_per_quarter;
            if (!ptx::mbar_wait(ptx::smem_u32(&s_acc_full), (uint32_t)(j & 1), &s_abort)) {
                if (lane == 0 && !s_abort) raise_abort(&s_abort, t.stat, 0x214u);
                break;
            }
            ptx::tc_fence_after_sync();
            Stats st = stats_empty();
            const bool warp_has_rows = (mt == 0 || it.two) && row0 < R_live;
            if (warp_has_rows) {
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * kTileNMax);
                for (int c0 = 0; c0 < it.N; c0 += 32) {
                    float z[32];
                    ptx::tmem_ld_32x32(taddr + (uint32_t)c0, z);
                    int n_valid = it.N - c0;
                    if (h.V - (it.v0 + c0) < n_valid) n_valid = h.V - (it.v0 + c0);
                    if (n_valid > 32) n_valid = 32;
                    if (lane_has_row && row < R_live && n_valid > 0)
                        fold_chunk(st, z, n_valid, it.v0 + c0, h.sample, (uint32_t)row);
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&s_acc_empty));
            if (warp_has_rows && lane_has_row && row < R_live)
                partial_store(P, (size_t)row * n_slices + (size_t)(it.v0 / kTileNMax), st);
        }
    }

    ptx::tc_fence_before_sync();
    __threadfence();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// hidden[row_idx[r]] -> packed[r] (zero for rows past the live count or with a bad index).
__global__ void __launch_bounds__(128)
gather_rows_kernel(HeadArgs h, uint4 *packed, int rows_padded, DevStat *stat)
{
    // the head kernel behind this one may start on W_head at once; it waits for this kernel before it
    // reads the packed rows, as this kernel waits for the ones that wrote the index list and the count
    ptx::grid_dep_launch_dependents();
    ptx::grid_dep_wait();
    const int r = blockIdx.x;
    const int d8 = h.d >> 3;
    int R_live = h.R;
    if (h.n_rows_dev) { int n = *h.n_rows_dev; R_live = n < 0 ? 0 : (n < h.R ? n : h.R); }
    int src = -1;
    if (r < R_live) {
        src = h.row_idx ? h.row_idx[r] : r;
        if (src < 0 || src >= h.n_src) {
            if (threadIdx.x == 0) atomicAdd(&stat->bad_row_idx, 1u);
            src = 0;
        }
    }
    const uint4 *in = (const uint4 *)h.hidden;
    for (int c = threadIdx.x; c < d8; c += blockDim.x)
        packed[(size_t)r * d8 + c] = src >= 0 ? in[(size_t)src * d8 + c] : make_uint4(0, 0, 0, 0);
    (void)rows_padded;
}

// ---- host side: tensor maps -----------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        else
            cudaGetLastError();
    }
    return fn;
}

// bf16 [rows, d] row-major, box = 64 elements along d by box_rows rows, 128-byte swizzle,
// out-of-range elements read as zero.
bool encode_map(CUtensorMap *m, const void *base, int rows, int d, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2]    = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2]     = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
    cuuint32_t estr[2]    = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same through the caller's cache: a decode loop presents the same W_head and the same hidden
// buffers call after call, and encoding six maps costs the host more than the two launches do.
bool make_map(TmapCache *cache, CUtensorMap *m, const void *base, int rows, int d, int box_rows)
{
    if (!cache) return encode_map(m, base, rows, d, box_rows);
    TmapCache::Entry *victim = &cache->e[0];
    for (TmapCache::Entry &e : cache->e) {
        if (e.used && e.base == base && e.rows == rows && e.d == d && e.box_rows == box_rows) {
            e.used = ++cache->clock;
            std::memcpy(m, e.map, sizeof(CUtensorMap));
            return true;
        }
        if (e.used < victim->used) victim = &e;
    }
    if (!encode_map(m, base, rows, d, box_rows)) return false;
    victim->base = base; victim->rows = rows; victim->d = d; victim->box_rows = box_rows;
    victim->used = ++cache->clock;
    std::memcpy(victim->map, m, sizeof(CUtensorMap));
    return true;
}

}  // namespace

bool umma_shape_ok(int R, int d, int V)
{
    return R >= 1 && d >= kTileK && V >= kTileNMax && encode_fn() != nullptr;
}

size_t umma_gather_bytes(int R, int d)
{
    size_t rows = (size_t)((R + kTileM - 1) / kTileM) * kTileM;
    return rows * (size_t)d * 2;
}

static_assert(sizeof(CUtensorMap) == sizeof(TmapCache::Entry::map), "tensor-map cache entry size");

cudaError_t launch_head_umma(const HeadArgs &h, const TailArgs &t, const Scratch &s, void *gather_buf,
                             int sm_count, cudaStream_t stream, int *launched, TmapCache *cache)
{
    *launched = 0;
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        e = cudaFuncSetAttribute(head_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(head_umma2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDynSmem2);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    UmmaPlan plan;
    plan.nM = (h.R + kTileM - 1) / kTileM;
    int grid = sm_count;
    if (grid > kMaxSlices) grid = kMaxSlices;
    int n_max = kTileNMax;
    plan.tiles_per_block = 0;
    if (plan.nM == 1) {
        int units = (h.V + 15) / 16;
        if (grid > units) grid = units;
        int nu = (units + grid - 1) / grid;              // largest range of any block, in 16-row units
        plan.tiles_per_block = (nu + 15) / 16;
        n_max = ((nu + plan.tiles_per_block - 1) / plan.tiles_per_block) * 16;
    }
    plan.n_slices = plan.nM == 1 ? grid : (h.V + kTileNMax - 1) / kTileNMax;
    // Stage = the hidden rows actually fetched + the largest W tile of this launch.  The MMA reads
    // 128 hidden rows from the stage's start whatever was fetched, so the last stage keeps that
    // much room inside the ring.
    plan.a_rows = plan.nM == 1 ? ((h.R + 7) / 8) * 8 : kTileM;
    plan.m64 = (plan.nM == 1 && h.R <= 64) ? 1 : 0;
    plan.a_bytes = ((plan.a_rows * kTileK * 2 + 1023) / 1024) * 1024;
    plan.stage_bytes = plan.a_bytes + n_max * kTileK * 2;
    plan.n_stages = (kRingBytes - (kABytes - plan.a_bytes)) / plan.stage_bytes;
    if (plan.n_stages > kMaxStages) plan.n_stages = kMaxStages;
    Partials P = partials_carve(s.partials, (size_t)h.R, (size_t)plan.n_slices);

    HeadArgs hk = h;
    const void *hid_base = h.hidden;
    int hid_rows = h.n_src > 0 ? h.n_src : h.R;
    if (h.row_idx) {
        // the tensor-map copy cannot follow an index list: pack the gathered rows first
        const int rows_padded = plan.nM * kTileM;
        HeadArgs hg = h;
        uint4 *packed = (uint4 *)gather_buf;
        int padded = rows_padded;
        DevStat *stat = t.stat;
        void *gargs[] = {&hg, &packed, &padded, &stat};
        e = launch_dependent((const void *)gather_rows_kernel, dim3((unsigned)rows_padded), dim3(128), 0, stream, gargs);
        if (e != cudaSuccess) return e;
        ++*launched;
        hid_base = gather_buf;
        hid_rows = rows_padded;
        hk.row_idx = nullptr;
    }
    CUtensorMap tm_h;
    WMaps tm_w;
    if (!make_map(cache, &tm_h, hid_base, hid_rows, h.d, plan.a_rows)) return cudaErrorInvalidValue;
    for (int b = 0; b < 5; ++b)
        if (!make_map(cache, &tm_w.box[b], h.W, h.V, h.d, 16 << b)) return cudaErrorInvalidValue;
    Partials Pk = P;
    HeadArgs hk2 = hk;
    TailArgs tk = t;
    if (plan.nM == 1) {
        void *args[] = {&tm_h, &tm_w, &hk2, &tk, &Pk, &plan};
        e = launch_dependent((const void *)head_umma_kernel, dim3((unsigned)grid), dim3(kThreads), kDynSmem, stream, args);
    } else {
        void *args[] = {&tm_h, &tm_w, &hk2, &tk, &Pk, &plan.nM, &plan.n_slices};
        e = launch_dependent((const void *)head_umma2_kernel, dim3((unsigned)grid), dim3(kThreads2), kDynSmem2, stream, args);
    }
    if (e != cudaSuccess) return e;
    ++*launched;
    e = launch_head_finalize(P, plan.n_slices, h.R, hk.n_rows_dev, t, s.ticket, sm_count, stream);
    if (e == cudaSuccess) ++*launched;
    return e;
}

}  // namespace rstitch
