/*
 * CPU oracle for the R-Stitch routing decision.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the path computes, written from the
 * paper's definitions.  It shares no code, header, table or constant with the
 * CUDA library; only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  Inputs are the same bf16 bit patterns the GPU consumes,
 * widened exactly to double.
 *
 * Every function below is pinned by CPU tests against closed forms, textbook
 * special cases, an extended-precision brute force and a library log-softmax.
 * The paper prints no numeric entropy, token id or mask for any input, so
 * agreement with the paper's own numbers is "parity unpinned": only the
 * definition (Eq. 1), the rule (Eq. 2, Algorithm 1) and the span arithmetic
 * (Algorithm 1, prefill branch) are pinned.
 *
 * The vocabulary loop of the logit step is split over OpenMP threads; that
 * is the only parallelism, and no blocking, fusion or reordering is applied.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 -> double, exact: bf16 is the top 16 bits of an IEEE float32. */
static double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Logits of one row (Section 3.1: the active model's last linear map turns
 * the final hidden state into the distribution p_t over V entries):
 *     z[v] = sum_{k=0}^{d-1} hidden[k] * W_head[v, k],   k ascending.
 * W_head is row-major [V, d].
 */
void oracle_logits_row(const uint16_t *hidden_row, const uint16_t *w_head,
                       int d, int V, double *z)
{
    double *h = (double *)malloc((size_t)d * sizeof(double));
    for (int k = 0; k < d; ++k) h[k] = bf16_to_double(hidden_row[k]);
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v) {
        const uint16_t *wv = w_head + (size_t)v * (size_t)d;
        double acc = 0.0;
        for (int k = 0; k < d; ++k) acc += h[k] * bf16_to_double(wv[k]);
        z[v] = acc;
    }
    free(h);
}

/*
 * Greedy token (Section 3.1, y_t; greedy reading) and the top-2 logit gap.
 * tok = lowest index attaining the maximum, NaN logits ignored; 0 if every
 * logit is NaN.  gap = z[tok] - max_{v != tok} z[v] (0 on an exact tie).
 */
void oracle_greedy(const double *z, int V, int32_t *tok, double *gap)
{
    int best = -1;
    for (int v = 0; v < V; ++v) {
        if (isnan(z[v])) continue;
        if (best < 0 || z[v] > z[best]) best = v;
    }
    if (best < 0) { *tok = 0; *gap = NAN; return; }
    double second = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (v == best || isnan(z[v])) continue;
        if (z[v] > second) second = z[v];
    }
    *tok = (int32_t)best;
    *gap = z[best] - second;
}

/*
 * Softmax entropy in nats (numerator of Eq. 1), two passes, no online trick:
 *     m      = max_v z[v]
 *     lse    = m + log sum_v exp(z[v] - m)
 *     logp_v = z[v] - lse,  p_v = exp(logp_v)
 *     H      = - sum_v p_v * logp_v        (a term is 0 when p_v underflows to 0)
 * NaN logits propagate to a NaN entropy.
 */
double oracle_entropy_nats(const double *z, int V)
{
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (isnan(z[v])) return NAN;
        if (z[v] > m) m = z[v];
    }
    double sum = 0.0;
    for (int v = 0; v < V; ++v) sum += exp(z[v] - m);
    double lse = m + log(sum);
    double H = 0.0;
    for (int v = 0; v < V; ++v) {
        double logp = z[v] - lse;
        double p = exp(logp);
        if (p > 0.0) H -= p * logp;
    }
    return H;
}

/* Eq. 1 in full: entropy divided by log V, a value in [0, 1]. */
double oracle_entropy_normalized(const double *z, int V)
{
    return oracle_entropy_nats(z, V) / log((double)V);
}

/*
 * Switching predicate (Eq. 2; Algorithm 1, "if H_t > tau"): strict.  On the
 * SLM head 1 means hand the step to the LLM; on the LLM head 1 means stay on
 * the LLM and 0 means return to the SLM.  A NaN entropy routes to the LLM.
 */
uint8_t oracle_rule(double H, double tau)
{
    if (isnan(H)) return 1;
    return (H > tau) ? 1 : 0;
}

/*
 * Head + entropy + greedy token for R rows.
 *   hidden  bf16 bits, row-major [n_src, d]; row r reads hidden[row_idx[r]]
 *           when row_idx != NULL, else hidden[r].
 *   outputs per row: tok, H (nats), H / log V, top-2 gap.
 */
void oracle_head_rows(const uint16_t *hidden, const int32_t *row_idx,
                      const uint16_t *w_head, int R, int d, int V,
                      int32_t *tok, double *H_nats, double *H_norm, double *gap)
{
    double *z = (double *)malloc((size_t)V * sizeof(double));
    for (int r = 0; r < R; ++r) {
        size_t src = row_idx ? (size_t)row_idx[r] : (size_t)r;
        oracle_logits_row(hidden + src * (size_t)d, w_head, d, V, z);
        oracle_greedy(z, V, &tok[r], &gap[r]);
        H_nats[r] = oracle_entropy_nats(z, V);
        H_norm[r] = oracle_entropy_normalized(z, V);
    }
    free(z);
}

/*
 * Per-sequence mask.  Without row_seq, sequence b is decided by row b
 * (B == R).  With row_seq (int32 [R], non-decreasing sequence ids), the rows
 * of one sequence are one stitched span run through a prefill, which yields
 * one (p_t, y_t) at the end of the span (Algorithm 1, prefill branch): the
 * decision row of a sequence is its last row.  Sequences without rows get 0.
 */
void oracle_mask(const double *H_nats, const int32_t *row_seq, int R, int B,
                 double tau, uint8_t *mask)
{
    for (int b = 0; b < B; ++b) mask[b] = 0;
    if (!row_seq) {
        for (int b = 0; b < B && b < R; ++b) mask[b] = oracle_rule(H_nats[b], tau);
        return;
    }
    for (int r = 0; r < R; ++r) {
        int last = (r == R - 1) || (row_seq[r + 1] != row_seq[r]);
        if (last && row_seq[r] >= 0 && row_seq[r] < B)
            mask[row_seq[r]] = oracle_rule(H_nats[r], tau);
    }
}

/* Ordered compaction: ascending list of b with mask[b] != 0, and its length. */
void oracle_compact(const uint8_t *mask, int B, int32_t *idx, int32_t *count)
{
    int32_t n = 0;
    for (int b = 0; b < B; ++b)
        if (mask[b]) idx[n++] = (int32_t)b;
    *count = n;
}

/*
 * Stitched-span lengths of the routed sequences (Algorithm 1, prefill branch:
 * the model that takes over prefills (x + y)[L:], i.e. |x + y| - L tokens) and
 * their exclusive prefix sum, the row offsets of the catch-up batch;
 * row_off[count] is the total number of rows.
 */
void oracle_spans(const int32_t *idx, int32_t count, const int32_t *seq_len,
                  const int32_t *kv_len, int32_t *span, int32_t *row_off)
{
    int32_t acc = 0;
    for (int32_t j = 0; j < count; ++j) {
        span[j] = seq_len[idx[j]] - kv_len[idx[j]];
        row_off[j] = acc;
        acc += span[j];
    }
    row_off[count] = acc;
}

/* ------------------------------------------------------------------------
 * Latency estimator and the hybrid decode loop (the steps either side of the
 * routing decision).
 * ------------------------------------------------------------------------ */

/*
 * Eq. 5: estimated latency of one model step that processes n_inf tokens on
 * top of a KV cache of n_kv entries,
 *     T = a * n_inf * n_kv + b * n_inf^2 + c * n_inf + d      (milliseconds),
 * coef = {a, b, c, d} fitted per model (the appendix on latency regression
 * prints three sets).  A decode step is the same expression at n_inf = 1
 * (Eq. 6 is read as that special case; its printed right-hand side reuses
 * the letters c and d for the collapsed coefficients a and b + c + d).
 */
double oracle_latency_ms(const double *coef, int32_t n_inf, int32_t n_kv)
{
    double ni = (double)n_inf, nk = (double)n_kv;
    return coef[0] * ni * nk + coef[1] * ni * ni + coef[2] * ni + coef[3];
}

/*
 * Algorithm 1 for ONE sequence, written out in the paper's order, with the
 * two models replaced by recorded streams: at loop index t (0-based here)
 * the active model m (0 = SLM, 1 = LLM) "generates" token tok[m][t] with
 * entropy ent[m][t] (nats).  KV caches are represented by their sizes only.
 *
 *   L[0] = L[1] = 0, y = [], active = SLM
 *   for t = 1 .. T_max:
 *     if L[active] < |x + y|:  prefill on (x + y)[L[active]:]  -> n_inf = |x + y| - L[active],
 *                              n_kv = L[active];  L[active] <- |x + y| + 1
 *     else:                    decode -> n_inf = 1, n_kv = L[active];  L[active] <- L[active] + 1
 *     H_t > tau:   switch = true (R-Stitch), or the router's decision for this step (R-Stitch+:
 *                  switch = (argmax_a pi(a | s_t) == LLM), recorded in switch_slm[t]; NULL means R-Stitch)
 *        active == SLM and switch: discard y_t, roll KV^SLM back by the one entry just added,
 *                                  active <- LLM, continue
 *        otherwise (SLM without switch, or LLM): the active model stays and y_t is kept
 *     else if active == LLM: active <- SLM
 *     append y_t;  stop after appending EOS
 * The router is consulted only when H_t > tau and only changes what an SLM step does: low-entropy tokens
 * always stay with the SLM, and on the LLM the rule is the entropy test alone.
 *
 * The latency estimate sums Eq. 5 over every model step taken, discarded ones included.
 *
 * Outputs: y (capacity y_cap >= t_max), *n_out = |y|, final active, L[2], *len = |x + y|,
 * *lat_ms, tokens kept from each model, model steps taken by each model, *done = 1 if EOS ended it,
 * *iters = loop iterations executed.
 */
void oracle_alg1_sequence(int32_t prompt_len, int32_t t_max, double tau, int32_t eos_id,
                          const int32_t *tok_slm, const double *ent_slm,
                          const int32_t *tok_llm, const double *ent_llm,
                          const double *coef_slm, const double *coef_llm, const uint8_t *switch_slm,
                          int32_t *y, int32_t *n_out, int32_t *active_out, int32_t *L_out,
                          int32_t *len_out, double *lat_ms, int32_t *kept, int32_t *steps,
                          int32_t *done, int32_t *iters)
{
    int32_t L[2] = {0, 0};
    int32_t len = prompt_len;
    int active = 0;
    int32_t n = 0;
    double lat = 0.0;
    kept[0] = kept[1] = 0;
    steps[0] = steps[1] = 0;
    *done = 0;
    int32_t t = 0;
    for (t = 0; t < t_max; ++t) {
        int32_t n_inf, n_kv;
        if (L[active] < len) {              /* KV cache not up to date: prefill the missing span */
            n_inf = len - L[active];
            n_kv = L[active];
            L[active] = len + 1;
        } else {                            /* decode */
            n_inf = 1;
            n_kv = L[active];
            L[active] = L[active] + 1;
        }
        lat += oracle_latency_ms(active == 0 ? coef_slm : coef_llm, n_inf, n_kv);
        steps[active] += 1;
        double H = active == 0 ? ent_slm[t] : ent_llm[t];
        int32_t yt = active == 0 ? tok_slm[t] : tok_llm[t];
        const int gen = active;             /* the model that produced y_t */
        if (oracle_rule(H, tau)) {
            const int sw = switch_slm ? (switch_slm[t] != 0) : 1;
            if (active == 0 && sw) {        /* SLM -> LLM: token not kept */
                L[0] -= 1;                  /* roll back the cache entry this step added */
                active = 1;
                continue;
            }                               /* the router kept the SLM, or the LLM keeps decoding */
        } else if (active == 1) {
            active = 0;                     /* LLM -> SLM */
        }
        kept[gen] += 1;                     /* append y_t */
        y[n++] = yt;
        len += 1;
        if (yt == eos_id) { *done = 1; ++t; break; }
    }
    *n_out = n;
    *active_out = active;
    L_out[0] = L[0];
    L_out[1] = L[1];
    *len_out = len;
    *lat_ms = lat;
    *iters = t;
}

/* ------------------------------------------------------------------------
 * Sampled token (Section 3.1 says y_t is "sampled" from p_t; the sampler is
 * not specified -- reading: y_t ~ softmax(z / T_s) drawn by the Gumbel-max
 * construction from a counter-based generator, so that both implementations
 * draw the same numbers without exchanging them).
 * ------------------------------------------------------------------------ */

/*
 * Philox-4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
 * as 1, 2, 3", SC'11): ten rounds of
 *     (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0))
 * with the key bumped by the Weyl constants (W0, W1) between rounds.
 */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += W0; k1 += W1; }
        uint64_t p0 = (uint64_t)M0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * The uniform attached to vocabulary entry v of output row `row` at draw number `draw`:
 * word (v mod 4) of Philox(counter = (v div 4, row, draw_lo, draw_hi), key = (seed_lo, seed_hi)),
 * mapped to U = ((x >> 9) + 1/2) / 2^23, an odd multiple of 2^-24 strictly inside (0, 1), which
 * both float32 and float64 hold exactly.
 */
double oracle_sample_uniform(uint64_t seed, uint64_t draw, uint32_t row, uint32_t v)
{
    uint32_t ctr[4] = {v >> 2, row, (uint32_t)draw, (uint32_t)(draw >> 32)};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    uint32_t x = out[v & 3u];
    return ((double)(x >> 9) + 0.5) / 8388608.0;
}

/*
 * Gumbel-max draw: tok = argmax_v ( z[v] / temperature - ln(-ln U_v) ), lowest index on ties;
 * the argmax of logits plus independent standard Gumbel noise is distributed as softmax(z / T_s).
 * gap = best score minus the runner-up's.  NaN logits never win; 0 if all are NaN.
 */
void oracle_sample_token(const double *z, int V, double temperature, uint64_t seed, uint64_t draw,
                         uint32_t row, int32_t *tok, double *gap)
{
    int best = -1;
    double best_s = 0.0, second = -INFINITY;
    for (int v = 0; v < V; ++v) {
        if (isnan(z[v])) continue;
        double u = oracle_sample_uniform(seed, draw, row, (uint32_t)v);
        double s = z[v] / temperature - log(-log(u));
        if (best < 0) { best = v; best_s = s; }
        else if (s > best_s) { second = best_s; best = v; best_s = s; }
        else if (s > second) second = s;
    }
    if (best < 0) { *tok = 0; *gap = NAN; return; }
    *tok = (int32_t)best;
    *gap = best_s - second;
}

/* Sampled tokens for R rows (same row addressing as oracle_head_rows); row r draws with row id r. */
void oracle_sample_rows(const uint16_t *hidden, const int32_t *row_idx, const uint16_t *w_head,
                        int R, int d, int V, double temperature, uint64_t seed, uint64_t draw,
                        int32_t *tok, double *gap)
{
    double *z = (double *)malloc((size_t)V * sizeof(double));
    for (int r = 0; r < R; ++r) {
        size_t src = row_idx ? (size_t)row_idx[r] : (size_t)r;
        oracle_logits_row(hidden + src * (size_t)d, w_head, d, V, z);
        oracle_sample_token(z, V, temperature, seed, draw, (uint32_t)r, &tok[r], &gap[r]);
    }
    free(z);
}

/* ------------------------------------------------------------------------
 * R-Stitch+ router forward (the "Architecture and Overhead of Router" appendix:
 * a small feed-forward network on the hidden state -- 6 FFN blocks with GELU and
 * residual connections, then normalisation, then a two-head linear layer).  The
 * paper gives neither widths nor weights; the reading taken is
 *     x0 = W_in s + b_in                                   (d -> h)
 *     x_{l+1} = x_l + W2_l GELU(W1_l x_l + b1_l) + b2_l      (h -> ff -> h), l = 0 .. n_blocks-1
 *     y = LayerNorm(x) * g + beta                           (eps = 1e-5, biased variance)
 *     logits = W_out y + b_out                              (h -> 2: SLM, LLM)
 * with the exact (erf) GELU.  Algorithm 1: switch = (argmax_a pi(a | s_t) == LLM).
 * ------------------------------------------------------------------------ */
static double gelu_exact(double x) { return 0.5 * x * (1.0 + erf(x / sqrt(2.0))); }

/* hidden: bf16 bits [d].  All weights fp32, row-major as named above.  logits[2]. */
void oracle_router_row(const uint16_t *hidden, int d, int h, int ff, int n_blocks,
                       const float *W_in, const float *b_in, const float *W1, const float *b1,
                       const float *W2, const float *b2, const float *ln_g, const float *ln_b,
                       const float *W_out, const float *b_out, double *logits)
{
    double *x = (double *)malloc((size_t)h * sizeof(double));
    double *t = (double *)malloc((size_t)ff * sizeof(double));
    for (int i = 0; i < h; ++i) {
        double acc = (double)b_in[i];
        for (int k = 0; k < d; ++k) acc += (double)W_in[(size_t)i * d + k] * bf16_to_double(hidden[k]);
        x[i] = acc;
    }
    for (int l = 0; l < n_blocks; ++l) {
        const float *w1 = W1 + (size_t)l * ff * h, *w2 = W2 + (size_t)l * h * ff;
        for (int j = 0; j < ff; ++j) {
            double acc = (double)b1[(size_t)l * ff + j];
            for (int i = 0; i < h; ++i) acc += (double)w1[(size_t)j * h + i] * x[i];
            t[j] = gelu_exact(acc);
        }
        for (int i = 0; i < h; ++i) {
            double acc = (double)b2[(size_t)l * h + i];
            for (int j = 0; j < ff; ++j) acc += (double)w2[(size_t)i * ff + j] * t[j];
            x[i] += acc;                                    /* residual */
        }
    }
    double mean = 0.0, var = 0.0;
    for (int i = 0; i < h; ++i) mean += x[i];
    mean /= (double)h;
    for (int i = 0; i < h; ++i) var += (x[i] - mean) * (x[i] - mean);
    var /= (double)h;
    const double inv = 1.0 / sqrt(var + 1e-5);
    for (int a = 0; a < 2; ++a) {
        double acc = (double)b_out[a];
        for (int i = 0; i < h; ++i)
            acc += (double)W_out[(size_t)a * h + i] * ((x[i] - mean) * inv * (double)ln_g[i] + (double)ln_b[i]);
        logits[a] = acc;
    }
    free(x);
    free(t);
}

/* R rows (row r reads hidden[row_idx[r]] when row_idx != NULL); logits [R, 2];
 * switch_llm[r] = 1 iff the LLM logit is strictly larger (a tie keeps the SLM). */
void oracle_router_rows(const uint16_t *hidden, const int32_t *row_idx, int R, int d, int h, int ff,
                        int n_blocks, const float *W_in, const float *b_in, const float *W1,
                        const float *b1, const float *W2, const float *b2, const float *ln_g,
                        const float *ln_b, const float *W_out, const float *b_out, double *logits,
                        uint8_t *switch_llm)
{
    for (int r = 0; r < R; ++r) {
        size_t src = row_idx ? (size_t)row_idx[r] : (size_t)r;
        oracle_router_row(hidden + src * (size_t)d, d, h, ff, n_blocks, W_in, b_in, W1, b1, W2, b2, ln_g, ln_b,
                          W_out, b_out, logits + 2 * (size_t)r);
        switch_llm[r] = logits[2 * r + 1] > logits[2 * r] ? 1 : 0;
    }
}
