/*
 * rstitch.h -- C ABI of the R-Stitch routing-decision library (sm_100a).
 *
 * One call evaluates, for every active sequence of a hybrid SLM/LLM decode
 * step, the tail of the model forward and the routing decision of the paper:
 *
 *   S1  logits   z[r,v] = sum_k hidden[r,k] * W_head[v,k]      (Section 3.1: p_t = f(y_{1:t-1}))
 *   S2  entropy  H[r]   = -sum_v p_v ln p_v,  p = softmax(z_r) (Eq. 1, numerator; nats)
 *   S3  token    tok[r] = argmax_v z[r,v], lowest index on ties (Section 3.1, y_t; greedy reading)
 *   S4  rule     mask[b] = H[decision row of b] > tau           (Eq. 2; Algorithm 1 "if H_t > tau")
 *   S5  compaction  llm_idx = ascending {b : mask[b] = 1}, llm_count = |llm_idx|
 *   S6  spans    llm_span[j] = seq_len[llm_idx[j]] - kv_len[llm_idx[j]]  (Algorithm 1, prefill branch)
 *                llm_row_off = exclusive prefix sum of llm_span, llm_row_off[llm_count] = total rows
 *
 * On the SLM head mask = 1 hands the step to the LLM (the SLM token is
 * discarded by the caller); on the LLM head mask = 1 keeps the LLM active and
 * mask = 0 returns control to the SLM.  Logits are never written to memory.
 *
 * Units: ent_out and tau are in nats.  The paper's normalised threshold
 * (Eq. 1 divides by ln V) is tau_nats = tau_paper * ln V; pass
 * RSTITCH_TAU_NORMALIZED to have the library do that multiplication.
 *
 * Conventions
 *  - Every entry point returns an int status (0 = RSTITCH_OK, < 0 = error) and
 *    never throws, exits or traps.  Arguments are validated on the host before
 *    anything is launched; a failed validation launches nothing.
 *  - Unless a parameter says "host", pointers are DEVICE pointers owned by the
 *    caller.  The library neither frees nor reallocates them.  Device pointers
 *    must be 16-byte aligned (hidden, W_head) or naturally aligned (the rest).
 *  - Calls are asynchronous on the given CUDA stream: outputs are valid once
 *    that stream has been synchronised.  llm_count stays on the device so that
 *    the next model's step can be enqueued without a host round trip.
 *  - Host threads: a handle, and the per-device internal handle behind the entry points that take none
 *    (rstitch_route, rstitch_compact, rstitch_route_static's set-up), may be used by one host thread at
 *    a time.  Different handles may be used from different threads at once.
 *  - A routing call enqueues two kernels (the head kernel and the kernel that merges its per-block
 *    statistics and decides) with programmatic stream serialisation: the call's own head kernel may begin
 *    to read W_head while the kernel before it on the stream is still running, and waits for that kernel
 *    to complete before it reads anything else.  W_head must therefore not be written by a kernel
 *    that may still be running then -- the kernel enqueued directly before the call on the same stream
 *    and, if that one was itself launched with programmatic serialisation, those before it (weights are
 *    not expected to be); every other input may be.
 *  - bf16 tensors are row-major with the contraction index k contiguous.
 *  - Non-finite inputs: a row whose entropy is NaN is routed (mask = 1), its
 *    token is the lowest index of the largest non-NaN logit (0 if none), and
 *    the row is counted in rstitch_devstat_t.nan_rows.
 */
#ifndef RSTITCH_H_
#define RSTITCH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------ */
#define RSTITCH_OK                     0
#define RSTITCH_ERR_INVALID_ARG      (-1)  /* null pointer, negative size, non-finite tau, bad flag mix */
#define RSTITCH_ERR_BAD_ALIGN        (-2)  /* a pointer misses its alignment */
#define RSTITCH_ERR_UNSUPPORTED_SHAPE (-3) /* d % 8 != 0, d < 8, V < 2, or a size above the handle's maxima */
#define RSTITCH_ERR_CUDA             (-4)  /* a CUDA runtime or driver call failed */
#define RSTITCH_ERR_WORKSPACE        (-5)  /* caller workspace too small or misaligned */
#define RSTITCH_ERR_TIMEOUT          (-6)  /* a bounded device-side wait gave up (see rstitch_last_status) */

/* ---- flags for rstitch_args_t.flags ------------------------------------ */
#define RSTITCH_TAU_NORMALIZED   0x1u  /* tau is the paper's normalised threshold in [0,1]; multiplied by ln V */
#define RSTITCH_SAMPLE           0x2u  /* tok_out is sampled from softmax(z / temperature), not the greedy token */
#define RSTITCH_PATH_GEMV        0x10u /* testing only: force the CUDA-core streaming kernel */
#define RSTITCH_PATH_UMMA        0x20u /* testing only: force the tcgen05 tensor-core kernel */

typedef struct rstitch_handle_s *rstitch_handle_t;

/*
 * Arguments of the extended call.  Zero-initialise, then fill.
 *
 *   hidden      bf16 [n_src, d]   final hidden states
 *   W_head      bf16 [V, d]       LM-head weights (no bias)
 *   R           rows evaluated (each gives tok_out[r], ent_out[r])
 *   B           sequences decided (route_mask has B entries).  Without row_seq, B must equal R
 *               and sequence b is decided by row b.
 *   n_src       rows present in hidden (only used to bound row_idx; 0 means R)
 *   row_idx     optional int32 [R]: row r reads hidden[row_idx[r]] -- the LLM head evaluated on the
 *               compacted subset llm_idx of an earlier SLM call.  Out-of-range entries are not
 *               dereferenced; they read row 0 and are counted in devstat.bad_row_idx.
 *   row_seq     optional int32 [R], non-decreasing sequence ids in [0, B): the rows of one sequence are
 *               one stitched span pushed through a prefill.  A prefill yields one (p_t, y_t), at the
 *               end of the span (Algorithm 1, prefill branch), so sequence b is decided by its LAST
 *               row; sequences without rows get mask 0.
 *   n_rows_dev  optional device int32 [1]: the live row count (<= R), e.g. the llm_count of an earlier
 *               call.  Rows r >= *n_rows_dev are skipped and their outputs left untouched; B is
 *               clamped the same way.  Not allowed together with row_seq.
 *   seq_len, kv_len   optional int32 [B] (both or neither): |x + y| and the KV-cache length L of the
 *               model that takes over, per sequence.
 *   tok_out     int32 [R];  ent_out float32 [R] (nats)
 *   route_mask  uint8 [B];  llm_idx int32 [B] (entries >= llm_count are left untouched);
 *   llm_count   int32 [1]
 *   llm_span    optional int32 [B], llm_row_off optional int32 [B + 1] (required iff seq_len is given).
 *               A routed sequence with span < 1 is counted in devstat.bad_span.
 *   temperature, seed, draw   with RSTITCH_SAMPLE, tok_out[r] is a draw from softmax(z_r / temperature)
 *               instead of the greedy token (Section 3.1 says y_t is sampled and names no sampler): the
 *               Gumbel-max construction tok = argmax_v (z_v / T_s - ln(-ln U_v)), lowest index on ties,
 *               with U_v word (v mod 4) of Philox-4x32-10(counter = (v div 4, r, draw), key = seed) mapped
 *               to ((x >> 9) + 1/2) / 2^23.  Entropy, mask and compaction do not depend on the draw.
 *   workspace   optional caller scratch of at least rstitch_workspace_bytes(R, d, V) bytes, 256-byte
 *               aligned; NULL uses the handle's own.  Two calls in flight at once on different
 *               streams must not share a workspace.
 */
struct rstitch_alg1_tail_s;
typedef struct rstitch_args_s {
    const void    *hidden;
    const void    *W_head;
    int32_t        R, B, d, V, n_src;
    float          tau;
    uint32_t       flags;
    const int32_t *row_idx;
    const int32_t *row_seq;
    const int32_t *n_rows_dev;
    const int32_t *seq_len;
    const int32_t *kv_len;
    int32_t       *tok_out;
    float         *ent_out;
    uint8_t       *route_mask;
    int32_t       *llm_idx;
    int32_t       *llm_count;
    int32_t       *llm_span;
    int32_t       *llm_row_off;
    void          *workspace;
    size_t         workspace_bytes;
    /* with RSTITCH_SAMPLE (ignored otherwise): */
    float          temperature;     /* T_s > 0 */
    uint64_t       seed;            /* generator key */
    uint64_t       draw;            /* draw number: use a new one for every step */
    /* optional (NULL: none): Algorithm 1's decision block run by this call itself, see rstitch_alg1_tail_t */
    const struct rstitch_alg1_tail_s *alg1_tail;
} rstitch_args_t;

/* Device status word, accumulated since the handle was created or last read. */
typedef struct rstitch_devstat_s {
    uint32_t nan_rows;      /* rows whose entropy came out NaN (routed, see above) */
    uint32_t bad_row_idx;   /* row_idx entries outside [0, n_src) */
    uint32_t bad_span;      /* routed sequences with seq_len - kv_len < 1 */
    uint32_t timeouts;      /* bounded device-side waits that gave up */
    uint32_t timeout_site;  /* where the last one gave up (kernel-internal site id) */
    uint32_t launches;      /* kernels enqueued through this handle (counted on the host) */
    uint32_t reserved[2];
} rstitch_devstat_t;

/*
 * Basic form (the routing problem as the paper states it, batched): B rows, one decision per row,
 * S1-S5.  Runs on the legacy default stream with a per-device internal handle that is created on
 * first use (that first call allocates device memory).  B = 0 is valid and sets *llm_count = 0.
 */
int rstitch_route(const void *hidden /* bf16 [B,d] */, const void *W_head /* bf16 [V,d] */,
                  int B, int d, int V, float tau /* nats */,
                  int32_t *tok_out /* [B] */, float *ent_out /* [B], nats */,
                  uint8_t *route_mask /* [B] */, int32_t *llm_idx /* [B] */,
                  int32_t *llm_count /* [1] */);

/* Extended form, same arithmetic: explicit handle, stream (a cudaStream_t passed as void*), row
 * gather, multi-row spans, S6.  See rstitch_args_t. */
int rstitch_route_ex(rstitch_handle_t h, const rstitch_args_t *a, void *cuda_stream);

/*
 * Same decision as rstitch_route with HOST buffers for the per-step data: hidden_host (bf16 [B,d],
 * ideally pinned) is copied to the device, the step runs, and tok/ent/mask/llm_idx/llm_count are
 * copied back to the given host buffers; the call returns after the stream has been synchronised.
 * W_head is a model weight and stays a device pointer.  Staging buffers live in the handle.
 */
int rstitch_route_host(rstitch_handle_t h, const void *hidden_host, const void *W_head_dev,
                       int B, int d, int V, float tau,
                       int32_t *tok_host, float *ent_host, uint8_t *mask_host,
                       int32_t *llm_idx_host, int32_t *llm_count_host, void *cuda_stream);

/*
 * rstitch_route_ex with HOST buffers for everything that changes per step, for a host-driven decode
 * loop (Algorithm 1 run from the host): in *a, hidden (bf16 [n_src,d]), row_idx, row_seq, seq_len,
 * kv_len and every output pointer are host pointers (ideally pinned); W_head stays a device pointer.
 * n_rows_dev and workspace must be NULL (the live row count is simply R, and the scratch is the
 * handle's).  The inputs are copied to a staging block owned by the handle, the step runs, the
 * outputs are copied back and the call returns after the stream has been synchronised.  llm_idx
 * comes back in full (B entries); only the first llm_count are meaningful.  The first call, and any
 * call needing a larger staging block, allocates device memory.
 */
int rstitch_route_ex_host(rstitch_handle_t h, const rstitch_args_t *a, void *cuda_stream);

/*
 * The same decision as rstitch_route (S1-S5, B rows, one decision per row) for callers that cannot
 * allocate device memory.  (The paper has no counterpart; this is a deployment variant.)
 *
 * Who needs it: code running inside a serving engine whose memory pool already owns the whole
 * device, a decode loop that cannot afford the device-wide synchronisation an allocation may cause,
 * or a process whose device budget is fixed at start-up.  This entry point calls no cudaMalloc,
 * cudaFree or any other allocating routine, on any call: its scratch (ticket counter, per-slice
 * partial statistics, status word) is a fixed array of about RSTITCH_STATIC_MAX_ROWS * 20 KiB inside
 * the library image, which every GPU that loads the library holds until the process exits.
 *
 *  - B > RSTITCH_STATIC_MAX_ROWS returns RSTITCH_ERR_UNSUPPORTED_SHAPE (the scratch is fixed); the
 *    other argument rules are those of rstitch_route.  Inputs and outputs are still the caller's.
 *  - The first call on each device looks up the array's device address (no allocation); make that
 *    first call with the device current and before any stream capture begins.
 *  - All calls on a device share the one array, which keeps the previous call's contents: each call
 *    clears what must start at zero on the given stream.  Two calls that overlap on the GPU (different
 *    streams, no ordering between them) race on it; order them.
 *  - No status word is reported back: NaN rows are still routed, but not counted anywhere, and a bounded
 *    device-side wait that gave up (which the other entry points report through rstitch_last_status as
 *    RSTITCH_ERR_TIMEOUT) goes unreported here; the outputs of such a call are undefined.
 */
#define RSTITCH_STATIC_MAX_ROWS 16
int rstitch_route_static(const void *hidden /* bf16 [B,d] */, const void *W_head /* bf16 [V,d] */,
                         int B, int d, int V, float tau /* nats */,
                         int32_t *tok_out, float *ent_out, uint8_t *route_mask, int32_t *llm_idx,
                         int32_t *llm_count, void *cuda_stream);

/* ---- the steps of Algorithm 1 either side of the decision, batched ------------------------------ */

/* Eq. 5 coefficients of one model (the appendix on latency regression prints three sets), ms:
 * T(N_inf, N_kv) = a N_inf N_kv + b N_inf^2 + c N_inf + d; a decode step is N_inf = 1 (Eq. 6). */
typedef struct rstitch_latency_model_s { double a, b, c, d; } rstitch_latency_model_t;

/*
 * Per-sequence state of the hybrid decode loop (Algorithm 1), a structure of DEVICE arrays owned by
 * the caller, B entries each unless noted.  The paper runs one sequence; here every sequence of a
 * batch carries its own copy of the algorithm's variables and all advance one loop iteration per round.
 *   active   0 = SLM, 1 = LLM          kv_slm, kv_llm   L^SLM, L^LLM (KV-cache sizes)
 *   seq_len  |x + y|                   n_out            |y|
 *   done     1 once EOS was appended (a sequence is finished when done = 1 or iters = T_max)
 *   iters    loop iterations executed
 *   kept     [2 B]: tokens kept from the SLM at [b], from the LLM at [B + b]
 *   steps    [2 B]: model steps taken, same layout (discarded SLM steps included)
 *   lat_ms   float64: latency estimate, the sum of Eq. 5 over every model step taken
 *   y        [B, y_cap] generated tokens (tokens past y_cap are counted but not stored)
 */
typedef struct rstitch_alg1_state_s {
    int32_t *active, *kv_slm, *kv_llm, *seq_len, *n_out, *done, *iters, *kept, *steps;
    double  *lat_ms;
    int32_t *y;
    int32_t  y_cap;
} rstitch_alg1_state_t;

/* Algorithm 1's initialisation: both caches empty, y = [], active = SLM, |x + y| = prompt_len[b]. */
int rstitch_alg1_init(const rstitch_alg1_state_t *s, int B, const int32_t *prompt_len /* device [B] */,
                      void *cuda_stream);

/*
 * Before the engine of `model` (0 = SLM, 1 = LLM) runs in this round: the prefill-or-decode test of
 * Algorithm 1 for every sequence that is not done and whose active model is `model`.
 *   run_idx [B]      ascending ids of those sequences;  run_count [1] their number
 *   n_inf [B]        per run entry: tokens to process -- |x + y| - L (prefill of the missing span)
 *                    when L < |x + y|, else 1 (decode);  n_kv [B]: L before the step
 *   row_off [B + 1]  exclusive prefix sum of n_inf: the row offsets of the model's batch
 * Side effects per selected sequence: L <- |x + y| + 1 (prefill) or L + 1 (decode), iters += 1,
 * steps += 1, lat_ms += Eq. 5 with *latency (a HOST pointer).  A sequence that has used t_max
 * iterations is no longer selected.  All outputs are device arrays.  One round of the loop is
 * plan(SLM), plan(LLM), the two model steps and routing decisions, commit(SLM), commit(LLM): both
 * plans come before either commit (with separate run-list buffers), so that a sequence handed over
 * by a commit does not run a second time in the same round.
 */
int rstitch_alg1_plan(const rstitch_alg1_state_t *s, int B, int model, int t_max,
                      const rstitch_latency_model_t *latency, int32_t *run_idx, int32_t *run_count,
                      int32_t *n_inf, int32_t *n_kv, int32_t *row_off, void *cuda_stream);

/*
 * After the routing decision of that model's batch (Algorithm 1 from "if H_t > tau" to the EOS test):
 * run entry j (sequence run_idx[j]) has route_mask[j] = (H_t > tau) and the token tok[row], row being
 * the LAST row of its span (row_off[j + 1] - 1; with row_off = NULL, row = j).
 *   SLM, mask 1: y_t discarded, L^SLM rolled back by the entry the step added, active <- LLM
 *   LLM, mask 0: active <- SLM, y_t kept          otherwise: y_t kept, same model
 * A kept token is appended (y, n_out, seq_len, kept) and ends the sequence if it equals eos_id.
 */
int rstitch_alg1_commit(const rstitch_alg1_state_t *s, int B, int model, const int32_t *run_idx,
                        const int32_t *run_count, const int32_t *row_off, const int32_t *tok,
                        const uint8_t *route_mask, int32_t eos_id, void *cuda_stream);

/*
 * The same steps without launches of their own: a routing call whose rstitch_args_t.alg1_tail points to one
 * of these (a HOST structure, read during the call) goes on, in the block that has just written its tokens
 * and mask, with the decision block of Algorithm 1 for the model's batch (exactly rstitch_alg1_commit with
 * tok = tok_out and route_mask = route_mask of the call) and then, with plan_next != 0, with the planning of
 * the next round for BOTH models (exactly rstitch_alg1_plan for model 0, then 1, writing the next_* arrays,
 * which may be the buffers of the run lists just consumed).  A round of the loop is then two launches:
 * the SLM head with {model 0, plan_next 0}, the LLM head with {model 1, plan_next 1}; only the first
 * round's plans are calls of their own.  The routing call's rows are the model's batch: n_rows_dev =
 * run_count, B at least the largest run count (without multi-row spans, row j belongs to run entry j and
 * row_off is NULL).  Accepted by rstitch_route_ex and rstitch_shard_route.
 */
typedef struct rstitch_alg1_tail_s {
    const rstitch_alg1_state_t *state;     /* HOST pointer to the structure of device arrays */
    int32_t n_seq;                         /* sequences in the state */
    int32_t model;                         /* 0 = SLM, 1 = LLM: whose batch this call decides */
    const int32_t *run_idx, *run_count;    /* DEVICE: the model's run list from the last planning */
    const int32_t *row_off;                /* DEVICE, optional: row offsets of the run entries' spans */
    int32_t eos_id;
    int32_t plan_next;                     /* non-zero: plan the next round for both models afterwards */
    int32_t t_max;                         /* as in rstitch_alg1_plan (with plan_next) */
    rstitch_latency_model_t latency[2];    /* Eq. 5 coefficients of model 0 and 1 (with plan_next) */
    int32_t *next_run_idx[2], *next_run_count[2], *next_n_inf[2], *next_n_kv[2], *next_row_off[2];
} rstitch_alg1_tail_t;

/* ---- R-Stitch+ router ---------------------------------------------------------------------------- */

/*
 * Weights of the lightweight router (the appendix "Architecture and Overhead of Router": 6 FFN blocks
 * with GELU and residual connections, a normalisation, a two-head linear layer, on the hidden state;
 * widths are not given in the paper and are parameters here).  DEVICE pointers to float32, row-major:
 *   W_in [h, d], b_in [h]            x0 = W_in s + b_in
 *   W1 [n_blocks, ff, h], b1 [n_blocks, ff], W2 [n_blocks, h, ff], b2 [n_blocks, h]
 *                                    x <- x + W2 GELU(W1 x + b1) + b2   (exact erf GELU)
 *   ln_g [h], ln_b [h]               y = LayerNorm(x) ln_g + ln_b       (eps 1e-5)
 *   W_out [2, h], b_out [2]          logits = W_out y + b_out           (index 0 = SLM, 1 = LLM)
 * Limits: h <= 256, ff <= 1024, d <= 16384 and a multiple of 4, W_in 16-byte aligned.
 */
typedef struct rstitch_router_s {
    int32_t d, h, ff, n_blocks;
    const float *W_in, *b_in, *W1, *b1, *W2, *b2, *ln_g, *ln_b, *W_out, *b_out;
} rstitch_router_t;

/*
 * Algorithm 1, R-Stitch+ branch: for the rows whose entropy exceeded tau, switch = (argmax_a pi(a | s_t)
 * == LLM).  Row r reads hidden[row_idx[r]] (bf16 [n_src, d]; row_idx optional) -- typically row_idx =
 * llm_idx and n_rows_dev = llm_count of the SLM head's call, both on the device.
 *   logits_out  float32 [R, 2];  switch_out optional uint8 [R] (1 = hand the step to the LLM; a tie keeps
 *   the SLM);  refine_mask optional uint8 [n_src] (needs row_idx): refine_mask[row_idx[r]] = switch, which
 *   turns the entropy rule's route_mask into the router's; compact it again with rstitch_compact.
 * An entry of row_idx outside [0, n_src) reads row 0, gets switch 0 and leaves refine_mask alone; R > 0 with
 * n_src = 0 is an invalid argument.
 */
int rstitch_router_forward(const rstitch_router_t *w, const void *hidden, int n_src, const int32_t *row_idx,
                           const int32_t *n_rows_dev, int R, float *logits_out, uint8_t *switch_out,
                           uint8_t *refine_mask, void *cuda_stream);

/*
 * The R-Stitch+ decision in one launch: rstitch_router_forward with refine_mask = route_mask, followed in
 * the same kernel (its last block to finish) by the ordered compaction of the refined route_mask [n_src]
 * into llm_idx [n_src] and llm_count [1], exactly as rstitch_compact(route_mask, n_src, ...) would give
 * afterwards.  row_idx, route_mask and llm_count are required; typically row_idx = llm_idx of the SLM head's
 * call (the list is consumed before it is rewritten only if the two are DIFFERENT buffers: pass another
 * llm_idx here).  n_src <= 65536.  Calls of this function that may overlap on one device must be ordered
 * by the caller (they share one ticket counter).
 */
int rstitch_router_route(const rstitch_router_t *w, const void *hidden, int n_src, const int32_t *row_idx,
                         const int32_t *n_rows_dev, int R, float *logits_out, uint8_t *switch_out,
                         uint8_t *route_mask, int32_t *llm_idx, int32_t *llm_count, void *cuda_stream);

/*
 * The SLM's step of an R-Stitch+ round (Algorithm 1: "if H_t > tau: switch <- (argmax_a pi(a | s_t) = LLM);
 * if active = SLM and switch: discard y_t, roll back, active <- LLM"; Section 3.3: low-entropy tokens
 * always stay with the SLM).  Issued behind the SLM head's rstitch_route_ex call of the round, which was
 * made WITHOUT an alg1_tail: rstitch_router_route on that call's llm_idx / llm_count (the run entries
 * whose entropy exceeded tau) refines its route_mask to (H_t > tau and switch), and the kernel's last block
 * then runs Algorithm 1's decision block for the SLM's batch on the refined mask and the call's tokens
 * -- exactly rstitch_alg1_commit(model 0, tok, route_mask) -- and, with plan_next, the next planning.  A
 * round is then three launches (SLM head, this, LLM head with its own alg1_tail), all on the device.
 *   n_seq_dev   optional device int32 [1]: the live length of route_mask (the SLM call's n_rows_dev, i.e.
 *               its run count); entries at or past it are neither compacted nor decided.  NULL: n_src.
 *   tok         device int32: the SLM call's tok_out;  alg1_tail: as in rstitch_args_t, model must be 0.
 * The other arguments are those of rstitch_router_route.  Entries of row_idx outside [0, n_src) read row 0,
 * leave route_mask alone and get switch 0.
 */
int rstitch_router_route_alg1(const rstitch_router_t *w, const void *hidden, int n_src, const int32_t *n_seq_dev,
                              const int32_t *row_idx, const int32_t *n_rows_dev, int R, float *logits_out,
                              uint8_t *switch_out, uint8_t *route_mask, int32_t *llm_idx, int32_t *llm_count,
                              const int32_t *tok, const rstitch_alg1_tail_t *alg1_tail, void *cuda_stream);

/* Handle: owns the scratch memory and the device status word for problems up to the given maxima on
 * the current device.  rstitch_destroy(NULL) is a no-op. */
int rstitch_create(rstitch_handle_t *out, int maxR, int max_d, int maxV);
int rstitch_destroy(rstitch_handle_t h);

/* Scratch bytes one call of that shape needs (0 for an unsupported shape). */
size_t rstitch_workspace_bytes(int R, int d, int V);

/* ---- vocabulary-parallel head ------------------------------------------------------------------- */

/*
 * The LM head split by vocabulary rows across GPUs (tensor-parallel head): GPU g holds W_head rows
 * [v_base_g, v_base_g + V_g) and every GPU the same hidden rows.  Eq. 1 needs sums over the whole
 * vocabulary; they come from per-shard statistics, 20 bytes per row, that are gathered and merged:
 *   1. rstitch_shard_stats on every GPU: the head kernels on the shard, nothing decided;
 *   2. the caller gathers the shards' outputs into one buffer, shard-major (an all-gather over NCCL;
 *      this library does no communication);
 *   3. rstitch_shard_route on any GPU that needs the decision: merge in ascending shard order, then
 *      entropy, token, Eq. 2, mask, compaction and spans exactly as rstitch_route_ex.
 * The result equals the single-GPU call on the whole vocabulary up to the rounding order of the merge.
 *
 * rstitch_shard_stats reads from *a: hidden, W_head (the shard's rows), R, d, V (= V_g, the shard's row
 * count), n_src, row_idx, n_rows_dev, flags (RSTITCH_SAMPLE and the path flags), temperature, seed, draw,
 * workspace; B, tau and every output pointer are ignored.  v_base >= 0 is the global index of the shard's
 * first row; token indices and the sampling noise use global indices, so the draw does not depend on the
 * split.  shard_stats: DEVICE, R x RSTITCH_SHARD_WORDS 32-bit words, per row
 *   float m (largest logit), float s = sum e^(z-m), float u = sum e^(z-m) (z-m), float best score,
 *   int32 global index of the best entry (INT32_MAX if the shard saw no finite logit).
 * Rows at or past *n_rows_dev are not written.
 */
#define RSTITCH_SHARD_WORDS 5
#define RSTITCH_MAX_SHARDS  1024
int rstitch_shard_stats(rstitch_handle_t h, const rstitch_args_t *a, int32_t v_base, void *shard_stats,
                        void *cuda_stream);

/*
 * gathered: DEVICE, [n_shards][R][RSTITCH_SHARD_WORDS] words (shard g's shard_stats at word offset
 * g * R * RSTITCH_SHARD_WORDS), 1 <= n_shards <= RSTITCH_MAX_SHARDS.  Reads from *a: R, B, V (the WHOLE
 * vocabulary size, which bounds the token index and scales tau with RSTITCH_TAU_NORMALIZED), tau, flags,
 * row_seq, seq_len, kv_len, n_rows_dev and the output pointers, with the meaning they have in
 * rstitch_route_ex; hidden, W_head, d, row_idx and workspace are ignored.  One kernel launch.
 */
int rstitch_shard_route(rstitch_handle_t h, const rstitch_args_t *a, const void *gathered, int32_t n_shards,
                        void *cuda_stream);

/* S5 alone: ordered compaction of a uint8 mask [B] into idx [B] and count [1] (warp ballot + prefix
 * sums).  Needs no handle; scratch for very large B is taken from a per-device internal handle. */
int rstitch_compact(const uint8_t *mask, int B, int32_t *idx, int32_t *count, void *cuda_stream);

/* Synchronises the handle's last stream, copies the device status word to *out (host) and clears it.
 * h = NULL reads the per-device internal handle behind rstitch_route / rstitch_compact.
 * Returns RSTITCH_ERR_TIMEOUT if a bounded wait gave up since the last read. */
int rstitch_last_status(rstitch_handle_t h, rstitch_devstat_t *out);

/*
 * Self-test of the error path of the kernels' bounded waits (every wait on a copy or on the tensor pipe
 * gives up after a cycle limit instead of hanging): enqueues one tiny kernel whose only wait can never be
 * satisfied and is limited to about a millisecond.  It gives up, records that in the status word like any
 * other wait and returns; the next rstitch_last_status(h, ...) returns RSTITCH_ERR_TIMEOUT with
 * timeouts = 1 and timeout_site = RSTITCH_SELFTEST_SITE, and the handle and the context stay usable.
 */
#define RSTITCH_SELFTEST_SITE 0x7e57u
int rstitch_selftest_wait(rstitch_handle_t h, void *cuda_stream);

/*
 * Measurement aid (not part of the routing path): one pass over buf [bytes] (device, 16-byte aligned) that
 * only reads it, through the pipeline of the streaming head kernel (one block per SM, bulk copies of a
 * contiguous slice into a shared-memory ring) with nothing done to the bytes.  Timed by the caller with
 * CUDA events it gives the bandwidth ceiling of a read-only stream on this GPU, the regime of the head
 * kernels at small batch (Section 3.1's last linear map read once per step), beside the usual copy
 * figure.  Whole 16 KiB chunks are read; a remainder is skipped.  *gave_up (device, zeroed by the
 * caller) counts bounded waits that ran out, which voids the measurement.
 */
int rstitch_probe_read_stream(const void *buf, size_t bytes, uint32_t *gave_up, void *cuda_stream);

/* Static, never NULL. */
const char *rstitch_status_string(int status);

/* Name of the kernel family a call of that shape takes: "gemv" or "umma" (static string). */
const char *rstitch_path_name(int R, int d, int V, uint32_t flags);

#ifdef __cplusplus
}
#endif
#endif /* RSTITCH_H_ */
