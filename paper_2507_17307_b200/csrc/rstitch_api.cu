// C ABI of the routing-decision library: argument validation, handles, scratch memory and the
// choice of kernel family.  All arithmetic of the path runs in the kernels; nothing here computes.
#include "../../include/rstitch.h"
#include "rstitch_kernels.cuh"

#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

using namespace rstitch;

static_assert(sizeof(DevStat) == sizeof(rstitch_devstat_t), "device status word layout");

struct rstitch_handle_s {
    int      device      = -1;
    int      sm_count    = 0;
    int      maxR = 0, max_d = 0, maxV = 0;
    void    *ws          = nullptr;      // scratch: ticket + partials
    size_t   ws_bytes    = 0;
    DevStat *stat        = nullptr;      // device status word
    int32_t *tile_counts = nullptr;      // scratch of the multi-block compaction
    int      tile_cap    = 0;
    // staging of rstitch_route_host
    void    *st = nullptr;  size_t st_bytes = 0;     // staging block of the host-buffer calls
    void    *st_host = nullptr;  size_t st_host_bytes = 0;   // pinned mirror of its output part
    void    *st_in = nullptr;  size_t st_in_bytes = 0;       // pinned mirror of its input part (small inputs)
    cudaStream_t last_stream = nullptr;
    unsigned launch_count = 0;           // kernels enqueued since the status word was last read
    TmapCache tmaps;                     // encoded tensor maps of the tensor-core kernels
};

namespace rstitch {

// rstitch_alg1_tail_t (host) -> the device copy the tails carry; false: a bad structure.
bool make_alg1_tail(const rstitch_alg1_tail_t *t, Alg1Tail *out)
{
    out->on = 0;
    if (!t) return true;
    if (!alg1_state_ok(t->state) || t->n_seq < 0 || (t->model != 0 && t->model != 1) || !t->run_count ||
        (t->n_seq > 0 && !t->run_idx))
        return false;
    out->on = 1;
    out->s = *t->state;
    out->n_seq = t->n_seq; out->model = t->model;
    out->run_idx = t->run_idx; out->run_count = t->run_count; out->row_off = t->row_off;
    out->eos_id = t->eos_id; out->plan_next = t->plan_next ? 1 : 0; out->t_max = t->t_max;
    for (int m = 0; m < 2; ++m) {
        out->lat[m] = t->latency[m];
        out->nx_idx[m] = t->next_run_idx[m]; out->nx_cnt[m] = t->next_run_count[m];
        out->nx_ninf[m] = t->next_n_inf[m]; out->nx_nkv[m] = t->next_n_kv[m]; out->nx_off[m] = t->next_row_off[m];
        if (t->plan_next) {
            if (t->t_max < 0 || !out->nx_cnt[m] || !out->nx_off[m]) return false;
            if (t->n_seq > 0 && (!out->nx_idx[m] || !out->nx_ninf[m] || !out->nx_nkv[m])) return false;
            if (!std::isfinite(t->latency[m].a) || !std::isfinite(t->latency[m].b) ||
                !std::isfinite(t->latency[m].c) || !std::isfinite(t->latency[m].d))
                return false;
        }
    }
    return true;
}

}  // namespace rstitch

namespace {

constexpr size_t kMirrorMax = 16 * 1024;        // host-buffer calls: outputs up to this size are written to the host by the kernel
constexpr size_t kPackedInputMax = 64 * 1024;   // host-buffer calls: inputs up to this size travel as one copy
constexpr int kMaxD = 16384;
constexpr int kMaxRows = 16384;

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Rows up to which the CUDA-core streaming kernel is taken.  Measured (us per call, rows 1 / 2 / 3 / 4 / 8):
//   3584 x 152064 head   streaming 160 / 175-189 / 211 / 228 / 453    tcgen05 171 / 173 / 175 / 173 / 173
//   1536 x 151936 head   streaming  77 /  79     / 100 / 101 / 186    tcgen05  81 /  81 /  81 /  82 /  82
// One row streams best as contiguous bulk copies; from two rows on the FMA work shows (and more so on a
// power-capped GPU), while the tensor-core kernel costs the same from 1 to 128 rows.
constexpr int kGemvMaxRows = 1;

size_t ws_partials_bytes(int R, int V)
{
    return partials_bytes((size_t)(R > 0 ? R : 1), max_slices_for(V));
}

// [header][partials][gather buffer of the tensor-core kernel]
size_t ws_bytes_for(int R, int d, int V)
{
    return kWsHeader + ws_partials_bytes(R, V) + ((umma_gather_bytes(R > 0 ? R : 1, d) + 255) / 256) * 256;
}

int shape_status(int R, int d, int V)
{
    if (R < 0) return RSTITCH_ERR_INVALID_ARG;
    if (d < 8 || (d % 8) != 0 || d > kMaxD || V < 2 || R > kMaxRows) return RSTITCH_ERR_UNSUPPORTED_SHAPE;
    return RSTITCH_OK;
}

int grow_handle(rstitch_handle_s *h, int R, int d, int V)
{
    if (R < h->maxR) R = h->maxR;          // the layout depends on all three: never shrink any of them
    if (d < h->max_d) d = h->max_d;
    if (V < h->maxV) V = h->maxV;
    size_t need = ws_bytes_for(R, d, V);
    if (need > h->ws_bytes) {
        if (h->ws) { if (cudaDeviceSynchronize() != cudaSuccess) return RSTITCH_ERR_CUDA; cudaFree(h->ws); h->ws = nullptr; h->ws_bytes = 0; }
        if (cudaMalloc(&h->ws, need) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
        if (cudaMemset(h->ws, 0, kWsHeader) != cudaSuccess) return RSTITCH_ERR_CUDA;
        h->ws_bytes = need;
    }
    if (R > h->maxR) h->maxR = R;
    if (d > h->max_d) h->max_d = d;
    if (V > h->maxV) h->maxV = V;
    return RSTITCH_OK;
}

std::mutex       g_default_mutex;
rstitch_handle_s *g_default[64] = {};

// Per-device handle behind the entry points that take none; grows on demand.
int default_handle(rstitch_handle_s **out, int R, int d, int V)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return RSTITCH_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_default_mutex);
    if (!g_default[dev]) {
        rstitch_handle_t h = nullptr;
        int st = rstitch_create(&h, R > 64 ? R : 64, d, V);
        if (st != RSTITCH_OK) return st;
        g_default[dev] = h;
    }
    int st = grow_handle(g_default[dev], R, d, V);
    if (st != RSTITCH_OK) return st;
    *out = g_default[dev];
    return RSTITCH_OK;
}

enum ValidateMode { kWholeCall = 0, kShardStats = 1, kShardRoute = 2 };

// kShardStats checks what the head reads (no routing argument), kShardRoute what the tail reads and writes.
int validate(const rstitch_handle_s *h, const rstitch_args_t *a, ValidateMode mode = kWholeCall)
{
    if (!h || !a) return RSTITCH_ERR_INVALID_ARG;
    if (mode == kShardStats) {
        int st = shape_status(a->R, a->d, a->V);
        if (st != RSTITCH_OK) return st;
        if (a->n_src < 0) return RSTITCH_ERR_INVALID_ARG;
        if ((a->flags & RSTITCH_PATH_GEMV) && (a->flags & RSTITCH_PATH_UMMA)) return RSTITCH_ERR_INVALID_ARG;
        if (a->flags & ~(RSTITCH_TAU_NORMALIZED | RSTITCH_SAMPLE | RSTITCH_PATH_GEMV | RSTITCH_PATH_UMMA))
            return RSTITCH_ERR_INVALID_ARG;
        if ((a->flags & RSTITCH_SAMPLE) && !(std::isfinite(a->temperature) && a->temperature > 0.f))
            return RSTITCH_ERR_INVALID_ARG;
        if (a->R > 0 && (!a->hidden || !a->W_head)) return RSTITCH_ERR_INVALID_ARG;
        if (!aligned(a->hidden, 16) || !aligned(a->W_head, 16)) return RSTITCH_ERR_BAD_ALIGN;
        if (!aligned(a->row_idx, 4) || !aligned(a->n_rows_dev, 4)) return RSTITCH_ERR_BAD_ALIGN;
        if (a->workspace) {
            if (!aligned(a->workspace, 256) || a->workspace_bytes < ws_bytes_for(a->R, a->d, a->V))
                return RSTITCH_ERR_WORKSPACE;
        } else if (a->R > h->maxR || a->d > h->max_d || a->V > h->maxV) {
            return RSTITCH_ERR_UNSUPPORTED_SHAPE;
        }
        return RSTITCH_OK;
    }
    if (mode == kShardRoute) {
        if (a->R < 0 || a->B < 0 || a->V < 2) return RSTITCH_ERR_INVALID_ARG;
        if (a->R > kMaxRows) return RSTITCH_ERR_UNSUPPORTED_SHAPE;
        if (!std::isfinite(a->tau)) return RSTITCH_ERR_INVALID_ARG;
        if (a->flags & ~(RSTITCH_TAU_NORMALIZED | RSTITCH_SAMPLE | RSTITCH_PATH_GEMV | RSTITCH_PATH_UMMA))
            return RSTITCH_ERR_INVALID_ARG;
        if (!a->llm_count) return RSTITCH_ERR_INVALID_ARG;
        if (a->row_seq == nullptr && a->B != a->R) return RSTITCH_ERR_INVALID_ARG;
        if (a->row_seq != nullptr && a->n_rows_dev != nullptr) return RSTITCH_ERR_INVALID_ARG;
        if ((a->seq_len == nullptr) != (a->kv_len == nullptr)) return RSTITCH_ERR_INVALID_ARG;
        if (a->seq_len && a->B > 0 && (!a->llm_span || !a->llm_row_off)) return RSTITCH_ERR_INVALID_ARG;
        if (a->R > 0 && (!a->tok_out || !a->ent_out)) return RSTITCH_ERR_INVALID_ARG;
        if (a->B > 0 && (!a->route_mask || !a->llm_idx)) return RSTITCH_ERR_INVALID_ARG;
        if (!aligned(a->tok_out, 4) || !aligned(a->ent_out, 4) || !aligned(a->llm_idx, 4) ||
            !aligned(a->llm_count, 4) || !aligned(a->row_seq, 4) || !aligned(a->n_rows_dev, 4) ||
            !aligned(a->seq_len, 4) || !aligned(a->kv_len, 4) || !aligned(a->llm_span, 4) ||
            !aligned(a->llm_row_off, 4))
            return RSTITCH_ERR_BAD_ALIGN;
        return RSTITCH_OK;
    }
    int st = shape_status(a->R, a->d, a->V);
    if (st != RSTITCH_OK) return st;
    if (a->B < 0 || a->n_src < 0) return RSTITCH_ERR_INVALID_ARG;
    if (!std::isfinite(a->tau)) return RSTITCH_ERR_INVALID_ARG;
    if ((a->flags & RSTITCH_PATH_GEMV) && (a->flags & RSTITCH_PATH_UMMA)) return RSTITCH_ERR_INVALID_ARG;
    if (a->flags & ~(RSTITCH_TAU_NORMALIZED | RSTITCH_SAMPLE | RSTITCH_PATH_GEMV | RSTITCH_PATH_UMMA))
        return RSTITCH_ERR_INVALID_ARG;
    if ((a->flags & RSTITCH_SAMPLE) && !(std::isfinite(a->temperature) && a->temperature > 0.f))
        return RSTITCH_ERR_INVALID_ARG;
    if (!a->llm_count) return RSTITCH_ERR_INVALID_ARG;
    if (a->row_seq == nullptr && a->B != a->R) return RSTITCH_ERR_INVALID_ARG;
    if (a->row_seq != nullptr && a->n_rows_dev != nullptr) return RSTITCH_ERR_INVALID_ARG;
    if ((a->seq_len == nullptr) != (a->kv_len == nullptr)) return RSTITCH_ERR_INVALID_ARG;
    if (a->seq_len && a->B > 0 && (!a->llm_span || !a->llm_row_off)) return RSTITCH_ERR_INVALID_ARG;
    if (a->R > 0 && (!a->hidden || !a->W_head || !a->tok_out || !a->ent_out)) return RSTITCH_ERR_INVALID_ARG;
    if (a->B > 0 && (!a->route_mask || !a->llm_idx)) return RSTITCH_ERR_INVALID_ARG;
    if (!aligned(a->hidden, 16) || !aligned(a->W_head, 16)) return RSTITCH_ERR_BAD_ALIGN;
    if (!aligned(a->tok_out, 4) || !aligned(a->ent_out, 4) || !aligned(a->llm_idx, 4) ||
        !aligned(a->llm_count, 4) || !aligned(a->row_idx, 4) || !aligned(a->row_seq, 4) ||
        !aligned(a->n_rows_dev, 4) || !aligned(a->seq_len, 4) || !aligned(a->kv_len, 4) ||
        !aligned(a->llm_span, 4) || !aligned(a->llm_row_off, 4))
        return RSTITCH_ERR_BAD_ALIGN;
    if (a->workspace) {
        if (!aligned(a->workspace, 256) || a->workspace_bytes < ws_bytes_for(a->R, a->d, a->V))
            return RSTITCH_ERR_WORKSPACE;
    } else if (a->R > h->maxR || a->d > h->max_d || a->V > h->maxV) {
        return RSTITCH_ERR_UNSUPPORTED_SHAPE;
    }
    return RSTITCH_OK;
}

bool use_umma(int R, int d, int V, uint32_t flags)
{
    if (flags & RSTITCH_PATH_GEMV) return false;
    if (!umma_shape_ok(R, d, V)) return false;       // tiny shapes stay on the streaming kernel
    if (flags & RSTITCH_PATH_UMMA) return true;
    return R > kGemvMaxRows;
}

// Validated arguments -> kernels.  With shard_stats the head is a vocabulary shard starting at entry
// v_base: per-row statistics go to shard_stats and no routing output is touched.
struct Mirror { const void *src = nullptr; void *dst = nullptr; size_t bytes = 0; };

int enqueue_head(rstitch_handle_s *h, const rstitch_args_t *a, cudaStream_t stream, float *shard_stats,
                 int v_base, Mirror mirror = Mirror())
{
    Alg1Tail alg1;
    if (!make_alg1_tail(shard_stats ? nullptr : a->alg1_tail, &alg1)) return RSTITCH_ERR_INVALID_ARG;
    if (!shard_stats && (a->R == 0 || a->B == 0)) {
        // nothing to evaluate or nothing to decide: the compaction of an empty mask
        if (cudaMemsetAsync(a->llm_count, 0, sizeof(int32_t), stream) != cudaSuccess) return RSTITCH_ERR_CUDA;
        if (a->seq_len && a->llm_row_off &&
            cudaMemsetAsync(a->llm_row_off, 0, sizeof(int32_t), stream) != cudaSuccess) return RSTITCH_ERR_CUDA;
        if (a->R == 0) {
            if (alg1.on) {                 // no rows, but the loop goes on: the block on its own
                if (launch_alg1_tail(alg1, a->tok_out, a->route_mask, stream) != cudaSuccess) {
                    cudaGetLastError();
                    return RSTITCH_ERR_CUDA;
                }
                h->launch_count += 1;
            }
            return RSTITCH_OK;
        }
    }

    HeadArgs ha;
    ha.hidden = a->hidden; ha.W = a->W_head; ha.R = a->R; ha.d = a->d; ha.V = a->V;
    ha.n_src = a->n_src > 0 ? a->n_src : a->R;
    ha.row_idx = a->row_idx; ha.n_rows_dev = a->n_rows_dev;
    ha.sample = SampleArgs{};
    if (a->flags & RSTITCH_SAMPLE) {
        ha.sample.on = 1;
        ha.sample.inv_t = 1.0f / a->temperature;
        ha.sample.k0 = (uint32_t)a->seed; ha.sample.k1 = (uint32_t)(a->seed >> 32);
        ha.sample.d0 = (uint32_t)a->draw; ha.sample.d1 = (uint32_t)(a->draw >> 32);
        ha.sample.v0 = (uint32_t)v_base;
    }

    TailArgs ta;
    ta.R = a->R; ta.B = a->B; ta.V = a->V;
    ta.tau = (a->flags & RSTITCH_TAU_NORMALIZED) ? a->tau * logf((float)a->V) : a->tau;
    ta.row_seq = a->row_seq; ta.seq_len = a->seq_len; ta.kv_len = a->kv_len;
    ta.tok_out = a->tok_out; ta.ent_out = a->ent_out; ta.route_mask = a->route_mask;
    ta.llm_idx = a->llm_idx; ta.llm_count = a->llm_count;
    ta.llm_span = a->llm_span; ta.llm_row_off = a->llm_row_off;
    ta.stat = h->stat;
    ta.shard_stats = shard_stats; ta.v_base = v_base;
    ta.alg1 = alg1;
    ta.mirror_src = (const uint4 *)mirror.src; ta.mirror_dst = (uint4 *)mirror.dst;
    ta.mirror_vec = (uint32_t)(mirror.bytes / 16);

    void *ws = a->workspace ? a->workspace : h->ws;
    Scratch sc = scratch_carve(ws);
    if (a->workspace) {
        // caller scratch: the ticket must start at zero
        if (cudaMemsetAsync(sc.ticket, 0, sizeof(unsigned), stream) != cudaSuccess) return RSTITCH_ERR_CUDA;
    }
    cudaError_t e;
    int launched = 0;
    if (use_umma(a->R, a->d, a->V, a->flags)) {
        // the partials region is sized for the shape the scratch was made for
        size_t part = a->workspace ? ws_partials_bytes(a->R, a->V) : ws_partials_bytes(h->maxR, h->maxV);
        e = launch_head_umma(ha, ta, sc, (char *)ws + kWsHeader + part, h->sm_count, stream, &launched,
                             &h->tmaps);
    } else {
        e = launch_head_gemv(ha, ta, sc, h->sm_count, stream, &launched);
    }
    h->launch_count += (unsigned)launched;
    if (e != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    return RSTITCH_OK;
}

}  // namespace

extern "C" {

const char *rstitch_status_string(int status)
{
    switch (status) {
        case RSTITCH_OK:                    return "ok";
        case RSTITCH_ERR_INVALID_ARG:       return "invalid argument";
        case RSTITCH_ERR_BAD_ALIGN:         return "misaligned pointer";
        case RSTITCH_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case RSTITCH_ERR_CUDA:              return "CUDA call failed";
        case RSTITCH_ERR_WORKSPACE:         return "workspace too small or misaligned";
        case RSTITCH_ERR_TIMEOUT:           return "device-side wait timed out";
        default:                            return "unknown status";
    }
}

const char *rstitch_path_name(int R, int d, int V, uint32_t flags)
{
    return use_umma(R, d, V, flags) ? "umma" : "gemv";
}

size_t rstitch_workspace_bytes(int R, int d, int V)
{
    if (shape_status(R, d, V) != RSTITCH_OK) return 0;
    return ws_bytes_for(R, d, V);
}

int rstitch_create(rstitch_handle_t *out, int maxR, int max_d, int maxV)
{
    if (!out) return RSTITCH_ERR_INVALID_ARG;
    *out = nullptr;
    int st = shape_status(maxR, max_d, maxV);
    if (st != RSTITCH_OK) return st;
    rstitch_handle_s *h = new (std::nothrow) rstitch_handle_s();
    if (!h) return RSTITCH_ERR_CUDA;
    bool ok = cudaGetDevice(&h->device) == cudaSuccess &&
              cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) == cudaSuccess &&
              cudaMalloc((void **)&h->stat, sizeof(DevStat)) == cudaSuccess &&
              cudaMemset(h->stat, 0, sizeof(DevStat)) == cudaSuccess;
    if (ok) ok = grow_handle(h, maxR, max_d, maxV) == RSTITCH_OK;
    if (!ok) { cudaGetLastError(); rstitch_destroy(h); return RSTITCH_ERR_CUDA; }
    *out = h;
    return RSTITCH_OK;
}

int rstitch_destroy(rstitch_handle_t h)
{
    if (!h) return RSTITCH_OK;
    cudaFree(h->ws); cudaFree(h->stat); cudaFree(h->tile_counts); cudaFree(h->st);
    cudaFreeHost(h->st_host); cudaFreeHost(h->st_in);
    cudaGetLastError();
    delete h;
    return RSTITCH_OK;
}

int rstitch_route_ex(rstitch_handle_t h, const rstitch_args_t *a, void *cuda_stream)
{
    int st = validate(h, a);
    if (st != RSTITCH_OK) return st;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    h->last_stream = stream;
    return enqueue_head(h, a, stream, nullptr, 0);
}

int rstitch_shard_stats(rstitch_handle_t h, const rstitch_args_t *a, int32_t v_base, void *shard_stats,
                        void *cuda_stream)
{
    int st = validate(h, a, kShardStats);
    if (st != RSTITCH_OK) return st;
    if (v_base < 0 || (a->R > 0 && !shard_stats)) return RSTITCH_ERR_INVALID_ARG;
    if (!aligned(shard_stats, 4)) return RSTITCH_ERR_BAD_ALIGN;
    if (a->R == 0) return RSTITCH_OK;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    h->last_stream = stream;
    return enqueue_head(h, a, stream, (float *)shard_stats, v_base);
}

int rstitch_shard_route(rstitch_handle_t h, const rstitch_args_t *a, const void *gathered, int32_t n_shards,
                        void *cuda_stream)
{
    int st = validate(h, a, kShardRoute);
    if (st != RSTITCH_OK) return st;
    if (n_shards < 1 || n_shards > RSTITCH_MAX_SHARDS || (a->R > 0 && !gathered)) return RSTITCH_ERR_INVALID_ARG;
    if (!aligned(gathered, 4)) return RSTITCH_ERR_BAD_ALIGN;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    h->last_stream = stream;
    Alg1Tail alg1;
    if (!make_alg1_tail(a->alg1_tail, &alg1)) return RSTITCH_ERR_INVALID_ARG;
    if (a->R == 0 || a->B == 0) {
        if (cudaMemsetAsync(a->llm_count, 0, sizeof(int32_t), stream) != cudaSuccess) return RSTITCH_ERR_CUDA;
        if (a->seq_len && a->llm_row_off &&
            cudaMemsetAsync(a->llm_row_off, 0, sizeof(int32_t), stream) != cudaSuccess) return RSTITCH_ERR_CUDA;
        if (a->R == 0) {
            if (alg1.on) {
                if (launch_alg1_tail(alg1, a->tok_out, a->route_mask, stream) != cudaSuccess) {
                    cudaGetLastError();
                    return RSTITCH_ERR_CUDA;
                }
                h->launch_count += 1;
            }
            return RSTITCH_OK;
        }
    }
    TailArgs ta;
    ta.R = a->R; ta.B = a->B; ta.V = a->V;
    ta.tau = (a->flags & RSTITCH_TAU_NORMALIZED) ? a->tau * logf((float)a->V) : a->tau;
    ta.row_seq = a->row_seq; ta.seq_len = a->seq_len; ta.kv_len = a->kv_len;
    ta.tok_out = a->tok_out; ta.ent_out = a->ent_out; ta.route_mask = a->route_mask;
    ta.llm_idx = a->llm_idx; ta.llm_count = a->llm_count;
    ta.llm_span = a->llm_span; ta.llm_row_off = a->llm_row_off;
    ta.stat = h->stat;
    ta.shard_stats = nullptr; ta.v_base = 0;
    ta.alg1 = alg1;
    ta.mirror_src = nullptr; ta.mirror_dst = nullptr; ta.mirror_vec = 0;
    Scratch sc = scratch_carve(h->ws);
    int launched = 0;
    cudaError_t e = launch_shard_merge((const float *)gathered, n_shards, a->n_rows_dev, ta, sc.ticket, stream,
                                       &launched);
    h->launch_count += (unsigned)launched;
    if (e != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    return RSTITCH_OK;
}

int rstitch_route(const void *hidden, const void *W_head, int B, int d, int V, float tau,
                  int32_t *tok_out, float *ent_out, uint8_t *route_mask, int32_t *llm_idx,
                  int32_t *llm_count)
{
    int st = shape_status(B, d, V);
    if (st != RSTITCH_OK) return st;
    rstitch_handle_s *h = nullptr;
    st = default_handle(&h, B, d, V);
    if (st != RSTITCH_OK) return st;
    rstitch_args_t a;
    std::memset(&a, 0, sizeof a);
    a.hidden = hidden; a.W_head = W_head; a.R = B; a.B = B; a.d = d; a.V = V; a.n_src = B; a.tau = tau;
    a.tok_out = tok_out; a.ent_out = ent_out; a.route_mask = route_mask; a.llm_idx = llm_idx;
    a.llm_count = llm_count;
    return rstitch_route_ex(h, &a, nullptr);
}

int rstitch_route_ex_host(rstitch_handle_t h, const rstitch_args_t *a, void *cuda_stream)
{
    if (!h || !a) return RSTITCH_ERR_INVALID_ARG;
    if (a->n_rows_dev || a->workspace) return RSTITCH_ERR_INVALID_ARG;     // host-driven: no device-side inputs
    int st = shape_status(a->R, a->d, a->V);
    if (st != RSTITCH_OK) return st;
    if (a->B < 0 || a->n_src < 0 || !a->llm_count) return RSTITCH_ERR_INVALID_ARG;
    if (a->R > 0 && (!a->hidden || !a->W_head || !a->tok_out || !a->ent_out)) return RSTITCH_ERR_INVALID_ARG;
    if (a->B > 0 && (!a->route_mask || !a->llm_idx)) return RSTITCH_ERR_INVALID_ARG;
    if ((a->seq_len == nullptr) != (a->kv_len == nullptr)) return RSTITCH_ERR_INVALID_ARG;
    if (a->seq_len && a->B > 0 && (!a->llm_span || !a->llm_row_off)) return RSTITCH_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const size_t R = (size_t)a->R, B = (size_t)a->B;
    const size_t n_src = a->n_src > 0 ? (size_t)a->n_src : R;
    if (R == 0 || B == 0) {
        *a->llm_count = 0;
        if (a->seq_len && a->llm_row_off) a->llm_row_off[0] = 0;
        if (R == 0) return RSTITCH_OK;
    }

    // one staging block: inputs first, then the outputs; every piece 256-byte aligned
    auto up = [](size_t n) { return (n + 255) / 256 * 256; };
    size_t off = 0;
    const size_t o_hid = off;  off += up(n_src * a->d * 2);
    const size_t o_ridx = off; off += up(R * 4);
    const size_t o_rseq = off; off += up(R * 4);
    const size_t o_slen = off; off += up(B * 4);
    const size_t o_klen = off; off += up(B * 4);
    const size_t o_tok = off;  off += up(R * 4);
    const size_t o_ent = off;  off += up(R * 4);
    const size_t o_idx = off;  off += up(B * 4);
    const size_t o_span = off; off += up(B * 4);
    const size_t o_roff = off; off += up((B + 1) * 4);
    const size_t o_cnt = off;  off += 256;
    const size_t o_msk = off;  off += up(B);
    if (off > h->st_bytes) {
        if (h->st) { cudaDeviceSynchronize(); cudaFree(h->st); h->st = nullptr; h->st_bytes = 0; }
        if (cudaMalloc(&h->st, off) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
        h->st_bytes = off;
    }
    char *base = (char *)h->st;
    bool ok = true;
    const size_t in_bytes = o_tok;                  // the inputs lead the staging block
    if (in_bytes <= kPackedInputMax) {
        // a decode step's inputs are a few KB: gather them in a pinned mirror of the block's input part
        // and send them with one copy (each small copy costs microseconds of its own)
        if (in_bytes > h->st_in_bytes) {
            if (h->st_in) { cudaFreeHost(h->st_in); h->st_in = nullptr; h->st_in_bytes = 0; }
            if (cudaMallocHost(&h->st_in, kPackedInputMax) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
            h->st_in_bytes = kPackedInputMax;
        }
        char *in = (char *)h->st_in;
        std::memcpy(in + o_hid, a->hidden, n_src * a->d * 2);
        if (a->row_idx) std::memcpy(in + o_ridx, a->row_idx, R * 4);
        if (a->row_seq) std::memcpy(in + o_rseq, a->row_seq, R * 4);
        if (a->seq_len) { std::memcpy(in + o_slen, a->seq_len, B * 4); std::memcpy(in + o_klen, a->kv_len, B * 4); }
        ok = cudaMemcpyAsync(base, in, in_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    } else {
        auto h2d = [&](size_t o, const void *src, size_t n) {
            return n == 0 || cudaMemcpyAsync(base + o, src, n, cudaMemcpyHostToDevice, stream) == cudaSuccess;
        };
        ok = h2d(o_hid, a->hidden, n_src * a->d * 2);
        const size_t idx_bytes = o_tok - o_ridx;        // the index arrays follow the hidden rows
        const bool any_idx = a->row_idx || a->row_seq || a->seq_len;
        if (ok && any_idx && idx_bytes <= kPackedInputMax) {
            // a large batch of rows: they go as they are, the small index arrays still as one copy
            if (h->st_in_bytes < kPackedInputMax) {
                if (h->st_in) { cudaFreeHost(h->st_in); h->st_in = nullptr; h->st_in_bytes = 0; }
                if (cudaMallocHost(&h->st_in, kPackedInputMax) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
                h->st_in_bytes = kPackedInputMax;
            }
            char *in = (char *)h->st_in - o_ridx;
            if (a->row_idx) std::memcpy(in + o_ridx, a->row_idx, R * 4);
            if (a->row_seq) std::memcpy(in + o_rseq, a->row_seq, R * 4);
            if (a->seq_len) { std::memcpy(in + o_slen, a->seq_len, B * 4); std::memcpy(in + o_klen, a->kv_len, B * 4); }
            ok = cudaMemcpyAsync(base + o_ridx, h->st_in, idx_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
        } else {
            if (ok && a->row_idx) ok = h2d(o_ridx, a->row_idx, R * 4);
            if (ok && a->row_seq) ok = h2d(o_rseq, a->row_seq, R * 4);
            if (ok && a->seq_len) ok = h2d(o_slen, a->seq_len, B * 4) && h2d(o_klen, a->kv_len, B * 4);
        }
    }
    if (!ok) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }

    rstitch_args_t dv = *a;
    dv.hidden = base + o_hid;
    dv.n_src = (int32_t)n_src;
    dv.row_idx = a->row_idx ? (const int32_t *)(base + o_ridx) : nullptr;
    dv.row_seq = a->row_seq ? (const int32_t *)(base + o_rseq) : nullptr;
    dv.seq_len = a->seq_len ? (const int32_t *)(base + o_slen) : nullptr;
    dv.kv_len  = a->seq_len ? (const int32_t *)(base + o_klen) : nullptr;
    dv.tok_out = (int32_t *)(base + o_tok);
    dv.ent_out = (float *)(base + o_ent);
    dv.llm_idx = (int32_t *)(base + o_idx);
    dv.llm_span = a->seq_len ? (int32_t *)(base + o_span) : nullptr;
    dv.llm_row_off = a->seq_len ? (int32_t *)(base + o_roff) : nullptr;
    dv.llm_count = (int32_t *)(base + o_cnt);
    dv.route_mask = (uint8_t *)(base + o_msk);
    // The outputs are contiguous in the staging block and go to a pinned mirror in one piece, then with
    // plain host copies into the caller's buffers (a handful of small device-to-host copies costs more).
    // A few KB are written there by the deciding block itself (the mirror is mapped into the device's
    // address space), which saves the copy command and its latency; more goes through a copy.
    const size_t out_bytes = off - o_tok;
    if (out_bytes > h->st_host_bytes) {
        if (h->st_host) { cudaFreeHost(h->st_host); h->st_host = nullptr; h->st_host_bytes = 0; }
        if (cudaMallocHost(&h->st_host, out_bytes) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
        h->st_host_bytes = out_bytes;
    }
    Mirror mirror;
    void *mirror_dev = nullptr;
    if (out_bytes <= kMirrorMax && dv.alg1_tail == nullptr &&
        cudaHostGetDevicePointer(&mirror_dev, h->st_host, 0) == cudaSuccess && mirror_dev) {
        mirror.src = base + o_tok; mirror.dst = mirror_dev; mirror.bytes = out_bytes;
    } else {
        cudaGetLastError();
    }
    st = validate(h, &dv);
    if (st != RSTITCH_OK) return st;
    h->last_stream = stream;
    st = enqueue_head(h, &dv, stream, nullptr, 0, mirror);
    if (st != RSTITCH_OK) return st;
    ok = (mirror.dst != nullptr ||
          cudaMemcpyAsync(h->st_host, base + o_tok, out_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess) &&
         cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    const char *hb = (const char *)h->st_host - o_tok;
    std::memcpy(a->tok_out, hb + o_tok, R * 4);
    std::memcpy(a->ent_out, hb + o_ent, R * 4);
    std::memcpy(a->llm_idx, hb + o_idx, B * 4);
    std::memcpy(a->llm_count, hb + o_cnt, 4);
    std::memcpy(a->route_mask, hb + o_msk, B);
    if (a->seq_len) {
        std::memcpy(a->llm_span, hb + o_span, B * 4);
        std::memcpy(a->llm_row_off, hb + o_roff, (B + 1) * 4);
    }
    return RSTITCH_OK;
}

int rstitch_route_host(rstitch_handle_t h, const void *hidden_host, const void *W_head_dev,
                       int B, int d, int V, float tau, int32_t *tok_host, float *ent_host,
                       uint8_t *mask_host, int32_t *llm_idx_host, int32_t *llm_count_host,
                       void *cuda_stream)
{
    if (B < 0) return RSTITCH_ERR_INVALID_ARG;
    rstitch_args_t a;
    std::memset(&a, 0, sizeof a);
    a.hidden = hidden_host; a.W_head = W_head_dev; a.R = B; a.B = B; a.d = d; a.V = V; a.n_src = B; a.tau = tau;
    a.tok_out = tok_host; a.ent_out = ent_host; a.route_mask = mask_host; a.llm_idx = llm_idx_host;
    a.llm_count = llm_count_host;
    return rstitch_route_ex_host(h, &a, cuda_stream);
}

int rstitch_compact(const uint8_t *mask, int B, int32_t *idx, int32_t *count, void *cuda_stream)
{
    if (B < 0 || !count || (B > 0 && (!mask || !idx))) return RSTITCH_ERR_INVALID_ARG;
    if (!aligned(idx, 4) || !aligned(count, 4)) return RSTITCH_ERR_BAD_ALIGN;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (B == 0) {
        if (cudaMemsetAsync(count, 0, sizeof(int32_t), stream) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
        return RSTITCH_OK;
    }
    rstitch_handle_s *h = nullptr;
    int st = default_handle(&h, 1, 8, 2);
    if (st != RSTITCH_OK) return st;
    int32_t *tiles = nullptr;
    if (B > kCompactOneBlockMax) {
        int n_tiles = (B + kCompactTile - 1) / kCompactTile;
        std::lock_guard<std::mutex> lock(g_default_mutex);
        if (n_tiles > h->tile_cap) {
            if (h->tile_counts) { cudaDeviceSynchronize(); cudaFree(h->tile_counts); h->tile_counts = nullptr; h->tile_cap = 0; }
            if (cudaMalloc((void **)&h->tile_counts, (size_t)n_tiles * 4) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
            h->tile_cap = n_tiles;
        }
        tiles = h->tile_counts;
    }
    h->last_stream = stream;
    int launched = 0;
    cudaError_t e = launch_compact(mask, B, idx, count, h->stat, tiles, stream, &launched);
    h->launch_count += (unsigned)launched;
    if (e != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    return RSTITCH_OK;
}

int rstitch_selftest_wait(rstitch_handle_t h, void *cuda_stream)
{
    if (!h) return RSTITCH_ERR_INVALID_ARG;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    h->last_stream = stream;
    // ~1 ms at the top SM clock: long enough to be a real wait, far below anything a watchdog minds
    if (launch_wait_selftest(h->stat, 2000000ll, stream) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    h->launch_count += 1;
    return RSTITCH_OK;
}

int rstitch_last_status(rstitch_handle_t h, rstitch_devstat_t *out)
{
    if (!out) return RSTITCH_ERR_INVALID_ARG;
    if (!h) {
        // the per-device handle behind rstitch_route / rstitch_compact
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
        std::lock_guard<std::mutex> lock(g_default_mutex);
        h = g_default[dev];
        if (!h) { std::memset(out, 0, sizeof *out); return RSTITCH_OK; }
    }
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    if (cudaMemcpy(out, h->stat, sizeof(DevStat), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(h->stat, 0, sizeof(DevStat)) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    out->launches = h->launch_count;     // counted on the host as the kernels are enqueued
    h->launch_count = 0;
    return out->timeouts ? RSTITCH_ERR_TIMEOUT : RSTITCH_OK;
}

}  // extern "C"
