// rstitch_route_static: the routing decision for callers that must not allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving engine that has
// handed all device memory to its own pool, in a latency-critical decode loop where an allocation
// would synchronise the device, or in a process whose memory budget is fixed at start-up.  For
// them the scratch of the head kernels (the ticket counter, the per-slice partial statistics and
// the status word) lives in a fixed array inside the library image instead of in a handle.  Every GPU that loads the library holds that array until the process exits.
#include "../../include/rstitch.h"
#include "rstitch_kernels.cuh"

#include <cmath>
#include <mutex>

using namespace rstitch;

namespace {

constexpr int    kStaticMaxRows = RSTITCH_STATIC_MAX_ROWS;
constexpr size_t kStatOffset    = 128;      // status word inside the 256-byte header, after the ticket
constexpr size_t kStaticBytes   = kWsHeader + 5 * ((size_t)kStaticMaxRows * kMaxSlices * 4);

// The scratch itself.  In host code this name is only a stand-in for the symbol, never a device
// address: the address is fetched once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

std::mutex g_static_mutex;
void      *g_static_ptr[64] = {};
int        g_static_sms[64] = {};

// First call on a device: resolve the array's device address and the SM count.  Allocates nothing.
int static_setup(int dev, void **ptr, int *sms)
{
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        int n = 0;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            return RSTITCH_ERR_CUDA;
        }
        g_static_ptr[dev] = p;
        g_static_sms[dev] = n;
    }
    *ptr = g_static_ptr[dev];
    *sms = g_static_sms[dev];
    return RSTITCH_OK;
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" int rstitch_route_static(const void *hidden, const void *W_head, int B, int d, int V,
                                    float tau, int32_t *tok_out, float *ent_out, uint8_t *route_mask,
                                    int32_t *llm_idx, int32_t *llm_count, void *cuda_stream)
{
    if (B < 0 || !llm_count || !std::isfinite(tau)) return RSTITCH_ERR_INVALID_ARG;
    if (B > kStaticMaxRows) return RSTITCH_ERR_UNSUPPORTED_SHAPE;      // beyond the fixed scratch
    if (d < 8 || (d % 8) != 0 || d > 16384 || V < 2) return RSTITCH_ERR_UNSUPPORTED_SHAPE;
    if (B > 0 && (!hidden || !W_head || !tok_out || !ent_out || !route_mask || !llm_idx))
        return RSTITCH_ERR_INVALID_ARG;
    if (!aligned(hidden, 16) || !aligned(W_head, 16)) return RSTITCH_ERR_BAD_ALIGN;
    if (!aligned(tok_out, 4) || !aligned(ent_out, 4) || !aligned(llm_idx, 4) || !aligned(llm_count, 4))
        return RSTITCH_ERR_BAD_ALIGN;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    void *base = nullptr;
    int sms = 0;
    int st = static_setup(dev, &base, &sms);
    if (st != RSTITCH_OK) return st;

    // The array keeps whatever the previous call left: the ticket and the status word must start
    // at zero, the partials are fully rewritten before they are read.
    if (cudaMemsetAsync(base, 0, kWsHeader, stream) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    if (B == 0) {
        if (cudaMemsetAsync(llm_count, 0, sizeof(int32_t), stream) != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
        return RSTITCH_OK;
    }

    HeadArgs ha;
    ha.hidden = hidden; ha.W = W_head; ha.R = B; ha.d = d; ha.V = V; ha.n_src = B;
    ha.row_idx = nullptr; ha.n_rows_dev = nullptr;
    ha.sample = SampleArgs{};                                   // greedy token
    TailArgs ta;
    ta.R = B; ta.B = B; ta.V = V; ta.tau = tau;
    ta.row_seq = nullptr; ta.seq_len = nullptr; ta.kv_len = nullptr;
    ta.tok_out = tok_out; ta.ent_out = ent_out; ta.route_mask = route_mask;
    ta.llm_idx = llm_idx; ta.llm_count = llm_count; ta.llm_span = nullptr; ta.llm_row_off = nullptr;
    ta.stat = (DevStat *)((char *)base + kStatOffset);
    ta.shard_stats = nullptr; ta.v_base = 0;
    ta.alg1.on = 0;
    ta.mirror_src = nullptr; ta.mirror_dst = nullptr; ta.mirror_vec = 0;
    Scratch sc = scratch_carve(base);
    // Same choice of kernel as the regular entry points: one row streams on the CUDA cores, more rows go
    // to the tensor-core kernel (its tensor maps are encoded on the host and travel as kernel
    // parameters, its accumulators live in tensor memory: no device allocation either; at most
    // kStaticMaxRows x #blocks partials, well inside the array).
    cudaError_t e;
    if (B > 1 && umma_shape_ok(B, d, V)) {
        int launched = 0;
        e = launch_head_umma(ha, ta, sc, nullptr, sms, stream, &launched);
    } else {
        e = launch_head_gemv(ha, ta, sc, sms, stream);
    }
    if (e != cudaSuccess) { cudaGetLastError(); return RSTITCH_ERR_CUDA; }
    return RSTITCH_OK;
}
