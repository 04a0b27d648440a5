// san_attn_weights_static: the weights step (Eq. 1) for callers that have no device
// memory to give the library beyond their own inputs and outputs.
//
// Who this is for.  A decode loop embedded in a serving process often cannot allocate:
// the server's cache manager has reserved all of HBM up front, so cudaMalloc fails; the
// loop runs as a plug-in whose contract forbids allocation once serving has started; or
// the loop is latency-critical and cudaMalloc/cudaFree would stall every stream of the
// device while they run.  Such a caller cannot build a san_ctx (it needs a workspace
// buffer).  This entry point needs no context and no workspace: the little scratch that
// split rows use (one ticket per row, a max and a sum per span) lives in a fixed array
// that is part of the library image on every GPU that loads it.
//
// The kernel is the same weights_kernel the context path launches; only where its
// scratch pointers point differs.
#include <cmath>
#include <mutex>

#include "san_kernels.cuh"

using namespace san;

namespace {

// Fixed scratch, 1 MiB per GPU for as long as the library stays loaded:
//   [0, 256)              error words (used when the caller passes no status buffer)
//   [256, 256 + 256 KiB)  one int ticket per (item, head) row      -> at most 65536 rows
//   [.., 1 MiB)           (max, sum) per (row, query, span) of split rows
constexpr size_t kStaticBytes = (size_t)1 << 20;
constexpr int kStaticMaxRows = 65536;
constexpr size_t kTicketsOffset = 256;
constexpr size_t kPartOffset = kTicketsOffset + (size_t)kStaticMaxRows * sizeof(int);
constexpr size_t kPartFloats = (kStaticBytes - kPartOffset) / sizeof(float);

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not an address a
// kernel may use; the device address is looked up once per device and kept here.
struct DeviceSlot { char* scratch; int sm_count; bool ready; };
DeviceSlot g_slots[64];
std::mutex g_slots_mutex;

int32_t slot_for_current_device(DeviceSlot* out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SAN_ERR_CUDA;
    if (dev < 0 || dev >= 64) return SAN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_slots_mutex);
    DeviceSlot& s = g_slots[dev];
    if (!s.ready) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return SAN_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SAN_ERR_CUDA;
        s.scratch = static_cast<char*>(p);
        s.sm_count = sms;
        s.ready = true;
    }
    *out = s;
    return SAN_OK;
}

template <typename T>
cudaError_t launch(const WeightsParams& p, int nq, unsigned grid, cudaStream_t st) {
    const unsigned block = kWarpsPerCta * 32;
    if (nq <= 1) weights_kernel<T, 1><<<grid, block, 0, st>>>(p);
    else if (nq <= 2) weights_kernel<T, 2><<<grid, block, 0, st>>>(p);
    else if (nq <= 4) weights_kernel<T, 4><<<grid, block, 0, st>>>(p);
    else weights_kernel<T, 8><<<grid, block, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

extern "C" int32_t san_attn_weights_static(int32_t dtype, int32_t n_heads, int32_t n_queries,
                                           const void* d_q, const void* d_K, int32_t max_ids,
                                           int32_t cap_len, const int32_t* d_ids, const int32_t* d_lens,
                                           int32_t n_items, int32_t max_len, float* d_S, int64_t ld_s,
                                           int32_t* d_status, void* stream) {
    if (!d_q || !d_K || !d_ids || !d_lens || !d_S) return SAN_ERR_NULL;
    if (dtype != SAN_F32 && dtype != SAN_BF16) return SAN_ERR_DTYPE;
    if (n_heads < 1 || n_heads > 1024 || n_queries < 1 || n_queries > 8) return SAN_ERR_SHAPE;
    if (max_ids < 1 || cap_len < 1 || cap_len > (1 << 20)) return SAN_ERR_SHAPE;
    if (n_items < 0 || n_items > max_ids) return SAN_ERR_SHAPE;
    if (max_len == 0) max_len = cap_len;
    if (max_len < 1 || max_len > cap_len || ld_s < max_len) return SAN_ERR_SHAPE;
    const long long rows = (long long)n_items * n_heads;
    if (rows > kStaticMaxRows) return SAN_ERR_CAPACITY;   // beyond the fixed scratch: use a context
    if (n_items == 0) return SAN_OK;

    DeviceSlot slot;
    int32_t rc = slot_for_current_device(&slot);
    if (rc != SAN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    WeightsParams p;
    p.q = d_q; p.K = d_K; p.ids = d_ids; p.lens = d_lens; p.S = d_S; p.ld_s = ld_s;
    p.n_items = n_items; p.H = n_heads; p.nq = n_queries; p.nq_total = n_queries; p.q0 = 0;
    p.cap_len = cap_len; p.max_ids = max_ids; p.max_len = max_len;
    // spans: halve while SMs would idle, never more than the fixed scratch can hold
    const long long target = (long long)slot.sm_count * 16;
    int sl = (max_len + 31) / 32 * 32, ns = 1;
    while (rows * ns < target && sl > 32) {
        const int half = ((sl + 1) / 2 + 31) / 32 * 32;
        const int ns2 = (max_len + half - 1) / half;
        if (rows * n_queries * 2 * ns2 > (long long)kPartFloats) break;
        sl = half; ns = ns2;
    }
    p.span_len = sl; p.n_spans_max = ns;
    p.part = reinterpret_cast<float*>(slot.scratch + kPartOffset);
    p.tickets = reinterpret_cast<int*>(slot.scratch + kTicketsOffset);
    p.err = d_status ? d_status : reinterpret_cast<int*>(slot.scratch);
    p.scale_log2e = (float)(1.4426950408889634 / std::sqrt((double)kDh));

    // the array keeps whatever the previous call left: tickets must start at zero, and the
    // status words must not carry an old error
    cudaError_t e = cudaMemsetAsync(p.tickets, 0, (size_t)rows * sizeof(int), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.err, 0, 8 * sizeof(int), st);
    if (e != cudaSuccess) return SAN_ERR_CUDA;
    const long long warps = rows * ns;
    const unsigned grid = (unsigned)((warps + kWarpsPerCta - 1) / kWarpsPerCta);
    e = dtype == SAN_BF16 ? launch<__nv_bfloat16>(p, n_queries, grid, st) : launch<float>(p, n_queries, grid, st);
    return e == cudaSuccess ? SAN_OK : SAN_ERR_CUDA;
}
