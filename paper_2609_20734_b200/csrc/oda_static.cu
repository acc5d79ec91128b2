// oda_local_decode_static: the Local pass of one attention layer for callers that cannot
// allocate device memory.  Its scratch (split partials, merge tickets, layer table, status
// word) lives in a file-scope __device__ array instead of a caller-provided workspace.
#include <cmath>
#include <cstring>
#include <mutex>

#include "../../include/oda.h"
#include "oda_device.cuh"
#include "oda_launch.h"

using namespace oda;

namespace {

constexpr int kStaticMaxBatch = 16;
constexpr int kStaticMaxUnits = 256;   // batch * kv heads
constexpr int kStaticMaxGrid = 148;
constexpr int kStaticMaxItems = kStaticMaxGrid + kStaticMaxUnits;  // one partial slot per (span, unit) pair
constexpr size_t kOffStatus = 0;                              // int32
constexpr size_t kOffLayer = 256;                             // one LayerInfo
constexpr size_t kOffTickets = 512;                           // kStaticMaxUnits int32
constexpr size_t kOffPartials = kOffTickets + kStaticMaxUnits * 4;
constexpr size_t kStaticBytes = kOffPartials + (size_t)kStaticMaxItems * 8 * (128 + kPartHdr) * 4;  // ~2.2 MiB

// Every GPU that loads the library holds one copy of this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// Host code may not use g_static_scratch as an address (on the host the name is only a
// stand-in for the symbol): the device address is looked up once per device.
// The set-up is published under a mutex, so that two host threads making their first call on a
// device at the same time agree on it.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_scratch_ptr[kMaxDevices];
int g_sms[kMaxDevices];
int g_occ[kMaxDevices][2][4];   // resident CTAs per SM by (head_dim 64|128, group 1|2|4|8); 0 = not asked yet

// Device address of the array on the current device (nullptr on failure) and the device's index.
unsigned char* static_scratch(int* dev_out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {  // first call on this device: set-up, with the device current
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return nullptr;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return nullptr;
        // (the array is zero when the module is loaded, which is where the sticky status word starts)
        g_sms[dev] = sms;
        g_scratch_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    *dev_out = dev;
    return g_scratch_ptr[dev];
}

// The launch grid follows from the shape of THIS call (never from an earlier call's).
int static_grid(int dev, int head_dim, int group)
{
    const int di = head_dim == 128 ? 1 : 0, gi = group == 1 ? 0 : group == 2 ? 1 : group == 4 ? 2 : 3;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_occ[dev][di][gi]) {
        const int occ = occupancy_splitkv_simt(head_dim, group);
        g_occ[dev][di][gi] = occ > 0 ? occ : 1;
    }
    const int grid = g_sms[dev] * g_occ[dev][di][gi];
    return grid < kStaticMaxGrid ? grid : kStaticMaxGrid;
}

__global__ void static_scratch_prepare_kernel(unsigned char* scratch, int window, int sinks, int units)
{
    // the array keeps whatever the previous call left: reset what has to start at zero (the status
    // word is not among that: it collects bits until oda_local_decode_static_status reads it)
    int32_t* tickets = reinterpret_cast<int32_t*>(scratch + kOffTickets);
    for (int i = threadIdx.x; i < units; i += blockDim.x) tickets[i] = 0;
    if (threadIdx.x == 0) {
        LayerInfo li;
        li.window = window; li.sinks = sinks; li.gated = 1; li.kv_index = 0; li.cls = 0;
        li.pad0 = li.pad1 = li.pad2 = 0;
        *reinterpret_cast<LayerInfo*>(scratch + kOffLayer) = li;
    }
}

}  // namespace

extern "C" oda_status_t oda_local_decode_static(int32_t batch, int32_t num_q_heads, int32_t num_kv_heads,
                                                int32_t head_dim, int32_t window, int32_t sinks, float sm_scale,
                                                int64_t kv_block_stride, int64_t kv_token_stride,
                                                int64_t kv_head_stride, int32_t max_blocks_per_seq, const void* q,
                                                const void* k_cache, const void* v_cache,
                                                const int32_t* block_table, const int32_t* seq_lens, float* out,
                                                float* lse, void* stream)
{
    if (batch < 0 || num_kv_heads < 1 || num_q_heads < 1 || num_q_heads % num_kv_heads) return ODA_ERR_INVALID_ARG;
    if (window < 1 || sinks < 0 || max_blocks_per_seq < 1 || !(sm_scale >= 0.f) || !std::isfinite(sm_scale))
        return ODA_ERR_INVALID_ARG;
    const int group = num_q_heads / num_kv_heads;
    if ((head_dim != 64 && head_dim != 128) || (group != 1 && group != 2 && group != 4 && group != 8))
        return ODA_ERR_UNSUPPORTED;
    // sizes beyond what the fixed scratch was laid out for are refused, never truncated
    if (batch > kStaticMaxBatch || (int64_t)batch * num_kv_heads > kStaticMaxUnits) return ODA_ERR_UNSUPPORTED;
    if (batch == 0) return ODA_OK;
    if (!q || !k_cache || !v_cache || !block_table || !seq_lens || !out) return ODA_ERR_INVALID_ARG;
    const int64_t strides[3] = {kv_block_stride, kv_token_stride, kv_head_stride};
    for (int64_t s : strides)
        if (s < head_dim || (s % 8) != 0) return ODA_ERR_INVALID_ARG;
    if (kv_block_stride < (int64_t)head_dim * kPage) return ODA_ERR_INVALID_ARG;  // a block holds 16 rows of head_dim
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache) |
         reinterpret_cast<uintptr_t>(out)) & 15)
        return ODA_ERR_INVALID_ARG;

    int dev = -1;
    unsigned char* scratch = static_scratch(&dev);
    if (!scratch) return ODA_ERR_CUDA;
    const int grid = static_grid(dev, head_dim, group);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    static_scratch_prepare_kernel<<<1, 256, 0, st>>>(scratch, window, sinks, batch * num_kv_heads);
    if (cudaGetLastError() != cudaSuccess) return ODA_ERR_CUDA;

    AttnParams p;
    std::memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k_cache);
    p.v = static_cast<const __nv_bfloat16*>(v_cache);
    p.block_table = block_table;
    p.seq_lens = seq_lens;
    p.out = out;
    p.lse = lse;
    p.partials = reinterpret_cast<float*>(scratch + kOffPartials);
    p.tickets = reinterpret_cast<int32_t*>(scratch + kOffTickets);
    p.status = reinterpret_cast<int32_t*>(scratch + kOffStatus);
    p.layers = reinterpret_cast<const LayerInfo*>(scratch + kOffLayer);
    p.kv_block_stride = kv_block_stride;
    p.kv_token_stride = kv_token_stride;
    p.kv_head_stride = kv_head_stride;
    p.layer_begin = 0;
    p.layer_end = 1;
    p.batch = batch;
    p.max_batch = batch;
    p.num_q_heads = num_q_heads;
    p.num_kv_heads = num_kv_heads;
    p.max_blocks_per_seq = max_blocks_per_seq;
    p.ncls = 1;
    p.min_span_pages = 8;
    p.snap_span_pages = 0;
    p.direct_hint = 0;
    p.l2_keep_layer_end = 0;
    p.max_items = kStaticMaxItems;
    p.scale_log2e = (sm_scale > 0.f ? sm_scale : 1.0f / sqrtf((float)head_dim)) * 1.4426950408889634f;
    p.cls_window[0] = window;
    p.cls_sinks[0] = sinks;
    p.cls_gated[0] = 1;
    p.cls_layers_in_call[0] = 1;
    if (launch_splitkv_simt(p, head_dim, group, grid, st) != cudaSuccess) return ODA_ERR_CUDA;
    return ODA_OK;
}

extern "C" oda_status_t oda_local_decode_static_status(void* stream, int32_t* code)
{
    if (!code) return ODA_ERR_INVALID_ARG;
    int dev = -1;
    unsigned char* scratch = static_scratch(&dev);
    if (!scratch) return ODA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t v = 0;  // pageable destination: the copy returns once the value is here; the clear follows in stream order
    cudaError_t e = cudaMemcpyAsync(&v, scratch + kOffStatus, sizeof v, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(scratch + kOffStatus, 0, sizeof v, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return ODA_ERR_CUDA;
    *code = v;
    return v ? ODA_ERR_DEVICE_STATUS : ODA_OK;
}
