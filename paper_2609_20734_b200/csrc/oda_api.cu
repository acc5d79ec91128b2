// C-ABI layer of the ODA decode library: argument validation, workspace layout and
// stream-ordered kernel launches.  No device memory is allocated here, and nothing
// synchronises except the two entry points whose contract says so.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/oda.h"
#include "oda_device.cuh"
#include "oda_launch.h"

using namespace oda;

namespace {

constexpr size_t kAlign = 256;
size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct WsLayout {
    size_t status, layers, tickets, head_partial, head_pre, head_rb_tickets, sm_claims, sm_bytes, cum_share, partials;
    size_t st_q_local, st_q_full, st_feat, st_override, st_out, st_lse, st_scores, st_logits, st_flags, own_lse;
    size_t total;
};

}  // namespace

struct oda_ctx {
    oda_config_t cfg;
    std::vector<LayerInfo> layers;
    int ncls = 0;
    int cls_window[kMaxClasses], cls_sinks[kMaxClasses], cls_gated[kMaxClasses];
    int group = 1;
    int last_gated = -1;
    float scale = 0.f;
    int num_sms = 148;
    int variant = ODA_VARIANT_SIMT;
    int grid = 148;
    int min_span_pages = 16;  // four whole tiles; measured against 8 (one-layer launches 14.0 -> 13.4 us) and 12 / 24 (ragged tiles: slower)
    size_t l2_resident_bytes = 0;  // Local working set to keep in L2 between steps (oda_set_cache_resident_bytes)
    int snap_span_pages = 256;  // launches of up to 2 MiB per CTA may be cut at unit boundaries (measured against 128 and 512)
    bool calibrated = false;  // the per-SM split table in the workspace is valid
    bool calibrating = false; // attention launches record per-SM streaming rates
    double calib_spread = 0.0; // slowest / fastest SM share seen by oda_calibrate
    int max_items = 0;
    int head_grid = 1;
    WsLayout lay{};
    char* ws = nullptr;
    // TMA variant: tensor maps of the two caches, re-encoded when a base pointer changes
    alignas(64) unsigned char kmap[128];
    alignas(64) unsigned char vmap[128];
    const void* kmap_base = nullptr;
    const void* vmap_base = nullptr;
    int phys_layers = 1;
    int blocks_per_layer = 0;
    int64_t blocks_bound = 1;
    int64_t launches = 0;
    bool use_pdl = true;  // programmatic dependent launch between the kernels of a step
    bool allow_empty = false;  // gated passes skip requests of length 0 instead of reporting them
    bool reuse_local = false;  // the gated pass reads only S^F \ S^L and merges with the Local result
    std::string err;
};

namespace {

oda_status_t fail(oda_ctx* c, oda_status_t s, const std::string& msg)
{
    if (c) c->err = msg;
    return s;
}

oda_status_t cuda_fail(oda_ctx* c, cudaError_t e, const char* what)
{
    return fail(c, ODA_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

size_t out_elem(const oda_ctx* c) { return c->cfg.out_dtype ? 2 : 4; }

void compute_layout(oda_ctx* c)
{
    const oda_config_t& f = c->cfg;
    const size_t L = f.num_layers, B = f.max_batch, Hq = f.num_q_heads, D = f.head_dim;
    WsLayout& w = c->lay;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    w.status = take(256);
    w.layers = take(L * sizeof(LayerInfo));
    w.tickets = take(L * B * f.num_kv_heads * sizeof(int32_t));
    w.head_partial = take((size_t)c->head_grid * B * sizeof(float));
    w.head_rb_tickets = take((size_t)c->head_grid * sizeof(int32_t));
    {
        const size_t d_in = (size_t)std::max(0, f.head_d_ext) + (f.head_use_attn_out ? Hq * D : 0);
        w.head_pre = take((size_t)recall_head_ksplits((int)d_in) * (size_t)std::max(1, f.head_d_hidden) * B * sizeof(float));
    }
    w.sm_claims = take(1024 * sizeof(int32_t));
    w.sm_bytes = take(2 * 1024 * sizeof(unsigned long long));
    w.cum_share = take((kMaxGrid + 1) * sizeof(uint16_t));
    w.partials = take((size_t)c->max_items * std::max<size_t>(c->group * (D + kPartHdr), tma_partial_slot_floats()) * sizeof(float));
    w.st_q_local = take(L * B * Hq * D * 2);
    w.st_q_full = take(L * B * Hq * D * 2);
    w.st_feat = take(B * (size_t)(f.head_d_ext > 0 ? f.head_d_ext : 1) * 4);
    w.st_override = take(B);
    w.st_out = take(L * B * Hq * D * out_elem(c));
    w.st_lse = take(L * B * Hq * 4);
    w.st_scores = take(B * 4);
    w.st_logits = take(B * 4);
    w.st_flags = take(B);
    w.own_lse = take(L * B * Hq * 4);  // lse of the step when the caller keeps none (remainder mode needs it)
    w.total = off;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

oda_status_t check_attn_args(oda_ctx* c, int lb, int le, int batch, const void* q, const void* k,
                             const void* v, const int32_t* bt, const int32_t* sl, void* out)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    if (lb < 0 || le > c->cfg.num_layers || lb > le) return fail(c, ODA_ERR_INVALID_ARG, "bad layer range");
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0 || lb == le) return ODA_OK;
    if (!q || !k || !v || !bt || !sl || !out) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(c, ODA_ERR_INVALID_ARG, "q, k_cache, v_cache and out must be 16-byte aligned");
    return ODA_OK;
}

oda_status_t launch_attention(oda_ctx* c, int mode, int lb, int le, int batch, const void* q,
                              const void* k, const void* v, const int32_t* bt, const int32_t* sl,
                              const uint8_t* flags, void* out, float* lse, cudaStream_t st,
                              int32_t* advance = nullptr, bool* advanced = nullptr,
                              const oda_step_args_t* publish = nullptr)
{
    const oda_config_t& f = c->cfg;
    AttnParams p;
    std::memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.block_table = bt;
    p.seq_lens = sl;
    p.flags = flags;
    p.out = out;
    p.lse = lse;
    p.partials = reinterpret_cast<float*>(c->ws + c->lay.partials);
    p.tickets = reinterpret_cast<int32_t*>(c->ws + c->lay.tickets);
    p.status = reinterpret_cast<int32_t*>(c->ws + c->lay.status);
    p.layers = reinterpret_cast<const LayerInfo*>(c->ws + c->lay.layers);
    p.kv_layer_stride = f.kv_layer_stride;
    p.kv_block_stride = f.kv_block_stride;
    p.kv_token_stride = f.kv_token_stride;
    p.kv_head_stride = f.kv_head_stride;
    p.layer_begin = lb;
    p.layer_end = le;
    p.batch = batch;
    p.max_batch = f.max_batch;
    p.num_q_heads = f.num_q_heads;
    p.num_kv_heads = f.num_kv_heads;
    p.max_blocks_per_seq = f.max_blocks_per_seq;
    p.out_bf16 = f.out_dtype;
    p.mode = mode;
    p.ncls = c->ncls;
    p.min_span_pages = c->min_span_pages;
    p.snap_span_pages = c->snap_span_pages;
    if (mode == 0 && c->l2_resident_bytes > 0) {
        // leading layers of the call whose Local working set fits the budget: their pages are loaded
        // with an evict-last hint, so the next step finds them in L2
        size_t used = 0;
        int keep = lb;
        for (; keep < le; ++keep) {
            const int cls = c->layers[keep].cls;
            const size_t tokens = (size_t)c->cls_window[cls] + (size_t)c->cls_sinks[cls];
            const size_t bytes = (size_t)batch * f.num_kv_heads * tokens * f.head_dim * 4;  // K and V, bf16
            if (used + bytes > c->l2_resident_bytes) break;
            used += bytes;
        }
        p.l2_keep_layer_end = keep;
    }
    p.max_items = c->max_items;
    p.scale_log2e = c->scale * 1.4426950408889634f;
    bool any = false;
    for (int i = 0; i < c->ncls; ++i) {
        p.cls_window[i] = c->cls_window[i];
        p.cls_sinks[i] = c->cls_sinks[i];
        p.cls_gated[i] = c->cls_gated[i];
        int n = 0;
        for (int l = lb; l < le; ++l) n += (c->layers[l].cls == i);
        p.cls_layers_in_call[i] = n;
        if (n && (mode == 0 || c->cls_gated[i])) any = true;  // modes 1 and 2 touch gated layers only
    }
    if (!any) return ODA_OK;  // e.g. a Full call over fixed-window layers only
    p.advance_seq_lens = advance;
    p.allow_empty = c->allow_empty ? 1 : 0;
    if (publish) {
        p.flags_out = publish->flags;
        p.scores_out = publish->scores;
        p.logits_out = publish->logits;
        p.counters_out = publish->counters;
    }
    p.done_counter = reinterpret_cast<int32_t*>(c->ws + c->lay.status + 128);
    p.exit_counter = reinterpret_cast<int32_t*>(c->ws + c->lay.status + 192);
    p.num_sms = c->num_sms;
    if (c->calibrating) p.sm_stats = reinterpret_cast<unsigned long long*>(c->ws + c->lay.sm_bytes);
    if (c->calibrated) {
        p.cum_share = reinterpret_cast<const uint16_t*>(c->ws + c->lay.cum_share);
        p.sm_claims = reinterpret_cast<int32_t*>(c->ws + c->lay.sm_claims);
    }
    if (advanced) *advanced = advance != nullptr;
    // A Local call over few layers cannot fill the usual grid: the window bounds its pages whatever
    // the lengths are.  Launch only the CTAs the plan can give a span to (it cuts the page axis into
    // min(grid, max(1, pages / min_span_pages)) spans either way, so the split and the bits are the same);
    // the rest would only start, build the plan and leave.
    int grid = c->grid;
    if (mode == 0 && c->min_span_pages > 0) {
        long long bound = 0;  // pages on the axis, at most
        for (int l = lb; l < le; ++l) {
            const int cls = c->layers[l].cls;
            const long long tokens = (long long)c->cls_window[cls] + c->cls_sinks[cls];  // one range when they touch
            bound += (long long)batch * f.num_kv_heads * (tokens / kPage + 2);
        }
        const long long need = bound / c->min_span_pages;   // the plan rounds down too
        if (need < grid) grid = (int)std::max<long long>(need, 1);
    }
    {   // necessary for the batch-1 one-unit-per-CTA plan, whatever the length turns out to be
        const long long units = (long long)(le - lb) * f.num_kv_heads;
        // (the last condition of unit_aligned_shape at the longest unit the windows allow: where it fails, the
        // launch is better off with the plan in registers than with a hint the device then turns down)
        long long umax_bound = 0;
        for (int l = lb; l < le; ++l) {
            const int cls = c->layers[l].cls;
            umax_bound = std::max(umax_bound, ((long long)c->cls_window[cls] + c->cls_sinks[cls]) / kPage + 2);
        }
        const bool lone_cta_ok = units >= 150 || umax_bound * (150 - units) <= 4200;
        p.direct_hint = (mode == 0 && batch == 1 && c->snap_span_pages > 0 && units <= grid && grid <= 4 * units && lone_cta_ok) ? 1 : 0;
        // one request and one layer class in the call: every unit has the same length, whatever it turns out to be
        int classes_in_call = 0;
        for (int i = 0; i < c->ncls; ++i) classes_in_call += p.cls_layers_in_call[i] > 0;
        p.uniform_hint = (mode == 0 && batch == 1 && c->ncls == 1 && classes_in_call == 1) ? 1 : 0;
    }
    cudaError_t e;
    if (c->variant == ODA_VARIANT_TMA_MMA) {
        if (c->kmap_base != k) {
            if (!encode_kv_map(c->kmap, k, f.head_dim, f.num_kv_heads, f.kv_token_stride, f.kv_head_stride,
                               f.kv_block_stride, c->blocks_bound))
                return fail(c, ODA_ERR_CUDA, "cuTensorMapEncodeTiled failed for k_cache");
            c->kmap_base = k;
        }
        if (c->vmap_base != v) {
            if (!encode_kv_map(c->vmap, v, f.head_dim, f.num_kv_heads, f.kv_token_stride, f.kv_head_stride,
                               f.kv_block_stride, c->blocks_bound))
                return fail(c, ODA_ERR_CUDA, "cuTensorMapEncodeTiled failed for v_cache");
            c->vmap_base = v;
        }
        e = launch_splitkv_tma(p, c->kmap, c->vmap, c->blocks_per_layer, f.head_dim, c->group, grid, st, c->use_pdl);
    } else {
        e = launch_splitkv_simt(p, f.head_dim, c->group, grid, st, c->use_pdl);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "attention kernel launch");
    c->launches += 1;
    return ODA_OK;
}

}  // namespace

extern "C" {

const char* oda_version(void) { return "oda-b200 0.1 (sm_100a)"; }

const char* oda_status_string(oda_status_t s)
{
    switch (s) {
        case ODA_OK: return "ok";
        case ODA_ERR_INVALID_ARG: return "invalid argument";
        case ODA_ERR_UNSUPPORTED: return "unsupported shape";
        case ODA_ERR_WORKSPACE: return "workspace missing or too small";
        case ODA_ERR_CUDA: return "CUDA runtime error";
        case ODA_ERR_DEVICE_STATUS: return "device status word set";
    }
    return "unknown status";
}

const char* oda_last_error(const oda_ctx_t* ctx) { return ctx ? ctx->err.c_str() : "null context"; }
int64_t oda_launch_count(const oda_ctx_t* ctx) { return ctx ? ctx->launches : 0; }
int32_t oda_resolved_variant(const oda_ctx_t* ctx) { return ctx ? ctx->variant : 0; }
int32_t oda_attention_grid(const oda_ctx_t* ctx) { return ctx ? ctx->grid : 0; }

oda_status_t oda_create(const oda_config_t* cfg, oda_ctx_t** out_ctx)
{
    if (!cfg || !out_ctx) return ODA_ERR_INVALID_ARG;
    *out_ctx = nullptr;
    if (cfg->num_layers < 1 || cfg->num_layers > kMaxLayers) return ODA_ERR_INVALID_ARG;
    if (cfg->num_kv_heads < 1 || cfg->num_q_heads < 1 || cfg->num_q_heads % cfg->num_kv_heads)
        return ODA_ERR_INVALID_ARG;
    if (cfg->max_batch < 1 || cfg->max_batch > kMaxBatch || cfg->max_blocks_per_seq < 1)
        return ODA_ERR_INVALID_ARG;
    if (!cfg->layer_window || !cfg->layer_sinks || !cfg->layer_gated) return ODA_ERR_INVALID_ARG;
    if (cfg->out_dtype != 0 && cfg->out_dtype != 1) return ODA_ERR_INVALID_ARG;
    if (!(cfg->sm_scale >= 0.f) || !std::isfinite(cfg->sm_scale)) return ODA_ERR_INVALID_ARG;
    if (cfg->head_d_ext < 0 || cfg->head_d_hidden < 0) return ODA_ERR_INVALID_ARG;
    if (cfg->variant < ODA_VARIANT_AUTO || cfg->variant > ODA_VARIANT_TMA_MMA) return ODA_ERR_INVALID_ARG;
    const int group = cfg->num_q_heads / cfg->num_kv_heads;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return ODA_ERR_UNSUPPORTED;
    if (cfg->block_size != kPage) return ODA_ERR_UNSUPPORTED;
    if (group != 1 && group != 2 && group != 4 && group != 8) return ODA_ERR_UNSUPPORTED;
    const int64_t strides[4] = {cfg->kv_layer_stride, cfg->kv_block_stride, cfg->kv_token_stride, cfg->kv_head_stride};
    for (int64_t s : strides)
        if (s < 0 || (s % 8) != 0) return ODA_ERR_INVALID_ARG;
    if (cfg->kv_token_stride < cfg->head_dim || cfg->kv_head_stride < cfg->head_dim ||
        cfg->kv_block_stride < (int64_t)cfg->head_dim * kPage)
        return ODA_ERR_INVALID_ARG;

    oda_ctx* c = new (std::nothrow) oda_ctx();
    if (!c) return ODA_ERR_INVALID_ARG;
    c->cfg = *cfg;
    c->group = group;
    c->scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.0f / std::sqrt((float)cfg->head_dim);
    c->layers.resize(cfg->num_layers);
    int max_kv_index = 0;
    for (int l = 0; l < cfg->num_layers; ++l) {
        LayerInfo li{};
        li.window = cfg->layer_window[l];
        li.sinks = cfg->layer_sinks[l];
        li.gated = cfg->layer_gated[l] ? 1 : 0;
        li.kv_index = cfg->layer_kv_index ? cfg->layer_kv_index[l] : l;
        if (li.window < 1 || li.sinks < 0 || li.kv_index < 0 || li.kv_index > 65535) {
            delete c;
            return ODA_ERR_INVALID_ARG;
        }
        if (li.kv_index > max_kv_index) max_kv_index = li.kv_index;
        int cls = -1;
        for (int i = 0; i < c->ncls; ++i)
            if (c->cls_window[i] == li.window && c->cls_sinks[i] == li.sinks && c->cls_gated[i] == li.gated) cls = i;
        if (cls < 0) {
            if (c->ncls == kMaxClasses) {
                delete c;
                return ODA_ERR_UNSUPPORTED;  // more than kMaxClasses distinct (window, sinks, gated)
            }
            cls = c->ncls++;
            c->cls_window[cls] = li.window;
            c->cls_sinks[cls] = li.sinks;
            c->cls_gated[cls] = li.gated;
        }
        li.cls = cls;
        if (li.gated) c->last_gated = l;
        c->layers[l] = li;
    }
    c->cfg.layer_window = nullptr;  // the copies above are what the library uses
    c->cfg.layer_sinks = nullptr;
    c->cfg.layer_gated = nullptr;
    c->cfg.layer_kv_index = nullptr;
    c->phys_layers = max_kv_index + 1;
    const bool tma_ok = tma_variant_supported(cfg->head_dim, cfg->kv_layer_stride, cfg->kv_block_stride, c->phys_layers);
    if (c->phys_layers > 1) {
        c->blocks_per_layer = tma_ok ? (int)(cfg->kv_layer_stride / cfg->kv_block_stride) : 0;
        c->blocks_bound = (int64_t)c->phys_layers * c->blocks_per_layer;
    } else {
        c->blocks_per_layer = 0;
        c->blocks_bound = (int64_t)1 << 30;
    }
    if (cfg->variant == ODA_VARIANT_TMA_MMA && !tma_ok) {
        delete c;
        return ODA_ERR_UNSUPPORTED;  // layer stride is not a whole number of blocks
    }
    if (cfg->options < 0 || cfg->options > 7) {
        delete c;
        return ODA_ERR_INVALID_ARG;
    }
    c->use_pdl = (cfg->options & 1) == 0;
    c->reuse_local = (cfg->options & 2) != 0;
    c->allow_empty = (cfg->options & 4) != 0;
    c->variant = cfg->variant == ODA_VARIANT_AUTO ? (tma_ok ? ODA_VARIANT_TMA_MMA : ODA_VARIANT_SIMT) : cfg->variant;
    if (c->reuse_local && c->variant != ODA_VARIANT_TMA_MMA) {
        delete c;
        return ODA_ERR_UNSUPPORTED;  // the remainder-only gated pass exists in the TMA variant only
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
        c->num_sms = sms;
        int occ = c->variant == ODA_VARIANT_TMA_MMA ? occupancy_splitkv_tma(cfg->head_dim, group)
                                                    : occupancy_splitkv_simt(cfg->head_dim, group);
        c->grid = sms * (occ > 0 ? occ : 1);
    } else {
        (void)cudaGetLastError();
        c->num_sms = 148;  // no device visible: sizes follow a B200 so that host-only checks still work
        c->grid = 148 * 2;
    }
    c->max_items = c->grid + cfg->num_layers * cfg->max_batch * cfg->num_kv_heads;
    c->head_grid = cfg->head_d_hidden > 0 ? recall_head_grid(cfg->head_d_hidden) : 1;
    compute_layout(c);
    *out_ctx = c;
    return ODA_OK;
}

void oda_destroy(oda_ctx_t* ctx) { delete ctx; }

oda_status_t oda_workspace_bytes(const oda_ctx_t* ctx, size_t* bytes)
{
    if (!ctx || !bytes) return ODA_ERR_INVALID_ARG;
    *bytes = ctx->lay.total;
    return ODA_OK;
}

oda_status_t oda_set_workspace(oda_ctx_t* c, void* dev_ptr, size_t bytes, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!dev_ptr || (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) != 0)
        return fail(c, ODA_ERR_WORKSPACE, "workspace pointer is null or not 256-byte aligned");
    if (bytes < c->lay.total) return fail(c, ODA_ERR_WORKSPACE, "workspace smaller than oda_workspace_bytes()");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(dev_ptr);
    cudaError_t e = cudaMemsetAsync(ws, 0, c->lay.partials, st);  // status, tickets, head scratch
    if (e != cudaSuccess) return cuda_fail(c, e, "workspace memset");
    e = cudaMemcpyAsync(ws + c->lay.layers, c->layers.data(), c->layers.size() * sizeof(LayerInfo),
                        cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(c, e, "layer table upload");
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "workspace initialisation");
    c->ws = ws;
    c->calibrated = false;  // the table lives in the workspace
    return ODA_OK;
}

oda_status_t oda_set_cache_resident_bytes(oda_ctx_t* c, size_t bytes)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    c->l2_resident_bytes = bytes;
    return ODA_OK;
}

oda_status_t oda_calibration_begin(oda_ctx_t* c, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    cudaError_t e = cudaMemsetAsync(c->ws + c->lay.sm_bytes, 0, 2 * 1024 * sizeof(unsigned long long),
                                    static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(c, e, "calibration memset");
    c->calibrated = false;  // measure under the equal split
    c->calibrating = true;
    return ODA_OK;
}

oda_status_t oda_calibration_end(oda_ctx_t* c, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    if (!c->calibrating) return fail(c, ODA_ERR_INVALID_ARG, "oda_calibration_begin has not been called");
    c->calibrating = false;
    // the weighted split assumes two resident CTAs per SM (the TMA variant's launch shape)
    if (c->variant != ODA_VARIANT_TMA_MMA || c->grid != 2 * c->num_sms || c->grid > kMaxGrid || c->num_sms > 1024)
        return ODA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<unsigned long long> h(2 * 1024);
    cudaError_t e = cudaMemcpyAsync(h.data(), c->ws + c->lay.sm_bytes, h.size() * sizeof(unsigned long long),
                                    cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "calibration read-back");
    std::vector<double> rate(c->num_sms);
    double total = 0.0, lo = 1e300, hi = 0.0;
    for (int i = 0; i < c->num_sms; ++i) {
        if (h[2 * i] == 0 || h[2 * i + 1] == 0) return ODA_OK;  // an SM saw no large launch: keep the equal split
        rate[i] = (double)h[2 * i] / (double)h[2 * i + 1];
        total += rate[i];
        lo = std::min(lo, rate[i]);
        hi = std::max(hi, rate[i]);
    }
    std::vector<uint16_t> cum(kMaxGrid + 1, 0);
    double acc = 0.0;
    for (int v = 0; v < c->grid; ++v) {
        cum[v] = (uint16_t)std::min(65535.0, std::floor(acc / total * 65536.0 + 0.5));
        acc += 0.5 * rate[v / 2];
    }
    e = cudaMemcpyAsync(c->ws + c->lay.cum_share, cum.data(), cum.size() * sizeof(uint16_t), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + c->lay.sm_claims, 0, 1024 * sizeof(int32_t), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "calibration table upload");
    c->calibrated = true;
    c->calib_spread = lo / hi;
    return ODA_OK;
}

double oda_calibration_spread(const oda_ctx_t* c) { return c && c->calibrated ? c->calib_spread : 0.0; }

oda_status_t oda_local_decode(oda_ctx_t* c, int32_t lb, int32_t le, int32_t batch, const void* q,
                              const void* k, const void* v, const int32_t* bt, const int32_t* sl,
                              void* out, float* lse, void* stream)
{
    oda_status_t s = check_attn_args(c, lb, le, batch, q, k, v, bt, sl, out);
    if (s != ODA_OK || batch == 0 || lb == le) return s;
    return launch_attention(c, 0, lb, le, batch, q, k, v, bt, sl, nullptr, out, lse,
                            static_cast<cudaStream_t>(stream));
}

oda_status_t oda_full_decode_gated(oda_ctx_t* c, int32_t lb, int32_t le, int32_t batch, const void* q,
                                   const void* k, const void* v, const int32_t* bt, const int32_t* sl,
                                   const uint8_t* flags, void* out, float* lse, void* stream)
{
    oda_status_t s = check_attn_args(c, lb, le, batch, q, k, v, bt, sl, out);
    if (s != ODA_OK || batch == 0 || lb == le) return s;
    if (!flags) return fail(c, ODA_ERR_INVALID_ARG, "flags is null");
    if (c->reuse_local && !lse) return fail(c, ODA_ERR_INVALID_ARG, "the remainder-only gated pass needs the Local pass's lse");
    return launch_attention(c, c->reuse_local ? 2 : 1, lb, le, batch, q, k, v, bt, sl, flags, out, lse,
                            static_cast<cudaStream_t>(stream));
}

oda_status_t oda_recall_score(oda_ctx_t* c, int32_t batch, const float* feat_ext, const void* attn_out_last,
                              const float* W1, const float* b1, const float* w2, const float* b2,
                              float threshold, const uint8_t* override_flags, float* scores,
                              float* logits, uint8_t* flags, int32_t* counters, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0) return ODA_OK;
    if (!scores || !flags) return fail(c, ODA_ERR_INVALID_ARG, "scores or flags is null");
    const oda_config_t& f = c->cfg;
    HeadParams p;
    std::memset(&p, 0, sizeof p);
    p.d_hidden = f.head_d_hidden;
    if (f.head_d_hidden > 0) {
        p.d_ext = f.head_d_ext;
        p.d_attn = f.head_use_attn_out ? f.num_q_heads * f.head_dim : 0;
        if (!W1 || !b1 || !w2 || !b2) return fail(c, ODA_ERR_INVALID_ARG, "head weights are null");
        if (p.d_ext > 0 && !feat_ext) return fail(c, ODA_ERR_INVALID_ARG, "feat_ext is null but head_d_ext > 0");
        if (p.d_attn > 0 && !attn_out_last) return fail(c, ODA_ERR_INVALID_ARG, "attn_out_last is null but head_use_attn_out is set");
        if (p.d_ext + p.d_attn < 1) return fail(c, ODA_ERR_INVALID_ARG, "the head has no input");
    } else if (!override_flags) {
        return fail(c, ODA_ERR_INVALID_ARG, "no head configured and no override_flags given");
    }
    p.feat_ext = feat_ext;
    p.attn_out = attn_out_last;
    p.W1 = W1; p.b1 = b1; p.w2 = w2; p.b2 = b2;
    p.override_flags = override_flags;
    p.scores = scores;
    p.logits = logits;
    p.flags = flags;
    p.counters = counters;
    p.partial = reinterpret_cast<float*>(c->ws + c->lay.head_partial);
    p.pre = reinterpret_cast<float*>(c->ws + c->lay.head_pre);
    p.rb_tickets = reinterpret_cast<int32_t*>(c->ws + c->lay.head_rb_tickets);
    p.ticket = reinterpret_cast<int32_t*>(c->ws + c->lay.status + 64);
    p.batch = batch;
    p.attn_bf16 = f.out_dtype;
    p.max_batch = f.max_batch;
    p.threshold = threshold;
    p.w1_stride = p.d_ext + p.d_attn;
    p.vec4 = (p.d_ext % 4 == 0) && (p.d_attn % 4 == 0) && aligned16(W1) && aligned16(feat_ext) &&
             aligned16(attn_out_last);
    cudaError_t e = launch_recall_head(p, static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "recall head launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_recall_preact(oda_ctx_t* c, int32_t batch, const float* feat_ext, const void* attn_out_last,
                               const float* W1_cols, int64_t w1_row_stride, float* pre_out, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0) return ODA_OK;
    const oda_config_t& f = c->cfg;
    if (f.head_d_hidden <= 0) return fail(c, ODA_ERR_INVALID_ARG, "no recall head configured");
    HeadParams p;
    std::memset(&p, 0, sizeof p);
    p.d_hidden = f.head_d_hidden;
    p.d_ext = f.head_d_ext;
    p.d_attn = f.head_use_attn_out ? f.num_q_heads * f.head_dim : 0;
    if (!W1_cols || !pre_out) return fail(c, ODA_ERR_INVALID_ARG, "W1_cols or pre_out is null");
    if (p.d_ext > 0 && !feat_ext) return fail(c, ODA_ERR_INVALID_ARG, "feat_ext is null but head_d_ext > 0");
    if (p.d_attn > 0 && !attn_out_last) return fail(c, ODA_ERR_INVALID_ARG, "attn_out_last is null but head_use_attn_out is set");
    if (p.d_ext + p.d_attn < 1) return fail(c, ODA_ERR_INVALID_ARG, "the head has no input on this rank");
    if (w1_row_stride < p.d_ext + p.d_attn) return fail(c, ODA_ERR_INVALID_ARG, "w1_row_stride is smaller than this rank's column count");
    p.feat_ext = feat_ext;
    p.attn_out = attn_out_last;
    p.W1 = W1_cols;
    p.w1_stride = w1_row_stride;
    p.pre_out = pre_out;
    p.pre = reinterpret_cast<float*>(c->ws + c->lay.head_pre);
    p.rb_tickets = reinterpret_cast<int32_t*>(c->ws + c->lay.head_rb_tickets);
    p.batch = batch;
    p.attn_bf16 = f.out_dtype;
    p.max_batch = f.max_batch;
    p.vec4 = (p.d_ext % 4 == 0) && (p.d_attn % 4 == 0) && (w1_row_stride % 4 == 0) && aligned16(W1_cols) &&
             aligned16(feat_ext) && aligned16(attn_out_last);
    cudaError_t e = launch_recall_head(p, static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "recall head (first layer) launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_recall_finalize(oda_ctx_t* c, int32_t batch, const float* pre_sum, const float* b1,
                                 const float* w2, const float* b2, float threshold, const uint8_t* override_flags,
                                 float* scores, float* logits, uint8_t* flags, int32_t* counters, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0) return ODA_OK;
    if (c->cfg.head_d_hidden <= 0) return fail(c, ODA_ERR_INVALID_ARG, "no recall head configured");
    if (!pre_sum || !b1 || !w2 || !b2 || !scores || !flags) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    HeadParams p;
    std::memset(&p, 0, sizeof p);
    p.d_hidden = c->cfg.head_d_hidden;
    p.b1 = b1; p.w2 = w2; p.b2 = b2;
    p.override_flags = override_flags;
    p.scores = scores;
    p.logits = logits;
    p.flags = flags;
    p.counters = counters;
    p.batch = batch;
    p.threshold = threshold;
    cudaError_t e = launch_recall_finalize(p, pre_sum, static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "recall head (second layer) launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_recall_finalize_exchange(oda_ctx_t* c, int32_t batch, int32_t world, int32_t rank_base,
                                          int32_t n_local, const oda_exchange_rank_t* ranks, float* const* recv,
                                          uint32_t* const* arrived, uint32_t epoch, uint64_t timeout_ns,
                                          const float* b1, const float* w2, const float* b2, float threshold,
                                          const uint8_t* override_flags, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0) return ODA_OK;
    if (c->cfg.head_d_hidden <= 0) return fail(c, ODA_ERR_INVALID_ARG, "no recall head configured");
    if (world < 1 || world > kExchangeMaxWorld) return fail(c, ODA_ERR_UNSUPPORTED, "world outside [1, 8]");
    if (n_local < 1 || rank_base < 0 || rank_base + n_local > world) return fail(c, ODA_ERR_INVALID_ARG, "ranks of this launch outside [0, world)");
    if (epoch == 0) return fail(c, ODA_ERR_INVALID_ARG, "epoch starts at 1 (the flag arrays start at 0)");
    if (!ranks || !recv || !arrived || !b1 || !w2 || !b2) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    ExchangeParams p;
    std::memset(&p, 0, sizeof p);
    for (int i = 0; i < n_local; ++i) {
        if (!ranks[i].pre_local || !ranks[i].scores || !ranks[i].flags) return fail(c, ODA_ERR_INVALID_ARG, "null rank buffer");
        if (!aligned16(ranks[i].pre_local)) return fail(c, ODA_ERR_INVALID_ARG, "pre_local must be 16-byte aligned");
        p.ranks[i].pre_local = ranks[i].pre_local;
        p.ranks[i].scores = ranks[i].scores;
        p.ranks[i].logits = ranks[i].logits;
        p.ranks[i].flags = ranks[i].flags;
        p.ranks[i].counters = ranks[i].counters;
    }
    for (int r = 0; r < world; ++r) {
        if (!recv[r] || !arrived[r]) return fail(c, ODA_ERR_INVALID_ARG, "null receive buffer or flag array");
        if (!aligned16(recv[r])) return fail(c, ODA_ERR_INVALID_ARG, "receive buffers must be 16-byte aligned");
        p.recv[r] = recv[r];
        p.arrived[r] = arrived[r];
    }
    p.b1 = b1; p.w2 = w2; p.b2 = b2;
    p.override_flags = override_flags;
    p.status = c->ws ? reinterpret_cast<int32_t*>(c->ws + c->lay.status) : nullptr;
    p.timeout_ns = timeout_ns ? timeout_ns : 1000000000ull;
    p.batch = batch;
    p.d_hidden = c->cfg.head_d_hidden;
    p.world = world;
    p.rank_base = rank_base;
    p.epoch = epoch;
    p.threshold = threshold;
    cudaError_t e = launch_recall_exchange(p, n_local, static_cast<cudaStream_t>(stream), c->use_pdl && n_local == 1);
    if (e != cudaSuccess) return cuda_fail(c, e, "recall head (exchange + second layer) launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_merge_partials_exchange(oda_ctx_t* c, int32_t world, int32_t rank_base, int32_t n_local,
                                         const oda_merge_exchange_rank_t* ranks, float* const* recv_out,
                                         float* const* recv_lse, uint32_t* const* arrived, uint32_t epoch,
                                         uint64_t timeout_ns, int32_t lb, int32_t le, int32_t batch, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    const oda_config_t& f = c->cfg;
    if (world < 1 || world > kExchangeMaxWorld) return fail(c, ODA_ERR_UNSUPPORTED, "world outside [1, 8]");
    if (n_local < 1 || rank_base < 0 || rank_base + n_local > world) return fail(c, ODA_ERR_INVALID_ARG, "ranks of this launch outside [0, world)");
    if (lb < 0 || le > f.num_layers || lb > le) return fail(c, ODA_ERR_INVALID_ARG, "bad layer range");
    if (batch < 0 || batch > f.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0 || lb == le) return ODA_OK;
    if (f.out_dtype != 0) return fail(c, ODA_ERR_UNSUPPORTED, "parts are merged in fp32: create the context with out_dtype 0");
    if (epoch == 0) return fail(c, ODA_ERR_INVALID_ARG, "epoch starts at 1 (the flag arrays start at 0)");
    if (!ranks || !recv_out || !recv_lse || !arrived) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    MergeExchangeParams p;
    std::memset(&p, 0, sizeof p);
    for (int i = 0; i < n_local; ++i) {
        if (!ranks[i].part_out || !ranks[i].part_lse || !ranks[i].out) return fail(c, ODA_ERR_INVALID_ARG, "null rank buffer");
        p.ranks[i].part_out = ranks[i].part_out;
        p.ranks[i].part_lse = ranks[i].part_lse;
        p.ranks[i].tokens_local = ranks[i].tokens_local;
        p.ranks[i].flags = ranks[i].flags;
        p.ranks[i].out = static_cast<float*>(ranks[i].out);
        p.ranks[i].lse = ranks[i].lse;
    }
    for (int r = 0; r < world; ++r) {
        if (!recv_out[r] || !recv_lse[r] || !arrived[r]) return fail(c, ODA_ERR_INVALID_ARG, "null receive buffer or flag array");
        p.recv_out[r] = recv_out[r];
        p.recv_lse[r] = recv_lse[r];
        p.arrived[r] = arrived[r];
    }
    p.layers = reinterpret_cast<const LayerInfo*>(c->ws + c->lay.layers);
    p.status = reinterpret_cast<int32_t*>(c->ws + c->lay.status);
    p.timeout_ns = timeout_ns ? timeout_ns : 1000000000ull;
    p.batch = batch;
    p.q_heads = f.num_q_heads;
    p.num_layers = f.num_layers;
    p.layer_begin = lb;
    p.layer_end = le;
    p.world = world;
    p.rank_base = rank_base;
    p.epoch = epoch;
    cudaError_t e = launch_merge_exchange(p, n_local, f.head_dim, static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "partial exchange + merge launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_write_current_kv(oda_ctx_t* c, int32_t batch, const void* k_cur, const void* v_cur,
                                  const uint8_t* mask, void* k_cache, void* v_cache, const int32_t* bt,
                                  const int32_t* sl, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0) return ODA_OK;
    if (!k_cur || !v_cur || !k_cache || !v_cache || !bt || !sl) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(k_cur) || !aligned16(v_cur) || !aligned16(k_cache) || !aligned16(v_cache))
        return fail(c, ODA_ERR_INVALID_ARG, "k_cur, v_cur and the caches must be 16-byte aligned");
    const oda_config_t& f = c->cfg;
    cudaError_t e = launch_write_current_kv(
        k_cur, v_cur, mask, k_cache, v_cache, bt, sl, reinterpret_cast<const LayerInfo*>(c->ws + c->lay.layers),
        f.num_layers, batch, f.num_kv_heads, f.head_dim, f.max_blocks_per_seq, f.kv_layer_stride, f.kv_block_stride,
        f.kv_token_stride, f.kv_head_stride, reinterpret_cast<int32_t*>(c->ws + c->lay.status),
        static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "commit kernel launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_merge_partials(oda_ctx_t* c, int32_t n_parts, int32_t lb, int32_t le, int32_t batch,
                                const float* parts_out, const float* parts_lse, const int32_t* part_tokens,
                                const uint8_t* flags, void* out, float* lse, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    const oda_config_t& f = c->cfg;
    if (n_parts < 1 || n_parts > 64) return fail(c, ODA_ERR_INVALID_ARG, "n_parts outside [1, 64]");
    if (lb < 0 || le > f.num_layers || lb > le) return fail(c, ODA_ERR_INVALID_ARG, "bad layer range");
    if (batch < 0 || batch > f.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0 || lb == le) return ODA_OK;
    if (f.out_dtype != 0) return fail(c, ODA_ERR_UNSUPPORTED, "parts are merged in fp32: create the context with out_dtype 0");
    if (!parts_out || !parts_lse || !out) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(parts_out) || !aligned16(out)) return fail(c, ODA_ERR_INVALID_ARG, "parts_out and out must be 16-byte aligned");
    cudaError_t e = launch_merge_partials(parts_out, parts_lse, part_tokens, flags,
                                          reinterpret_cast<const LayerInfo*>(c->ws + c->lay.layers),
                                          static_cast<float*>(out), lse, n_parts, lb, le, batch, f.num_q_heads,
                                          f.head_dim, f.num_layers, static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "partial merge launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_advance_seq_lens(oda_ctx_t* c, int32_t batch, int32_t* seq_lens, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (batch < 0 || batch > c->cfg.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (batch == 0) return ODA_OK;
    if (!seq_lens) return fail(c, ODA_ERR_INVALID_ARG, "seq_lens is null");
    cudaError_t e = launch_advance_seq_lens(seq_lens, batch, static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "seq_lens advance launch");
    c->launches += 1;
    return ODA_OK;
}

oda_status_t oda_select_rows(oda_ctx_t* c, int32_t batch, const void* local, const void* full,
                             const uint8_t* flags, void* out, int64_t row_bytes, void* stream)
{
    if (!c) return ODA_ERR_INVALID_ARG;
    if (batch < 0 || row_bytes < 0 || (row_bytes % 16) != 0) return fail(c, ODA_ERR_INVALID_ARG, "bad batch or row size");
    if (batch == 0 || row_bytes == 0) return ODA_OK;
    if (!local || !full || !flags || !out) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(local) || !aligned16(full) || !aligned16(out))
        return fail(c, ODA_ERR_INVALID_ARG, "rows must be 16-byte aligned");
    cudaError_t e = launch_select_rows(local, full, flags, out, batch, (size_t)row_bytes,
                                       static_cast<cudaStream_t>(stream), c->use_pdl);
    if (e != cudaSuccess) return cuda_fail(c, e, "select kernel launch");
    c->launches += 1;
    return ODA_OK;
}

int64_t oda_full_head_param_count(int32_t d_model, int32_t d_tower, int32_t d_ff, int32_t n_blocks)
{
    if (d_model < 1 || d_tower < 1 || d_ff < 1 || n_blocks < 0) return 0;
    return full_head_param_count(d_model, d_tower, d_ff, n_blocks);
}

size_t oda_full_head_scratch_bytes(const oda_full_head_t* h, int32_t batch)
{
    if (!h || batch < 1) return 0;
    return full_head_scratch_bytes(h->d_model, h->d_tower, h->d_ff, batch);
}

oda_status_t oda_recall_score_full(oda_ctx_t* c, int32_t batch, const oda_full_head_t* h, const float* h_prev,
                                   const float* emb, const float* h_local, float threshold,
                                   const uint8_t* override_flags, float* scores, float* logits, uint8_t* flags,
                                   int32_t* counters, void* scratch, size_t scratch_bytes, void* stream)
{
    if (!c || !h) return ODA_ERR_INVALID_ARG;
    if (batch < 0 || batch > kMaxBatch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, 128]");
    if (batch == 0) return ODA_OK;
    if (h->d_model < 4 || h->d_tower < 8 || h->d_ff < 4 || h->n_blocks < 0 || !(h->eps >= 0.f))
        return fail(c, ODA_ERR_INVALID_ARG, "bad head dimensions");
    if ((h->d_model % 4) || (h->d_tower % 8) || (h->d_ff % 4))
        return fail(c, ODA_ERR_UNSUPPORTED, "d_model and d_ff must be multiples of 4, d_tower of 8");
    if (!h->params || !h_prev || !emb || !h_local || !scores || !flags || !scratch)
        return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    if (h->variant < 0 || h->variant > 3) return fail(c, ODA_ERR_INVALID_ARG, "head variant outside 0..3");
    if (!aligned16(h->params) || !aligned16(h_prev) || !aligned16(emb) || !aligned16(h_local) ||
        (reinterpret_cast<uintptr_t>(scratch) % 256) != 0)
        return fail(c, ODA_ERR_INVALID_ARG, "parameters and inputs must be 16-byte aligned, scratch 256-byte aligned");
    if (scratch_bytes < full_head_scratch_bytes(h->d_model, h->d_tower, h->d_ff, batch))
        return fail(c, ODA_ERR_WORKSPACE, "scratch smaller than oda_full_head_scratch_bytes()");
    int launches = 0;
    cudaError_t e = launch_full_head(batch, h->d_model, h->d_tower, h->d_ff, h->n_blocks, h->eps, h->params, h_prev,
                                     emb, h_local, threshold, override_flags, scores, logits, flags, counters,
                                     scratch, static_cast<cudaStream_t>(stream), c->use_pdl, &launches,
                                     h->variant == 3 ? 0 : h->variant,
                                     c->ws ? reinterpret_cast<int32_t*>(c->ws + c->lay.status) : nullptr,
                                     h->variant == 3 ? 2 : 0);
    c->launches += launches;
    if (e == cudaErrorNotSupported) {
        (void)cudaGetLastError();
        return fail(c, ODA_ERR_UNSUPPORTED, "the fused head needs batch <= 4 and a device that can hold one CTA per SM cooperatively");
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "full recall head launch");
    return ODA_OK;
}

oda_status_t oda_recall_score_full_pre(oda_ctx_t* c, int32_t batch, const oda_full_head_t* h, const float* h_prev,
                                       const float* emb, void* scratch, size_t scratch_bytes, void* stream)
{
    if (!c || !h) return ODA_ERR_INVALID_ARG;
    if (batch < 0 || batch > kMaxBatch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, 128]");
    if (batch == 0) return ODA_OK;
    if (h->d_model < 4 || h->d_tower < 8 || h->d_ff < 4 || h->n_blocks < 0 || !(h->eps >= 0.f))
        return fail(c, ODA_ERR_INVALID_ARG, "bad head dimensions");
    if ((h->d_model % 4) || (h->d_tower % 8) || (h->d_ff % 4))
        return fail(c, ODA_ERR_UNSUPPORTED, "d_model and d_ff must be multiples of 4, d_tower of 8");
    if (!h->params || !h_prev || !emb || !scratch) return fail(c, ODA_ERR_INVALID_ARG, "null pointer");
    if (!aligned16(h->params) || !aligned16(h_prev) || !aligned16(emb) || (reinterpret_cast<uintptr_t>(scratch) % 256) != 0)
        return fail(c, ODA_ERR_INVALID_ARG, "parameters and inputs must be 16-byte aligned, scratch 256-byte aligned");
    if (scratch_bytes < full_head_scratch_bytes(h->d_model, h->d_tower, h->d_ff, batch))
        return fail(c, ODA_ERR_WORKSPACE, "scratch smaller than oda_full_head_scratch_bytes()");
    int launches = 0;
    cudaError_t e = launch_full_head(batch, h->d_model, h->d_tower, h->d_ff, h->n_blocks, h->eps, h->params, h_prev,
                                     emb, nullptr, 0.f, nullptr, nullptr, nullptr, nullptr, nullptr, scratch,
                                     static_cast<cudaStream_t>(stream), c->use_pdl, &launches, 0, nullptr, 1);
    c->launches += launches;
    if (e != cudaSuccess) return cuda_fail(c, e, "full recall head (first part) launch");
    return ODA_OK;
}

oda_status_t oda_step(oda_ctx_t* c, const oda_step_args_t* a, void* stream)
{
    if (!c || !a) return ODA_ERR_INVALID_ARG;
    const oda_config_t& f = c->cfg;
    const int B = a->batch, L = f.num_layers;
    oda_status_t s = check_attn_args(c, 0, L, B, a->q_local, a->k_cache, a->v_cache, a->block_table,
                                     a->seq_lens, a->out);
    if (s != ODA_OK || B == 0) return s;
    if (!a->scores || !a->flags) return fail(c, ODA_ERR_INVALID_ARG, "scores or flags is null");
    const bool paper_head = a->full_head != nullptr;
    if (f.head_d_hidden == 0 && !paper_head && !a->override_flags)
        return fail(c, ODA_ERR_INVALID_ARG, "no head configured and no override_flags given");
    const void* qf = a->q_full ? a->q_full : a->q_local;
    if (!aligned16(qf)) return fail(c, ODA_ERR_INVALID_ARG, "q_full must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((a->k_cur_local == nullptr) != (a->v_cur_local == nullptr) || (a->k_cur_full == nullptr) != (a->v_cur_full == nullptr))
        return fail(c, ODA_ERR_INVALID_ARG, "K and V candidates must be given together");
    if (a->hidden_out && (!a->hidden_local || !a->hidden_full))
        return fail(c, ODA_ERR_INVALID_ARG, "hidden_out needs hidden_local and hidden_full");
    if (a->k_cur_local) {  // the Local candidate of the current token, for every request
        s = oda_write_current_kv(c, B, a->k_cur_local, a->v_cur_local, nullptr, const_cast<void*>(a->k_cache),
                                 const_cast<void*>(a->v_cache), a->block_table, a->seq_lens, stream);
        if (s != ODA_OK) return s;
    }
    float* step_lse = a->lse;
    if (!step_lse && c->reuse_local) step_lse = reinterpret_cast<float*>(c->ws + c->lay.own_lse);
    s = launch_attention(c, 0, 0, L, B, a->q_local, a->k_cache, a->v_cache, a->block_table, a->seq_lens,
                         nullptr, a->out, step_lse, st);
    if (s != ODA_OK) return s;
    const char* attn_last = nullptr;
    if (c->last_gated >= 0 && f.head_use_attn_out)
        attn_last = static_cast<const char*>(a->out) + (size_t)c->last_gated * B * f.num_q_heads * f.head_dim * out_elem(c);
    // Without a head the decision is the caller's forced flags: the Full kernel reads them
    // directly and publishes them, which saves the decision kernel's launch.
    const bool fused_decision = !paper_head && f.head_d_hidden == 0 && c->last_gated >= 0;
    const uint8_t* decided = fused_decision ? a->override_flags : a->flags;  // valid once the head (if any) has run
    if (paper_head) {
        // (variant 3: the caller has run oda_recall_score_full_pre on head_scratch since the last step;
        // only the part that needs the Local hidden state is left for after the Local pass)
        s = oda_recall_score_full(c, B, a->full_head, a->head_h_prev, a->head_emb, a->head_h_local, a->threshold,
                                  a->override_flags, a->scores, a->logits, a->flags, a->counters, a->head_scratch,
                                  a->head_scratch_bytes, stream);
        if (s != ODA_OK) return s;
    } else if (!fused_decision) {
        s = oda_recall_score(c, B, a->feat_ext, attn_last, a->W1, a->b1, a->w2, a->b2, a->threshold,
                             a->override_flags, a->scores, a->logits, a->flags, a->counters, stream);
        if (s != ODA_OK) return s;
    }
    if (a->k_cur_full) {  // requests that recall keep the Full branch's candidate
        s = oda_write_current_kv(c, B, a->k_cur_full, a->v_cur_full, decided, const_cast<void*>(a->k_cache),
                                 const_cast<void*>(a->v_cache), a->block_table, a->seq_lens, stream);
        if (s != ODA_OK) return s;
    }
    if (a->hidden_out) {
        s = oda_select_rows(c, B, a->hidden_local, a->hidden_full, decided, a->hidden_out, a->hidden_row_bytes, stream);
        if (s != ODA_OK) return s;
    }
    bool advanced = false;
    if (c->last_gated >= 0) {
        // the Full kernel is the last reader of seq_lens in the step: it also advances them
        s = launch_attention(c, c->reuse_local ? 2 : 1, 0, L, B, qf, a->k_cache, a->v_cache, a->block_table, a->seq_lens,
                             fused_decision ? a->override_flags : a->flags, a->out, step_lse, st,
                             a->advance_seq_lens ? a->seq_lens : nullptr, &advanced, fused_decision ? a : nullptr);
        if (s != ODA_OK) return s;
    }
    if (a->advance_seq_lens && !advanced) {
        cudaError_t e = launch_advance_seq_lens(a->seq_lens, B, st, c->use_pdl);
        if (e != cudaSuccess) return cuda_fail(c, e, "seq_lens advance launch");
        c->launches += 1;
    }
    return ODA_OK;
}

// The device's address for a suitably aligned pointer into pinned (page-locked, mapped) host
// memory; nullptr for anything else (pageable memory is only reachable through a copy).
static void* device_view_of_pinned(const void* host, uintptr_t align)
{
    if (!host || (reinterpret_cast<uintptr_t>(host) & (align - 1))) return nullptr;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

oda_status_t oda_step_host(oda_ctx_t* c, const oda_step_args_t* a, void* stream, size_t* h2d_bytes,
                           size_t* d2h_bytes)
{
    if (!c || !a) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    const oda_config_t& f = c->cfg;
    const int B = a->batch;
    if (B < 0 || B > f.max_batch) return fail(c, ODA_ERR_INVALID_ARG, "batch outside [0, max_batch]");
    if (h2d_bytes) *h2d_bytes = 0;
    if (d2h_bytes) *d2h_bytes = 0;
    if (B == 0) return ODA_OK;
    if (!a->q_local || !a->out || !a->scores || !a->flags) return fail(c, ODA_ERR_INVALID_ARG, "null host pointer");
    if (a->k_cur_local || a->v_cur_local || a->k_cur_full || a->v_cur_full || a->hidden_out || a->full_head)
        return fail(c, ODA_ERR_INVALID_ARG, "the commit and full-head fields take device pointers: use oda_step");
    if (f.head_d_ext > 0 && f.head_d_hidden > 0 && !a->feat_ext) return fail(c, ODA_ERR_INVALID_ARG, "feat_ext is null");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)f.num_layers * B * f.num_q_heads;
    const size_t qbytes = rows * f.head_dim * 2;
    size_t up = 0, down = 0;
    oda_step_args_t d = *a;
    cudaError_t e;
    // Inputs: when every one of them is pinned memory the device can address, one kernel pulls them
    // all into the staging areas (one launch instead of up to four copy-engine transfers, and the
    // first attention kernel's set-up overlaps it); otherwise one copy each.
    const size_t feat_bytes = (a->feat_ext && f.head_d_ext > 0) ? (size_t)B * f.head_d_ext * 4 : 0;
    StageIn si;
    std::memset(&si, 0, sizeof si);
    const void* hosts[4] = {nullptr, nullptr, nullptr, nullptr};
    bool pull = true;
    int nsi = 0;
    auto want = [&](const void* host, size_t off, size_t bytes) {
        if (!host || !bytes) return;
        void* dv = device_view_of_pinned(host, bytes >= 16 ? 16 : 1);
        if (!dv) pull = false;
        hosts[nsi] = host;
        si.src[nsi] = dv;
        si.dst[nsi] = c->ws + off;
        si.bytes[nsi] = (long long)bytes;
        ++nsi;
        up += bytes;
    };
    want(a->q_local, c->lay.st_q_local, qbytes);
    want(a->q_full, c->lay.st_q_full, qbytes);
    want(a->feat_ext, c->lay.st_feat, feat_bytes);
    want(a->override_flags, c->lay.st_override, (size_t)B);
    if (pull) {
        e = launch_stage_in(si, st, c->use_pdl);
        if (e != cudaSuccess) return cuda_fail(c, e, "input staging kernel launch");
        c->launches += 1;
    } else {
        for (int k = 0; k < nsi; ++k) {
            e = cudaMemcpyAsync(si.dst[k], hosts[k], (size_t)si.bytes[k], cudaMemcpyHostToDevice, st);
            if (e != cudaSuccess) return cuda_fail(c, e, "host-to-device copy of a step input");
        }
    }
    d.q_local = c->ws + c->lay.st_q_local;
    if (a->q_full) d.q_full = c->ws + c->lay.st_q_full;
    if (feat_bytes) d.feat_ext = reinterpret_cast<const float*>(c->ws + c->lay.st_feat);
    if (a->override_flags) d.override_flags = reinterpret_cast<const uint8_t*>(c->ws + c->lay.st_override);
    // Where no kernel reads the step's outputs back (no recall head, no remainder-only Full pass: the
    // attention kernels only write them) and the caller's buffers are pinned memory the device can
    // address, the kernels write every output straight into them and no copy follows the last
    // kernel: the bus transfer overlaps the end of the launch and three engine switches go away.
    bool direct = f.head_d_hidden == 0 && !c->reuse_local;
    void* dv_out = nullptr; void* dv_lse = nullptr; void* dv_scores = nullptr; void* dv_logits = nullptr; void* dv_flags = nullptr;
    if (direct) {
        dv_out = device_view_of_pinned(a->out, 16);
        dv_scores = device_view_of_pinned(a->scores, 4);
        dv_flags = device_view_of_pinned(a->flags, 1);
        dv_lse = a->lse ? device_view_of_pinned(a->lse, 4) : nullptr;
        dv_logits = a->logits ? device_view_of_pinned(a->logits, 4) : nullptr;
        direct = dv_out && dv_scores && dv_flags && (!a->lse || dv_lse) && (!a->logits || dv_logits);
    }
    if (direct) {
        d.out = dv_out;
        d.lse = static_cast<float*>(dv_lse);
        d.scores = static_cast<float*>(dv_scores);
        d.logits = static_cast<float*>(dv_logits);
        d.flags = static_cast<uint8_t*>(dv_flags);
    } else {
        d.out = c->ws + c->lay.st_out;
        d.lse = a->lse ? reinterpret_cast<float*>(c->ws + c->lay.st_lse) : nullptr;
        d.scores = reinterpret_cast<float*>(c->ws + c->lay.st_scores);
        d.logits = a->logits ? reinterpret_cast<float*>(c->ws + c->lay.st_logits) : nullptr;
        d.flags = reinterpret_cast<uint8_t*>(c->ws + c->lay.st_flags);
    }
    oda_status_t s = oda_step(c, &d, stream);
    if (s != ODA_OK) return s;
#define ODA_DOWN(field, off, bytes)                                                                   \
    do {                                                                                              \
        e = cudaMemcpyAsync(a->field, c->ws + c->lay.off, (bytes), cudaMemcpyDeviceToHost, st);       \
        if (e != cudaSuccess) return cuda_fail(c, e, "device-to-host copy of " #field);               \
        down += (bytes);                                                                              \
    } while (0)
    if (direct) {  // already on their way; counted once per element
        down = rows * f.head_dim * out_elem(c) + (a->lse ? rows * 4 : 0) + (size_t)B * 4 + (a->logits ? (size_t)B * 4 : 0) + (size_t)B;
    } else {
        ODA_DOWN(out, st_out, rows * f.head_dim * out_elem(c));
        if (a->lse) ODA_DOWN(lse, st_lse, rows * 4);
        ODA_DOWN(scores, st_scores, (size_t)B * 4);
        if (a->logits) ODA_DOWN(logits, st_logits, (size_t)B * 4);
        ODA_DOWN(flags, st_flags, (size_t)B);
    }
#undef ODA_DOWN
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "stream synchronise");
    if (h2d_bytes) *h2d_bytes = up;
    if (d2h_bytes) *d2h_bytes = down;
    return ODA_OK;
}

oda_status_t oda_read_device_status(oda_ctx_t* c, void* stream, int32_t* code)
{
    if (!c || !code) return ODA_ERR_INVALID_ARG;
    if (!c->ws) return fail(c, ODA_ERR_WORKSPACE, "oda_set_workspace has not been called");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, c->ws + c->lay.status, sizeof v, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + c->lay.status, 0, sizeof v, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(c, e, "status read");
    *code = v;
    return v ? ODA_ERR_DEVICE_STATUS : ODA_OK;
}

}  // extern "C"
