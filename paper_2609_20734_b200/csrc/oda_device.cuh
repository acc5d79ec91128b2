// Shared device-side definitions of the ODA decode kernels: launch parameters, the
// per-CTA work plan (Eq. 1 ranges -> page chunks -> item list), item decoding and the
// log-sum-exp merge of split partials.  Used by both attention kernel variants.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace oda {

constexpr int kPage = 16;          // tokens per KV block
constexpr int kMaxBatch = 256;
constexpr int kMaxLayers = 256;
constexpr int kMaxClasses = 4;     // distinct (window, sinks, gated) triples in one stack

// device status bits
constexpr int kStatusBadSeqLen = 1;
constexpr int kStatusItemOverflow = 2;

struct LayerInfo {  // one per layer, in the workspace
    int32_t window, sinks, gated, kv_index, cls, pad0, pad1, pad2;
};

struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const int32_t* block_table;
    const int32_t* seq_lens;
    const uint8_t* flags;  // Full mode: per-request gate; Local mode: nullptr
    void* out;
    float* lse;
    float* partials;       // [max_items][G][D+2]: m (log2 units), l, unnormalised o
    int32_t* tickets;      // [num_layers][max_batch][Hkv], zero between launches
    int32_t* status;
    const LayerInfo* layers;
    int64_t kv_layer_stride, kv_block_stride, kv_token_stride, kv_head_stride;
    int32_t layer_begin, layer_end, batch, max_batch;
    int32_t num_q_heads, num_kv_heads, max_blocks_per_seq, out_bf16;
    int32_t mode;          // 0 = Local (Eq. 1 S^L), 1 = gated Full (S^F)
    int32_t ncls;
    int32_t items_per_cta; // target items per CTA used to size chunks
    int32_t min_chunk_pages;
    int32_t max_items;
    float scale_log2e;     // sm_scale * log2(e)
    int32_t cls_window[kMaxClasses], cls_sinks[kMaxClasses], cls_gated[kMaxClasses];
    int32_t cls_layers_in_call[kMaxClasses];
};

struct Plan {  // shared memory, one per CTA
    int32_t offsets[kMaxClasses][kMaxBatch + 1];  // exclusive prefix of chunks per request
    int32_t layer_base[kMaxLayers + 1];           // first item id of each layer in the call
    int32_t chunk_pages;
    int32_t total_items;
};

struct Item {
    int32_t layer, b, g;        // layer, request, kv head
    int32_t chunk, nchunks;     // this split and how many the unit has
    int32_t slot_base;          // partial slot of the unit's chunk 0
    int32_t t;                  // seq_len
    int32_t win_pg0, win_pg1;   // logical pages of this chunk
    int32_t win_lo, win_hi;     // valid positions of the window/full segment: [lo, hi)
    int32_t sink_pg1;           // sink pages [0, sink_pg1) (0 = none in this item)
    int32_t sink_hi;            // valid sink positions [0, sink_hi)
};

// Eq. 1 in 0-based form.  Local: sinks [0, min(s,t)), window [max(0,t-w), t); when they touch
// or overlap the set is the single range [0, t).  Full: [0, t).
struct Ranges {
    int32_t lo, hi;       // window (or whole) segment
    int32_t sink_hi;      // 0 if there is no separate sink segment
    int32_t pg0, pg1;     // pages of the window segment
};

__device__ __forceinline__ Ranges eq1_ranges(int mode, int t, int w, int s)
{
    Ranges r;
    r.hi = t;
    r.sink_hi = 0;
    if (mode == 1) {
        r.lo = 0;
    } else {
        int s_eff = s < t ? s : t;
        int lo = t - w > 0 ? t - w : 0;
        if (lo <= s_eff) {
            r.lo = 0;
        } else {
            r.lo = lo;
            r.sink_hi = s_eff;
        }
    }
    r.pg0 = r.lo / kPage;
    r.pg1 = (t + kPage - 1) / kPage;
    return r;
}

// Every CTA builds the same plan from device-resident seq_lens / flags: no host knowledge of
// lengths or flags is needed, so one captured launch serves every length and every gate.
__device__ inline void build_plan(const AttnParams& p, Plan& pl)
{
    const int tid = threadIdx.x, nth = blockDim.x;
    const int B = p.batch;
    for (int idx = tid; idx < p.ncls * B; idx += nth) {
        int c = idx / B, b = idx - c * B;
        int t = p.seq_lens[b];
        int np = 0;
        bool active = p.cls_layers_in_call[c] > 0 &&
                      (p.mode == 0 || (p.cls_gated[c] && p.flags[b] != 0));
        if (active) {
            if (t < 1) {
                atomicOr(p.status, kStatusBadSeqLen);
            } else {
                if (t > p.max_blocks_per_seq * kPage) {
                    t = p.max_blocks_per_seq * kPage;
                    atomicOr(p.status, kStatusBadSeqLen);
                }
                Ranges r = eq1_ranges(p.mode, t, p.cls_window[c], p.cls_sinks[c]);
                np = r.pg1 - r.pg0;
            }
        }
        pl.offsets[c][b + 1] = np;
    }
    __syncthreads();
    if (tid < 32) {
        long long tot = 0;
        for (int c = 0; c < p.ncls; ++c) {
            long long sc = 0;
            for (int b = tid; b < B; b += 32) sc += pl.offsets[c][b + 1];
            tot += sc * p.cls_layers_in_call[c];
        }
        for (int o = 16; o; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        tot *= p.num_kv_heads;
        long long denom = (long long)gridDim.x * p.items_per_cta;
        long long cp = (tot + denom - 1) / denom;
        if (cp < p.min_chunk_pages) cp = p.min_chunk_pages;
        if (tid == 0) pl.chunk_pages = (int)cp;
    }
    __syncthreads();
    const int cp = pl.chunk_pages;
    const int warp = tid >> 5, lane = tid & 31, nwarps = nth >> 5;
    for (int c = warp; c < p.ncls; c += nwarps) {  // one warp scans one class
        int carry = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            int b = b0 + lane;
            int np = b < B ? pl.offsets[c][b + 1] : 0;
            int n = (np + cp - 1) / cp;
            int x = n;
            for (int o = 1; o < 32; o <<= 1) {
                int y = __shfl_up_sync(0xffffffffu, x, o);
                if (lane >= o) x += y;
            }
            if (b < B) pl.offsets[c][b + 1] = carry + x;
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        if (lane == 0) pl.offsets[c][0] = 0;
    }
    __syncthreads();
    if (tid == 0) {
        int base = 0;
        for (int l = p.layer_begin; l < p.layer_end; ++l) {
            pl.layer_base[l - p.layer_begin] = base;
            base += p.num_kv_heads * pl.offsets[p.layers[l].cls][B];
        }
        pl.layer_base[p.layer_end - p.layer_begin] = base;
        if (base > p.max_items) {
            atomicOr(p.status, kStatusItemOverflow);
            base = 0;  // refuse to run rather than overrun the partial buffer
        }
        pl.total_items = base;
    }
    __syncthreads();
}

// item id -> (layer, request, kv head, chunk) and the token ranges it covers
__device__ inline Item decode_item(const AttnParams& p, const Plan& pl, int id)
{
    Item it;
    const int nl = p.layer_end - p.layer_begin;
    int lo = 0, hi = nl;  // last layer with layer_base <= id
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (pl.layer_base[mid] <= id) lo = mid; else hi = mid;
    }
    it.layer = p.layer_begin + lo;
    const LayerInfo li = p.layers[it.layer];
    const int c = li.cls;
    const int totc = pl.offsets[c][p.batch];
    int rem = id - pl.layer_base[lo];
    it.g = rem / totc;
    rem -= it.g * totc;
    int blo = 0, bhi = p.batch;  // last b with offsets[b] <= rem
    while (bhi - blo > 1) {
        int mid = (blo + bhi) >> 1;
        if (pl.offsets[c][mid] <= rem) blo = mid; else bhi = mid;
    }
    it.b = blo;
    it.chunk = rem - pl.offsets[c][blo];
    it.nchunks = pl.offsets[c][blo + 1] - pl.offsets[c][blo];
    it.slot_base = id - it.chunk;
    int t = p.seq_lens[it.b];
    if (t > p.max_blocks_per_seq * kPage) t = p.max_blocks_per_seq * kPage;
    it.t = t;
    Ranges r = eq1_ranges(p.mode, t, li.window, li.sinks);
    const int np = r.pg1 - r.pg0;
    const int per = (np + it.nchunks - 1) / it.nchunks;
    it.win_pg0 = r.pg0 + it.chunk * per;
    it.win_pg1 = min(it.win_pg0 + per, r.pg1);
    it.win_lo = r.lo;
    it.win_hi = r.hi;
    it.sink_hi = (it.chunk == 0) ? r.sink_hi : 0;
    it.sink_pg1 = (it.sink_hi + kPage - 1) / kPage;
    return it;
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Writes the normalised result of one (layer, request, kv head) unit for query head row hh.
template <int D>
__device__ __forceinline__ void store_out(const AttnParams& p, int layer, int b, int h, int d,
                                          float val)
{
    size_t idx = (((size_t)layer * p.batch + b) * p.num_q_heads + h) * D + d;
    if (p.out_bf16)
        reinterpret_cast<__nv_bfloat16*>(p.out)[idx] = __float2bfloat16_rn(val);
    else
        reinterpret_cast<float*>(p.out)[idx] = val;
}

// Split merge.  A unit (layer, request, kv head) with one chunk is normalised and stored by the
// CTA that computed it.  Otherwise each CTA publishes its partial [G][D+2] = (m, l, o[D]) in
// its slot, takes a ticket, and the CTA that arrives last (no waiting, one atomic) merges all
// chunks in chunk order, so the bits do not depend on scheduling.

__device__ __forceinline__ float* partial_slot(const AttnParams& p, const Item& it, int G, int W)
{
    return p.partials + (size_t)(it.slot_base + it.chunk) * (G * W);
}

// one thread calls this after the CTA's partial is visible (threadfence + barrier before)
__device__ __forceinline__ int take_ticket(const AttnParams& p, const Item& it)
{
    int* tk = p.tickets + ((size_t)it.layer * p.max_batch + it.b) * p.num_kv_heads + it.g;
    int old = atomicAdd(tk, 1);
    int last = (old == it.nchunks - 1);
    if (last) *tk = 0;  // ready for the next launch
    return last;
}

template <int D, int G>
__device__ inline void merge_chunks(const AttnParams& p, const Item& it, int tid, int nth)
{
    constexpr int W = D + 2;
    const float kLn2 = 0.6931471805599453f;
    const float* base = p.partials + (size_t)it.slot_base * (G * W);
    for (int e = tid; e < G * D; e += nth) {
        int h = e / D, d = e - h * D;
        float M = -INFINITY;
        for (int c = 0; c < it.nchunks; ++c) M = fmaxf(M, __ldcg(base + (size_t)c * (G * W) + h * W));
        float l = 0.f, o = 0.f;
        for (int c = 0; c < it.nchunks; ++c) {
            const float* pc = base + (size_t)c * (G * W) + h * W;
            float mc = __ldcg(pc);
            float sc = (mc == -INFINITY) ? 0.f : ex2(mc - M);
            l += __ldcg(pc + 1) * sc;
            o += __ldcg(pc + 2 + d) * sc;
        }
        store_out<D>(p, it.layer, it.b, it.g * G + h, d, o / l);
        if (d == 0 && p.lse)
            p.lse[((size_t)it.layer * p.batch + it.b) * p.num_q_heads + it.g * G + h] =
                (M + log2f(l)) * kLn2;
    }
}

// cta_part: [G][D+2] in shared memory holding this CTA's (m, l, o[D]) for the item; called by
// every thread of the CTA.
template <int D, int G>
__device__ inline void finish_item(const AttnParams& p, const Item& it, const float* cta_part,
                                   int* s_is_last)
{
    constexpr int W = D + 2;
    const int tid = threadIdx.x, nth = blockDim.x;
    const float kLn2 = 0.6931471805599453f;
    if (it.nchunks == 1) {
        for (int e = tid; e < G * D; e += nth) {
            int h = e / D, d = e - h * D;
            float l = cta_part[h * W + 1];
            store_out<D>(p, it.layer, it.b, it.g * G + h, d, cta_part[h * W + 2 + d] / l);
        }
        if (p.lse && tid < G) {
            float m = cta_part[tid * W], l = cta_part[tid * W + 1];
            p.lse[((size_t)it.layer * p.batch + it.b) * p.num_q_heads + it.g * G + tid] =
                (m + log2f(l)) * kLn2;
        }
        return;
    }
    float* slot = partial_slot(p, it, G, W);
    for (int e = tid; e < G * W; e += nth) __stcg(slot + e, cta_part[e]);
    __threadfence();
    __syncthreads();
    if (tid == 0) *s_is_last = take_ticket(p, it);
    __syncthreads();
    if (!*s_is_last) return;
    __threadfence();
    merge_chunks<D, G>(p, it, tid, nth);
}

}  // namespace oda
