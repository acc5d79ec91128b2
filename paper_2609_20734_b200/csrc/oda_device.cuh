// Shared device-side definitions of the ODA decode kernels: launch parameters, the
// per-CTA work plan (Eq. 1 ranges -> page chunks -> item list), item decoding and the
// log-sum-exp merge of split partials.  Used by both attention kernel variants.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace oda {

constexpr int kPage = 16;          // tokens per KV block
constexpr int kMaxBatch = 128;
constexpr int kMaxLayers = 256;
constexpr int kMaxClasses = 4;     // distinct (window, sinks, gated) triples in one stack
constexpr int kPartHdr = 4;        // a partial row is (m, l, -, -, o[D]): o starts 16-byte aligned

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
    float* partials;       // [max_items][G][kPartHdr + D]: m (log2 units), l, unnormalised o
    int32_t* tickets;      // [num_layers][max_batch][Hkv], zero between launches
    int32_t* status;
    const LayerInfo* layers;
    int64_t kv_layer_stride, kv_block_stride, kv_token_stride, kv_head_stride;
    int32_t layer_begin, layer_end, batch, max_batch;
    int32_t num_q_heads, num_kv_heads, max_blocks_per_seq, out_bf16;
    int32_t mode;          // 0 = Local (Eq. 1 S^L), 1 = gated Full (S^F), 2 = gated remainder S^F \ S^L,
                           //     merged into the Local result that out/lse already hold
    int32_t ncls;
    int32_t min_span_pages;  // a CTA is not given fewer pages than this (unless there are fewer)
    int32_t l2_keep_layer_end; // Local pass: pages of layers below this one are loaded with an L2 evict-last hint (0: none)
    int32_t direct_hint;     // batch-1 Local launch whose shape allows one unit per CTA (see build_plan)
    int32_t uniform_hint;    // batch-1 Local launch over layers of one class: every unit has the same length
    int32_t snap_span_pages; // launches with spans up to this long may be cut at unit boundaries (0: never)
    int32_t max_items;
    float scale_log2e;     // sm_scale * log2(e)
    int32_t cls_window[kMaxClasses], cls_sinks[kMaxClasses], cls_gated[kMaxClasses];
    int32_t cls_layers_in_call[kMaxClasses];
    int32_t allow_empty;   // gated passes: a request with seq_len 0 is skipped silently (a rank that holds none of it)
    int32_t* advance_seq_lens;  // nullable: seq_lens to increment once every CTA has read them
    int32_t* done_counter;      // zero between launches
    // Full pass of a step without a recall head: `flags` are the caller's forced flags, and the
    // CTA that finishes the plan last also publishes them as the step's decision (nullable).
    uint8_t* flags_out;
    float* scores_out;
    float* logits_out;
    int32_t* counters_out;
    // Optional per-SM weighting of the split (oda_calibrate): cum_share[v] / 65536 is the part of
    // the page axis that lies before span v; spans 2*sm and 2*sm+1 belong to SM `sm`.  nullptr =>
    // equal spans, span = blockIdx.x.
    const uint16_t* cum_share;
    int32_t* sm_claims;         // [num_sms] CTAs that have claimed a span of that SM; zero between launches
    int32_t* exit_counter;      // CTAs past their claim; zero between launches
    unsigned long long* sm_stats;  // calibration run: per SM (pages streamed, nanoseconds); else nullptr
    int32_t num_sms;
};

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start while its predecessor in the stream is still running; it must pass griddep_wait() before
// it touches memory the predecessor reads or writes.  Both are no-ops for an ordinary launch.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Loads of the small arrays a launch starts from (lengths, layer table, block-table entries), as
// volatile asm so that they are issued where they are written: early, ahead of the set-up code
// whose latency they overlap.  (An L2 evict-last hint on them was measured and changes nothing: the
// Local pass of the batch-1 benchmark shape reads 35.4 us with it and 35.4 us without.)
__device__ __forceinline__ int32_t ld_meta_s32(const int32_t* ptr)
{
    int32_t v;
    asm volatile("ld.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr));
    return v;
}

// Work decomposition.  A unit is one (layer, request, kv head); it owns np pages of KV (the
// pages of its Eq. 1 window segment, or of the whole history in Full mode; requests that are not
// flagged and layers that are not gated own none).  All units are laid end to end, layer-major
// then request then kv head, on one axis of P pages; the axis is cut into nseg <= gridDim.x spans
// and every CTA streams one span.  A span that crosses a unit boundary yields one item per unit it
// touches; a unit touched by several spans has that many partials.  By default the spans are
// equal (+-1 page): every CTA reads the same number of bytes whatever the mix of lengths and
// flags is.  SMs do not all get the same share of HBM bandwidth, though (on a B200 the streaming
// time of equal spans spreads over +-10 % and the pattern is a fixed property of the SM), so
// after a calibration run (oda_calibration_begin/end) the span lengths follow the measured rate
// of the SM the CTA runs on:
// the CTA reads %smid, claims one of that SM's two spans, and all CTAs finish together.
constexpr int kMaxGrid = 320;

struct Plan {  // shared memory, one per CTA
    int32_t pb[kMaxClasses][kMaxBatch + 1];  // exclusive prefix over requests of pages per kv head
    int32_t lb[kMaxLayers + 1];              // first axis page of each layer of the call
    int32_t seq[kMaxBatch];                  // seq_lens, clamped to the table capacity
    uint16_t kv_index[kMaxLayers];
    uint8_t cls[kMaxLayers];
    uint8_t active[kMaxBatch];               // request takes part in this launch (Full mode: flagged)
    uint16_t cum[kMaxGrid];                  // weighted split: share of the axis before span v (x 2^-16)
    int32_t weighted;                        // cum[] is in use
    int32_t my_span;                         // the span this CTA streams (-1: none)
    int32_t total_pages;
    int32_t nseg;
    int32_t snap;                            // 1: unit-aligned split, this CTA streams axis pages [x0, x1), whole units;
                                             // 2: batch 1, CTA u streams unit u (cls[0], kv_index[0] are its layer's)
    int32_t x0, x1;
    int32_t umin[kMaxClasses], umax[kMaxClasses];  // shortest / longest unit of each class (pages; 0 pages not counted)
};
static_assert(sizeof(Plan) % 8 == 0, "Plan is followed by 8-byte aligned barriers in shared memory");

struct Item {
    int32_t layer, b, g;        // layer, request, kv head
    int32_t chunk, nchunks;     // this split and how many the unit has
    int32_t slot_base;          // partial slot of the unit's chunk 0
    int32_t t;                  // seq_len
    int32_t win_pg0, win_pg1;   // logical pages of this item
    int32_t win_lo, win_hi;     // valid positions of the window/full segment: [lo, hi)
    int32_t sink_pg1;           // sink pages [0, sink_pg1) (0 = none in this item)
    int32_t sink_hi;            // valid sink positions [0, sink_hi)
    int32_t kv_layer;           // cache layer slice holding this layer's K/V
};

// Eq. 1 in 0-based form.  Local: sinks [0, min(s,t)), window [max(0,t-w), t); when they touch
// or overlap the set is the single range [0, t).  Full: [0, t).  Remainder (mode 2): the gap
// [min(s,t), max(0,t-w)) between sinks and window, empty when Local already covers everything.
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
    } else if (mode == 2) {
        const int s_eff = s < t ? s : t;
        const int lo = t - w > 0 ? t - w : 0;
        r.lo = s_eff;
        r.hi = lo > s_eff ? lo : s_eff;  // empty when the window reaches the sinks
        r.pg0 = r.lo / kPage;
        r.pg1 = r.hi > r.lo ? (r.hi + kPage - 1) / kPage : r.pg0;
        return r;
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
// Shape test of the unit-aligned split (one CTA streams a whole unit and writes its rows: no partials, no
// merge): units between one and four spans long -- shorter ones would double up on some CTAs -- and not so
// long that a CTA alone on its unit takes longer than the equal split would.  Measured: a CTA streams a page
// (K and V of 16 positions of one head) in about 0.18 us, a DRAM-bound launch as a whole moves one in 0.0012 us,
// and the equal split costs about 5 us of partials and merges: 0.18 umax <= 0.0012 total + 5, in integers.
__device__ __forceinline__ bool unit_aligned_shape(long long total, int umin, int umax, int nseg)
{
    return (long long)umin * nseg >= total && (long long)umax * nseg <= 4 * total && 150ll * umax <= total + 4200;
}

__device__ inline void build_plan(const AttnParams& p, Plan& pl)
{
    const int tid = threadIdx.x, nth = blockDim.x;
    const int B = p.batch;
    const int nl = p.layer_end - p.layer_begin;
    // Batch 1, Local pass, unit-aligned split: with one request every unit of a layer class has the
    // same length, so whether the launch falls under the unit-aligned rule (see below) follows from
    // the one length alone, and then CTA u simply takes unit u = (layer u / H, kv head u % H).  No
    // scans, no claims, one barrier: this is the latency-critical launch of batch-1 decoding.
    if (p.direct_hint && !p.sm_stats) {  // host side of the rule: mode 0, batch 1, units <= CTAs <= 4 units
        const int g = (int)gridDim.x, H = p.num_kv_heads;
        const int t = p.seq_lens[0];
        LayerInfo li;
        li.cls = li.kv_index = 0;
        if (tid == 0) li = p.layers[p.layer_begin + min((int)blockIdx.x / H, nl - 1)];
        long long total = 0;
        int umin = 0x7fffffff, umax = 0;
        if (t >= 1 && t <= p.max_blocks_per_seq * kPage) {  // anything else is the general path's to report
            for (int c = 0; c < p.ncls; ++c) {
                if (p.cls_layers_in_call[c] <= 0) continue;
                const Ranges r = eq1_ranges(0, t, p.cls_window[c], p.cls_sinks[c]);
                const int np = r.pg1 - r.pg0;
                total += (long long)p.cls_layers_in_call[c] * H * np;
                umin = min(umin, np);
                umax = max(umax, np);
            }
        }
        const int minS = p.min_span_pages > 0 ? p.min_span_pages : 1;
        if (total >= (long long)g * minS && total <= (long long)p.snap_span_pages * g && unit_aligned_shape(total, umin, umax, g)) {
            if (tid == 0) {
                pl.snap = 2;
                pl.weighted = 0;
                pl.nseg = g;
                pl.total_pages = (int32_t)total;
                pl.my_span = (int)blockIdx.x < nl * H ? (int)blockIdx.x : -1;
                pl.x0 = 0;
                pl.x1 = 1;
                pl.seq[0] = t;
                pl.active[0] = 1;
                pl.cls[0] = (uint8_t)li.cls;          // of this CTA's layer
                pl.kv_index[0] = (uint16_t)li.kv_index;
            }
            __syncthreads();
            return;
        }
    }
    // weighted split: claim one of the two spans of the SM this CTA runs on (answer used at the end)
    const bool weighted = p.cum_share != nullptr && (int)gridDim.x == 2 * p.num_sms && (int)gridDim.x <= kMaxGrid;
    int claim_sm = 0, claim_slot = 0;
    if (weighted && tid == 0) {
        asm volatile("mov.u32 %0, %%smid;" : "=r"(claim_sm));
        if (claim_sm >= p.num_sms) claim_sm = p.num_sms - 1;
        claim_slot = atomicAdd(p.sm_claims + claim_sm, 1);
    }
    uint16_t cum0 = 0, cum1 = 0;
    if (weighted) {
        if (tid < (int)gridDim.x) cum0 = p.cum_share[tid];
        if (tid + nth < (int)gridDim.x) cum1 = p.cum_share[tid + nth];
    }
    // issue every global load of the plan before using any of them: one memory latency, not three
    const bool has_b = tid < B;  // blockDim.x >= kMaxBatch
    const int t_raw = has_b ? p.seq_lens[tid] : 1;
    const int fl_raw = (has_b && p.mode != 0) ? p.flags[tid] : 1;
    LayerInfo li0, li1;
    li0.cls = li0.kv_index = li1.cls = li1.kv_index = 0;
    if (tid < nl) li0 = p.layers[p.layer_begin + tid];
    if (tid + nth < nl) li1 = p.layers[p.layer_begin + tid + nth];
    if (has_b) {
        int t = t_raw;
        if (t > p.max_blocks_per_seq * kPage) {
            t = p.max_blocks_per_seq * kPage;
            atomicOr(p.status, kStatusBadSeqLen);
        }
        pl.seq[tid] = t;
        pl.active[tid] = fl_raw != 0;
    }
    if (tid < nl) { pl.cls[tid] = (uint8_t)li0.cls; pl.kv_index[tid] = (uint16_t)li0.kv_index; }
    if (tid + nth < nl) { pl.cls[tid + nth] = (uint8_t)li1.cls; pl.kv_index[tid + nth] = (uint16_t)li1.kv_index; }
    if (weighted) {
        if (tid < (int)gridDim.x) pl.cum[tid] = cum0;
        if (tid + nth < (int)gridDim.x) pl.cum[tid + nth] = cum1;
    }
    __syncthreads();
    const int warp = tid >> 5, lane = tid & 31, nwarps = nth >> 5;
    for (int c = warp; c < p.ncls; c += nwarps) {  // one warp scans one class
        int carry = 0;
        int umin = 0x7fffffff, umax = 0;
        for (int b0 = 0; b0 < B; b0 += 32) {
            const int b = b0 + lane;
            int np = 0;
            if (b < B && p.cls_layers_in_call[c] > 0 && (p.mode == 0 || (p.cls_gated[c] && pl.active[b]))) {  // modes 1 and 2 are gated
                const int t = pl.seq[b];
                if (t < 1) {
                    if (!(t == 0 && p.allow_empty && p.mode != 0)) atomicOr(p.status, kStatusBadSeqLen);
                } else {
                    Ranges r = eq1_ranges(p.mode, t, p.cls_window[c], p.cls_sinks[c]);
                    np = r.pg1 - r.pg0;
                }
            }
            if (np > 0) { umin = min(umin, np); umax = max(umax, np); }
            int x = np;
            for (int o = 1; o < 32; o <<= 1) {
                int y = __shfl_up_sync(0xffffffffu, x, o);
                if (lane >= o) x += y;
            }
            if (b < B) pl.pb[c][b + 1] = carry + x;
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        umin = __reduce_min_sync(0xffffffffu, umin);
        umax = __reduce_max_sync(0xffffffffu, umax);
        if (lane == 0) {
            pl.pb[c][0] = 0;
            pl.umin[c] = umin;
            pl.umax[c] = umax;
        }
    }
    __syncthreads();
    if (tid < 32) {  // exclusive scan over the layers of the call
        long long carry = 0;
        for (int i0 = 0; i0 < nl; i0 += 32) {
            const int i = i0 + lane;
            long long x = i < nl ? (long long)p.num_kv_heads * pl.pb[pl.cls[i]][B] : 0;
            const long long own = x;
            for (int o = 1; o < 32; o <<= 1) {
                long long y = __shfl_up_sync(0xffffffffu, x, o);
                if (lane >= o) x += y;
            }
            if (i < nl) pl.lb[i] = (int32_t)(carry + x - own);
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        int span = -1, nseg = 0;
        if (lane == 0) {
            if (carry > 0x7fffffffll) {  // beyond the 32-bit page axis: refuse rather than wrap
                atomicOr(p.status, kStatusItemOverflow);
                carry = 0;
            }
            pl.lb[nl] = (int32_t)carry;
            pl.total_pages = (int32_t)carry;
            const int g = (int)gridDim.x;
            const int minS = p.min_span_pages > 0 ? p.min_span_pages : 1;
            long long n = g;  // the usual case, without the division
            // (rounded down: a launch of 17 pages is one span, not two of eight and a half with a merge
            // between them, and units of 65 pages on spans of 16 are cut at their own boundaries)
            if (carry < (long long)g * minS) n = carry > 0 ? max(1ll, carry / minS) : 0;
            nseg = (int)n;
            pl.nseg = nseg;
            // the weighted split needs every CTA to have real work; small launches stay equal
            pl.weighted = weighted && n == g;
            pl.snap = 0;
            span = (int)blockIdx.x;
            if (pl.weighted) {
                span = -1;
                if (claim_slot < 2) {
                    span = 2 * claim_sm + claim_slot;
                } else {
                    // more than two CTAs landed on this SM (not expected with two resident CTAs per
                    // SM): take any span that is still free
                    for (int k = 1; k < p.num_sms && span < 0; ++k) {
                        const int sm = (claim_sm + k) % p.num_sms;
                        const int slot = atomicAdd(p.sm_claims + sm, 1);
                        if (slot < 2) span = 2 * sm + slot;
                    }
                }
            }
            if (span >= nseg) span = -1;
            pl.my_span = span;
        }
        // Unit-aligned split.  A short launch whose units (one request's pages of one kv head of
        // one layer) are about as long as a span is cut at unit boundaries instead: each unit is
        // streamed by one CTA, which writes the unit's rows itself -- no partials, tickets or
        // merge at the end, where a launch of a few tens of microseconds notices them.  Some CTAs
        // get no unit; such a launch is bound by DRAM, not by the number of streaming CTAs.  Not
        // during calibration (which measures the equal split), and not when units are shorter than
        // a span (some CTAs would get two: measured 4-6 us slower than the equal split), more than
        // four spans long, or so long that a CTA alone on its unit would be the bottleneck
        // (unit_aligned_shape).
        span = __shfl_sync(0xffffffffu, span, 0);
        nseg = __shfl_sync(0xffffffffu, nseg, 0);
        const int total = (int)__shfl_sync(0xffffffffu, (int)carry, 0);
        if (p.snap_span_pages > 0 && !p.sm_stats && span >= 0 && nseg == (int)gridDim.x && total > 0 &&
            total <= p.snap_span_pages * nseg) {
            int umin = 0x7fffffff, umax = 0;
            for (int c = 0; c < p.ncls; ++c) {
                umin = min(umin, pl.umin[c]);
                umax = max(umax, pl.umax[c]);
            }
            if (unit_aligned_shape(total, umin, umax, nseg)) {
                __syncwarp();  // lb[] was written by other lanes of this warp
                int x = 0;
                const int j = span + lane;  // lane 0: where the span starts, lane 1: where it ends
                if (lane < 2) {
                    x = j >= nseg ? total : (j * total) / nseg;
                    if (j > 0 && j < nseg) {  // the nearer end of the unit that holds axis page x
                        int lo = 0, hi = nl;  // last layer with lb <= x
                        while (hi - lo > 1) {
                            const int mid = (lo + hi) >> 1;
                            if (pl.lb[mid] <= x) lo = mid; else hi = mid;
                        }
                        const int c = pl.cls[lo];
                        const int r = x - pl.lb[lo];
                        int blo = 0, bhi = B;  // last request with H * pb <= r
                        while (bhi - blo > 1) {
                            const int mid = (blo + bhi) >> 1;
                            if (p.num_kv_heads * pl.pb[c][mid] <= r) blo = mid; else bhi = mid;
                        }
                        const int np = pl.pb[c][blo + 1] - pl.pb[c][blo];
                        const int off = (r - p.num_kv_heads * pl.pb[c][blo]) % np;
                        x = 2 * off < np ? x - off : x - off + np;
                    }
                }
                const int x0 = __shfl_sync(0xffffffffu, x, 0), x1 = __shfl_sync(0xffffffffu, x, 1);
                if (lane == 0) {
                    pl.snap = 1;
                    pl.x0 = x0;
                    pl.x1 = x1;
                    if (x0 >= x1) pl.my_span = -1;  // no unit begins in this span
                }
            }
        }
    }
    __syncthreads();
    // Every CTA now works from its shared-memory copy of seq_lens.  If the step asked for it, the
    // CTA that gets here last moves the device-side lengths on (no CTA reads them again).
    if ((p.advance_seq_lens || p.flags_out) && tid == 0) {
        __threadfence();
        const int old = atomicAdd(p.done_counter, 1);
        if (old == (int)gridDim.x - 1) {
            *p.done_counter = 0;
            if (p.advance_seq_lens)
                for (int b = 0; b < B; ++b) p.advance_seq_lens[b] += 1;
            if (p.flags_out) {
                for (int b = 0; b < B; ++b) {
                    const uint8_t f = pl.active[b] ? 1 : 0;
                    p.flags_out[b] = f;
                    if (p.scores_out) p.scores_out[b] = 0.5f;
                    if (p.logits_out) p.logits_out[b] = 0.f;
                    if (p.counters_out) {
                        p.counters_out[2 * b] += 1;
                        p.counters_out[2 * b + 1] += f;
                    }
                }
            }
        }
    }
    // Every CTA has made its claim(s) by now; the one that notes this last re-arms the table.
    if (weighted && tid == 0) {
        __threadfence();
        const int old = atomicAdd(p.exit_counter, 1);
        if (old == (int)gridDim.x - 1) {
            *p.exit_counter = 0;
            for (int i = 0; i < p.num_sms; ++i) p.sm_claims[i] = 0;
        }
    }
}

// A gated pass in which no request is flagged has nothing to plan: every CTA finds that out from
// the flags alone and leaves; CTA 0 does the step's bookkeeping (lengths, published decision,
// counters) that the last CTA through the plan would otherwise do.  Uniform over the launch,
// since every CTA reads the same flags.
__device__ inline bool gated_pass_is_empty(const AttnParams& p)
{
    if (p.mode == 0 || p.sm_stats || !p.flags) return false;
    int f = 0;
    for (int b = threadIdx.x; b < p.batch; b += blockDim.x) f |= p.flags[b];
    if (__syncthreads_or(f)) return false;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int b = 0; b < p.batch; ++b) {
            if (p.advance_seq_lens) p.advance_seq_lens[b] += 1;
            if (p.flags_out) {
                p.flags_out[b] = 0;
                if (p.scores_out) p.scores_out[b] = 0.5f;
                if (p.logits_out) p.logits_out[b] = 0.f;
                if (p.counters_out) p.counters_out[2 * b] += 1;
            }
        }
    }
    return true;
}

// Warms L2 with the block table while the plan is being built (the table is not produced by the
// kernels of this library, so this may run before griddep_wait()).
__device__ __forceinline__ void prefetch_block_table(const AttnParams& p)
{
    const size_t bytes = (size_t)p.batch * p.max_blocks_per_seq * sizeof(int32_t);
    const size_t lines = (bytes + 127) / 128;
    if (lines > 8192) return;
    const char* base = reinterpret_cast<const char*>(p.block_table);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < lines; i += (size_t)gridDim.x * blockDim.x)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + i * 128));
    // the small arrays the plan starts from (a line that the previous kernel still rewrites is
    // updated in L2, where it is read from later)
    if (blockIdx.x == 0) {
        const int t = threadIdx.x;
        if (t * 32 < p.batch) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.seq_lens + t * 32));
        if (p.flags && t * 128 < p.batch) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.flags + t * 128));
        if (t * 4 < p.layer_end - p.layer_begin) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.layers + p.layer_begin + t * 4));
        if (p.cum_share && t < 6) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.cum_share + t * 64));
    }
}

__device__ __forceinline__ int span_begin(const Plan& pl, int j)
{
    if (j >= pl.nseg) return pl.total_pages;
    if (pl.weighted) return (int)(((long long)pl.cum[j] * pl.total_pages) >> 16);
    return (int)(((long long)j * pl.total_pages) / pl.nseg);
}
__device__ __forceinline__ void span_range(const Plan& pl, int j, int& x0, int& x1)
{
    if (pl.snap) {  // only ever asked for the CTA's own span
        x0 = pl.x0;
        x1 = pl.x1;
        return;
    }
    x0 = span_begin(pl, j);
    x1 = span_begin(pl, j + 1);
}
// the last span that begins at or before axis page x (the span that contains x)
__device__ __forceinline__ int span_of(const Plan& pl, int x)
{
    if (!pl.weighted) return (int)((((long long)x + 1) * pl.nseg - 1) / pl.total_pages);
    int lo = 0, hi = pl.nseg;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (span_begin(pl, mid) <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// span_of for a page known to lie at or before (dir < 0) / at or after (dir > 0) span j: a unit
// rarely covers more than a few spans, so a short walk from j beats the search over all spans
__device__ __forceinline__ int span_of_near(const Plan& pl, int x, int j, int dir)
{
    if (!pl.weighted) return span_of(pl, x);
    if (dir < 0) {
        for (int k = 0; k < 3; ++k) {
            if (span_begin(pl, j) <= x) return j;
            --j;
        }
        int lo = 0, hi = j + 1;  // span_begin(0) = 0 <= x
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (span_begin(pl, mid) <= x) lo = mid; else hi = mid;
        }
        return lo;
    }
    for (int k = 0; k < 3; ++k) {
        if (span_begin(pl, j + 1) > x) return j;
        ++j;
    }
    int lo = j, hi = pl.nseg;  // span_begin(nseg) = total_pages > x
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (span_begin(pl, mid) <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// Batch 1, Local pass: the whole plan in a few registers, the same in every thread of every CTA.
//   ok = 1  one unit per CTA (see build_plan): CTA u streams unit u;
//   ok = 2  layers of one class, so every unit has the same np pages: the equal split of build_plan in
//           closed form (same cut points, chunks and partial slots: same bits), without its loads,
//           scans and barriers -- what a launch over one or a few layers spends most of its time on.
struct DirectPlan {
    int32_t ok;
    int32_t t, cls, kv_index;   // ok = 1: of this CTA's layer
    int32_t np, total, nseg;    // ok = 2: pages per unit, pages on the axis, spans
};

// The rule of build_plan's batch-1 branch, evaluated from the one length.
__device__ __forceinline__ bool direct_rule(const AttnParams& p, int t)
{
    if (t < 1 || t > p.max_blocks_per_seq * kPage) return false;  // the general path reports these
    const int g = (int)gridDim.x, H = p.num_kv_heads;
    long long total = 0;
    int umin = 0x7fffffff, umax = 0;
    for (int c = 0; c < p.ncls; ++c) {
        if (p.cls_layers_in_call[c] <= 0) continue;
        const Ranges r = eq1_ranges(0, t, p.cls_window[c], p.cls_sinks[c]);
        const int np = r.pg1 - r.pg0;
        total += (long long)p.cls_layers_in_call[c] * H * np;
        umin = min(umin, np);
        umax = max(umax, np);
    }
    const int minS = p.min_span_pages > 0 ? p.min_span_pages : 1;
    return total >= (long long)g * minS && total <= (long long)p.snap_span_pages * g && unit_aligned_shape(total, umin, umax, g);
}

// ok = 2: does the launch qualify, and its three numbers.  Not when the per-SM weighted split would
// apply (a launch that fills the grid after a calibration), which needs the claims of build_plan.
__device__ __forceinline__ bool uniform_rule(const AttnParams& p, int t, DirectPlan& d)
{
    if (t < 1 || t > p.max_blocks_per_seq * kPage) return false;  // the general path reports these
    const Ranges r = eq1_ranges(0, t, p.cls_window[0], p.cls_sinks[0]);
    const int np = r.pg1 - r.pg0;
    const long long total = (long long)(p.layer_end - p.layer_begin) * p.num_kv_heads * np;
    if (np < 1 || total > 0x7fffffffll) return false;
    const int g = (int)gridDim.x;
    const int minS = p.min_span_pages > 0 ? p.min_span_pages : 1;
    long long n = g;
    if (total < (long long)g * minS) n = max(1ll, total / minS);
    if (p.cum_share != nullptr && n == g && g == 2 * p.num_sms && g <= kMaxGrid) return false;
    d.np = np;
    d.total = (int32_t)total;
    d.nseg = (int)n;
    d.t = t;
    return true;
}
__device__ __forceinline__ void uniform_span(const DirectPlan& d, int j, int& x0, int& x1)
{
    x0 = (int)(((long long)j * d.total) / d.nseg);
    x1 = j + 1 >= d.nseg ? d.total : (int)(((long long)(j + 1) * d.total) / d.nseg);
}
// the item of span j that starts at axis page x; returns the axis pages it covers
__device__ __forceinline__ int decode_item_uniform(const AttnParams& p, const DirectPlan& d, int j, int x, int x_end, Item& it)
{
    const int H = p.num_kv_heads;
    const int u = x / d.np, off = x - u * d.np;
    const int unit0 = x - off;
    const int take = min(d.np - off, x_end - x);
    // the spans that hold the unit's first and last page (equal split: span_of in closed form)
    const int j0 = (int)((((long long)unit0 + 1) * d.nseg - 1) / d.total);
    const int j1 = (int)((((long long)unit0 + d.np) * d.nseg - 1) / d.total);
    const int lo = u / H;
    const Ranges rg = eq1_ranges(0, d.t, p.cls_window[0], p.cls_sinks[0]);
    it.layer = p.layer_begin + lo;
    it.b = 0;
    it.g = u - lo * H;
    it.chunk = j - j0;
    it.nchunks = j1 - j0 + 1;
    it.slot_base = j0 + lo * H + it.g;
    it.kv_layer = __ldg(&p.layers[it.layer].kv_index);
    it.t = d.t;
    it.win_pg0 = rg.pg0 + off;
    it.win_pg1 = it.win_pg0 + take;
    it.win_lo = rg.lo;
    it.win_hi = rg.hi;
    it.sink_hi = (off == 0) ? rg.sink_hi : 0;
    it.sink_pg1 = (it.sink_hi + kPage - 1) / kPage;
    return take;
}

// Unit j = (layer j / H, kv head j % H) of the only request.
__device__ __forceinline__ void decode_item_direct(const AttnParams& p, const DirectPlan& d, int j, Item& it)
{
    const int H = p.num_kv_heads;
    const int lo = j / H;
    const Ranges rg = eq1_ranges(0, d.t, p.cls_window[d.cls], p.cls_sinks[d.cls]);
    it.layer = p.layer_begin + lo;
    it.b = 0;
    it.g = j - lo * H;
    it.chunk = 0;
    it.nchunks = 1;
    it.slot_base = 0;
    it.kv_layer = d.kv_index;
    it.t = d.t;
    it.win_pg0 = rg.pg0;
    it.win_pg1 = rg.pg1;
    it.win_lo = rg.lo;
    it.win_hi = rg.hi;
    it.sink_hi = rg.sink_hi;
    it.sink_pg1 = (it.sink_hi + kPage - 1) / kPage;
}

// The item of span j that starts at axis page x (x0 <= x < x_end of span_range(j)).
// Returns the number of axis pages it covers (>= 1).
__device__ inline int decode_item(const AttnParams& p, const Plan& pl, int j, int x, int x_end, Item& it)
{
    if (pl.snap == 2) {  // batch 1, one unit per CTA: span j is unit (layer j / H, kv head j % H)
        const int H = p.num_kv_heads;
        const int lo = j / H, c = pl.cls[0], t = pl.seq[0];
        const Ranges rg = eq1_ranges(p.mode, t, p.cls_window[c], p.cls_sinks[c]);
        it.layer = p.layer_begin + lo;
        it.b = 0;
        it.g = j - lo * H;
        it.chunk = 0;
        it.nchunks = 1;
        it.slot_base = 0;
        it.kv_layer = pl.kv_index[0];
        it.t = t;
        it.win_pg0 = rg.pg0;
        it.win_pg1 = rg.pg1;
        it.win_lo = rg.lo;
        it.win_hi = rg.hi;
        it.sink_hi = rg.sink_hi;
        it.sink_pg1 = (it.sink_hi + kPage - 1) / kPage;
        return 1;  // the span is [0, 1) on a nominal axis
    }
    const int nl = p.layer_end - p.layer_begin;
    int lo = 0, hi = nl;  // last layer with lb <= x
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (pl.lb[mid] <= x) lo = mid; else hi = mid;
    }
    const int c = pl.cls[lo];
    const int H = p.num_kv_heads;
    const int r = x - pl.lb[lo];
    int blo = 0, bhi = p.batch;  // last request with H * pb <= r
    while (bhi - blo > 1) {
        int mid = (blo + bhi) >> 1;
        if (H * pl.pb[c][mid] <= r) blo = mid; else bhi = mid;
    }
    const int np = pl.pb[c][blo + 1] - pl.pb[c][blo];
    const int r2 = r - H * pl.pb[c][blo];
    const int g = r2 / np;
    const int off = r2 - g * np;
    const int unit0 = x - off;                       // axis page where the unit starts
    const int take = min(np - off, x_end - x);
    // a unit-aligned span holds whole units: one chunk each
    const int j0 = pl.snap ? j : span_of_near(pl, unit0, j, -1);
    const int j1 = pl.snap ? j : span_of_near(pl, unit0 + np - 1, j, +1);
    it.layer = p.layer_begin + lo;
    it.b = blo;
    it.g = g;
    it.chunk = j - j0;
    it.nchunks = j1 - j0 + 1;
    // one slot per (span, unit) pair met along the axis: span index + unit index is unique
    it.slot_base = j0 + (lo * p.batch + blo) * H + g;
    it.kv_layer = pl.kv_index[lo];
    const int t = pl.seq[blo];
    it.t = t;
    Ranges rg = eq1_ranges(p.mode, t, p.cls_window[c], p.cls_sinks[c]);
    it.win_pg0 = rg.pg0 + off;
    it.win_pg1 = it.win_pg0 + take;
    it.win_lo = rg.lo;
    it.win_hi = rg.hi;
    it.sink_hi = (off == 0) ? rg.sink_hi : 0;
    it.sink_pg1 = (it.sink_hi + kPage - 1) / kPage;
    return take;
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
    constexpr int W = D + kPartHdr;
    constexpr int kBatch = 8;  // chunks whose loads are all issued before the first use
    const float kLn2 = 0.6931471805599453f;
    const float* base = p.partials + (size_t)it.slot_base * (G * W);
    for (int e = tid; e < G * (D / 4); e += nth) {
        const int h = e / (D / 4), d = (e - h * (D / 4)) * 4;
        float M = -INFINITY, l = 0.f;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c0 = 0; c0 < it.nchunks; c0 += kBatch) {  // chunk order is fixed: same bits every run
            float mc[kBatch], lc[kBatch];
            float4 oc[kBatch];
#pragma unroll
            for (int c = 0; c < kBatch; ++c) {
                if (c0 + c < it.nchunks) {
                    const float* pc = base + (size_t)(c0 + c) * (G * W) + h * W;
                    mc[c] = __ldcg(pc);
                    lc[c] = __ldcg(pc + 1);
                    oc[c] = __ldcg(reinterpret_cast<const float4*>(pc + kPartHdr + d));
                }
            }
            float Mn = M;
#pragma unroll
            for (int c = 0; c < kBatch; ++c)
                if (c0 + c < it.nchunks) Mn = fmaxf(Mn, mc[c]);
            const float mu = (Mn == -INFINITY) ? 0.f : Mn;
            const float a = ex2(M - mu);  // M = -inf -> 0
            l *= a;
            o.x *= a; o.y *= a; o.z *= a; o.w *= a;
            M = Mn;
#pragma unroll
            for (int c = 0; c < kBatch; ++c) {
                if (c0 + c < it.nchunks) {
                    const float sc = ex2(mc[c] - mu);
                    l += lc[c] * sc;
                    o.x += oc[c].x * sc; o.y += oc[c].y * sc; o.z += oc[c].z * sc; o.w += oc[c].w * sc;
                }
            }
        }
        const float inv = 1.f / l;
        const size_t idx = (((size_t)it.layer * p.batch + it.b) * p.num_q_heads + it.g * G + h) * D + d;
        if (p.out_bf16) {
            __nv_bfloat162* ob = reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(p.out) + idx);
            ob[0] = __floats2bfloat162_rn(o.x * inv, o.y * inv);
            ob[1] = __floats2bfloat162_rn(o.z * inv, o.w * inv);
        } else {
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + idx) =
                make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
        }
        if (d == 0 && p.lse)
            p.lse[((size_t)it.layer * p.batch + it.b) * p.num_q_heads + it.g * G + h] = (M + log2f(l)) * kLn2;
    }
}

// cta_part: [G][kPartHdr + D] in shared memory holding this CTA's (m, l, -, -, o[D]) for the item;
// called by every thread of the CTA.
template <int D, int G>
__device__ inline void finish_item(const AttnParams& p, const Item& it, const float* cta_part,
                                   int* s_is_last)
{
    constexpr int W = D + kPartHdr;
    const int tid = threadIdx.x, nth = blockDim.x;
    const float kLn2 = 0.6931471805599453f;
    if (it.nchunks == 1) {
        for (int e = tid; e < G * D; e += nth) {
            int h = e / D, d = e - h * D;
            float l = cta_part[h * W + 1];
            store_out<D>(p, it.layer, it.b, it.g * G + h, d, cta_part[h * W + kPartHdr + d] / l);
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
