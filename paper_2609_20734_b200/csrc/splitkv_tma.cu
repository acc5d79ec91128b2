// Split-KV paged decode attention, TMA + tensor-core variant for sm_100a.
//
// Six warps per CTA, two CTAs per SM, persistent:
//  * one producer warp walks the CTA's span of the page axis, looks up block ids a run of 32
//    pages ahead, and streams KV pages into a 96 KiB shared-memory ring with tiled TMA copies (cp.async.bulk.tensor, 128-byte swizzle,
//    completion on mbarriers); each item's q rows ride along with its first tile;
//  * four consumer warps each take one 16-token page of a tile and run the GQA group tile on the
//    tensor cores (mma.sync m16n8k16 bf16, fp32 accumulate), transposed so that every accumulator
//    register is live: S^T = K Q^T (tokens x heads), O^T += V^T P^T (head_dim x heads); online
//    softmax in fp32 registers; P split into a bf16 high and low part so the weights keep ~16 bits;
//  * one epilogue warp receives each finished item through shared memory and does everything that
//    waits on global memory -- result store, or partial store + ticket + merge of the unit's
//    partials -- so the consumers move straight on to the next item.
// The work is memory bound: the tensor cores take the dot products off the issue slots.
// Serves the Local pass (Eq. 1, S^L) and the gated Full pass (S^F) with one code path.
#include <cuda.h>

#include "oda_device.cuh"
#include "launch_ex.cuh"
#include "mbar.cuh"
#include "oda_launch.h"

namespace oda {



constexpr int kMaxStages = 6;
// a partial of the TMA variant: the epilogue warp's fragment, 9 rows of one float4 per lane
// (8 rows of O^T accumulators, 1 row of (m, l) pairs)
constexpr int kFragSlotFloats = 9 * 32 * 4;

struct EpiMeta {  // what the epilogue warp needs to know about a finished item
    int32_t layer, b, g, chunk, nchunks, slot_base, valid, pad;
};

struct Ctl {  // barriers and small hand-off slots, after the Plan in shared memory
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t efull, efree;
    int32_t abort;
    int32_t pad;
    EpiMeta meta;
    // the producer decodes every item anyway (it needs the pages); it hands the descriptor to the
    // consumers with the item's first tile, so that they do not decode it again on their critical path
    Item items[kMaxStages];
    int32_t item_take[kMaxStages];  // axis pages the item covers
};

template <int D>
struct TmaCfg {
    static constexpr int kConsumerWarps = 4;
    static constexpr int kProducerWarp = 4;
    static constexpr int kEpilogueWarp = 5;
    static constexpr int kThreads = 6 * 32;
    static constexpr int kTilePages = 4;                    // one page per consumer warp
    static constexpr int kPageBytes = kPage * D * 2;        // one tensor, one kv head
    static constexpr int kStageBytes = 2 * kTilePages * kPageBytes;  // K and V
    static constexpr int kStages = 98304 / kStageBytes;     // 96 KiB ring
    static constexpr int kQSlotBytes = 8 * D * 2;           // q of one kv-head group (up to 8 heads)
    static constexpr int kMergeBytes = 32 * 32 * 4 + 32 * 4 * 4;  // one warp's O fragment + (m, l) of two heads per lane
    static constexpr int kSmemBytes = kStages * (kStageBytes + kQSlotBytes) + kMergeBytes + (int)sizeof(Plan) + (int)sizeof(Ctl);
    static_assert(kStages <= kMaxStages, "ring deeper than the control block");
};

// ------------------------------------------------------------------ PTX helpers (mbarriers: mbar.cuh)
__device__ __forceinline__ void tma_load_page(uint32_t dst, const CUtensorMap* map, uint32_t bar, int head,
                                              int block, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;"
        ::"r"(dst), "l"(map), "r"(0), "r"(0), "r"(0), "r"(head), "r"(block), "r"(bar), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8) += A(16x16) * B(16x8), bf16 in, fp32 accumulate
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// transpose of an 8x8 matrix of 16-bit elements held as one register per lane
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(TmaCfg<128>::kConsumerWarps * 32) : "memory");
}

// ------------------------------------------------------------------ tile sequence of an item
// Both the producer and the consumers walk the same sequence: sink pages first (the item that
// starts a two-segment Local set), then the item's window / full pages, four pages per tile.
// An item's pages in the order they are streamed: its sink pages (if it has any), then its
// window / history pages, numbered 0 .. nv-1 and cut into tiles of four without regard to where
// one segment ends and the other begins.
__device__ __forceinline__ int item_pages(const Item& it) { return it.sink_pg1 + it.win_pg1 - it.win_pg0; }
__device__ __forceinline__ int item_logical_page(const Item& it, int v)
{
    return v < it.sink_pg1 ? v : it.win_pg0 + v - it.sink_pg1;
}
struct TileWalk {
    int v;         // first page (in streaming order) of the current tile
    int nv;        // pages of the item
    int npages;    // pages in the current tile (1..4; 0 when done)
    __device__ __forceinline__ void start(const Item& it)
    {
        v = 0;
        nv = item_pages(it);
        npages = min(4, nv);
    }
    __device__ __forceinline__ void next()
    {
        v += 4;
        npages = max(0, min(4, nv - v));
    }
    __device__ __forceinline__ bool done() const { return v >= nv; }
};

// Producer's view: runs of up to 32 consecutive pages (in streaming order) of one item (8 tiles), whose block
// ids are fetched with one warp-wide load well before the copies that need them are issued.
struct PageRun {
    int g, kv_layer, b, layer;
    const __nv_bfloat16* q;  // q rows of the item, copied with the first tile of the item
    int n;                   // pages in the run (1..32)
    bool first;              // first run of its item
    Item item;               // the item (meaningful in its first run)
    int take;
};

// kUniform = true: the instance launched for batch-1 Local calls over layers of one class that do not
// qualify for one unit per CTA (a call over one or a few layers): it can take its equal split in closed
// form from the one length.  The other instance does not carry that code.
template <int D, int G, bool kUniform>
__global__ void __launch_bounds__(TmaCfg<D>::kThreads, 2)
splitkv_tma_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap kmap,
                   const __grid_constant__ CUtensorMap vmap, const int blocks_per_layer)
{
    using C = TmaCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* ring = smem;                                                 // kStages * kStageBytes
    uint8_t* qring = ring + C::kStages * C::kStageBytes;                  // kStages * kQSlotBytes
    float* mbuf = reinterpret_cast<float*>(qring + C::kStages * C::kQSlotBytes);  // [32][32]
    float* mlbuf = mbuf + 32 * 32;                                        // [32][4]
    Plan& plan = *reinterpret_cast<Plan*>(mlbuf + 32 * 4);
    Ctl& ctl = *reinterpret_cast<Ctl*>(reinterpret_cast<uint8_t*>(&plan) + sizeof(Plan));
    const uint32_t full0 = smem_u32(ctl.full), empty0 = smem_u32(ctl.empty);
    const uint32_t efull = smem_u32(&ctl.efull), efree = smem_u32(&ctl.efree);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Batch-1 Local launch whose plan fits a few registers (one unit per CTA, or identical units cut
    // into equal spans): the one length -- and for the first kind this CTA's layer entry -- are read
    // ahead of the plan.  The one-unit-per-CTA launch is the first kernel of a step: its dependency wait
    // returns at once, and the loads go out before the barriers are set up, whose latency they overlap.
    // A launch over a few layers is one of a chain: its set-up runs first (it overlaps the previous
    // launch's tail), then the wait, then the load.
    const bool direct_try = p.direct_hint && !p.sm_stats;
    const bool early_try = (p.direct_hint || (kUniform && p.uniform_hint)) && !p.sm_stats;
    DirectPlan dp;
    dp.ok = dp.t = dp.cls = dp.kv_index = dp.np = dp.total = dp.nseg = 0;
    if (direct_try) {
        griddep_wait();
        const LayerInfo* lp = p.layers + p.layer_begin + min((int)blockIdx.x / p.num_kv_heads, p.layer_end - p.layer_begin - 1);
        dp.t = ld_meta_s32(p.seq_lens);
        dp.cls = ld_meta_s32(&lp->cls);
        dp.kv_index = ld_meta_s32(&lp->kv_index);
    }
    if (tid == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, C::kConsumerWarps);
        }
        mbar_init(efull, 1);
        mbar_init(efree, 1);
        ctl.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&kmap)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&vmap)) : "memory");
    }
    prefetch_block_table(p);
    if (kUniform && early_try && !direct_try) {
        griddep_wait();
        dp.t = ld_meta_s32(p.seq_lens);
    }
    __syncthreads();      // the barriers are initialised for every warp
    if (!early_try) griddep_wait();  // everything above is independent of the previous kernel in the stream
    // same registers in every thread: no barrier, no shared plan
    if (direct_try && direct_rule(p, dp.t)) dp.ok = 1;
    if constexpr (kUniform) {
        if (!dp.ok && early_try && p.uniform_hint && uniform_rule(p, dp.t, dp)) dp.ok = 2;
    }
    int span;             // the one span this CTA streams
    if (dp.ok == 1) {
        span = (int)blockIdx.x < (p.layer_end - p.layer_begin) * p.num_kv_heads ? (int)blockIdx.x : -1;
    } else if (kUniform && dp.ok == 2) {
        span = (int)blockIdx.x < dp.nseg ? (int)blockIdx.x : -1;
    } else {
        if (gated_pass_is_empty(p)) {
            griddep_launch_dependents();
            return;
        }
        build_plan(p, plan);  // ends with a barrier
        span = plan.my_span;
    }
    griddep_launch_dependents();
    volatile int* abort_flag = &ctl.abort;
    constexpr uint32_t kQBytes = G * D * 2;
    if (span < 0) return;

    if (warp == C::kProducerWarp) {
        // ============================ producer warp ============================
        const uint64_t policy_stream = 0x12F0000000000000ull;  // L2 evict-first: the KV stream is read once
        const uint64_t policy_keep = 0x14F0000000000000ull;    // L2 evict-last: windows the next step reads again
        uint32_t cnt = 0;
        bool dead = false;
        // walker over the runs of the CTA's span
        int x = 0, x_end = 1, take = 1;  // a one-unit-per-CTA span is [0, 1) on a nominal axis
        Item it;
        if (dp.ok == 1) {
            decode_item_direct(p, dp, span, it);
        } else if (kUniform && dp.ok == 2) {
            uniform_span(dp, span, x, x_end);
            take = decode_item_uniform(p, dp, span, x, x_end, it);
        } else {
            span_range(plan, span, x, x_end);
            take = decode_item(p, plan, span, x, x_end, it);
        }
        int v = 0, nv = item_pages(it);  // next page of the item in streaming order, pages it has
        bool more = true, item_first = true;
        auto fetch = [&](PageRun& r, int& blk) -> bool {  // next run and its block ids; false when the span is done
            if (!more) return false;
            r.g = it.g; r.kv_layer = it.kv_layer; r.b = it.b; r.layer = it.layer;
            r.q = p.q + (((size_t)it.layer * p.batch + it.b) * p.num_q_heads + (size_t)it.g * G) * D;
            r.n = min(32, nv - v);
            r.first = item_first;
            if (item_first) { r.item = it; r.take = take; }
            item_first = false;
            blk = lane < r.n ? __ldg(p.block_table + (size_t)it.b * p.max_blocks_per_seq + item_logical_page(it, v + lane)) : 0;
            v += r.n;
            if (v >= nv) {
                x += take;
                if (x < x_end) {
                    take = (kUniform && dp.ok == 2) ? decode_item_uniform(p, dp, span, x, x_end, it)
                                                    : decode_item(p, plan, span, x, x_end, it);
                    v = 0;
                    nv = item_pages(it);
                    item_first = true;
                } else {
                    more = false;
                }
            }
            return true;
        };
        PageRun cur, nxt;
        int blk_cur = 0, blk_nxt = 0;
        bool have = fetch(cur, blk_cur);
        while (have && !dead) {
            // the next run is decoded, and its block ids requested, once this run's first tile is on
            // its way (at the start of the span nothing may delay the first copy)
            bool have_next = false, fetched = false;
            for (int t0 = 0; t0 < cur.n; t0 += 4) {
                const int np = min(4, cur.n - t0);
                const uint32_t s = cnt % C::kStages, ph = (cnt / C::kStages) & 1;
                if (!mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag, p.status)) { dead = true; break; }
                const bool with_q = cur.first && t0 == 0;
                if (lane == 0) {
                    if (with_q) {  // visible to the consumers once the stage's barrier completes
                        ctl.items[s] = cur.item;
                        ctl.item_take[s] = cur.take;
                    }
                    mbar_expect_tx(full0 + 8 * s, (uint32_t)np * 2 * C::kPageBytes + (with_q ? kQBytes : 0u));
                }
                __syncwarp();
                const int blk = __shfl_sync(0xffffffffu, blk_cur, t0 + (lane & 3));
                if (lane < np) {
                    const uint32_t kdst = smem_u32(ring + s * C::kStageBytes + lane * C::kPageBytes);
                    const uint32_t vdst = kdst + C::kTilePages * C::kPageBytes;
                    const int bcoord = cur.kv_layer * blocks_per_layer + blk;
                    const uint64_t policy = cur.layer < p.l2_keep_layer_end ? policy_keep : policy_stream;
                    tma_load_page(kdst, &kmap, full0 + 8 * s, cur.g, bcoord, policy);
                    tma_load_page(vdst, &vmap, full0 + 8 * s, cur.g, bcoord, policy);
                } else if (lane == 4 && with_q) {
                    bulk_load(smem_u32(qring + s * C::kQSlotBytes), cur.q, kQBytes, full0 + 8 * s);
                }
                ++cnt;
                if (!fetched) {
                    have_next = fetch(nxt, blk_nxt);
                    fetched = true;
                }
            }
            cur = nxt;
            blk_cur = blk_nxt;
            have = have_next;
        }
        // Do not leave while copies may still be landing in this CTA's shared memory: wait
        // (bounded) until the consumers have released every stage that was armed.
        for (uint32_t k = 0; k < (uint32_t)C::kStages && k < cnt; ++k) {
            const uint32_t c2 = cnt - 1 - k;
            const uint32_t s = c2 % C::kStages, ph = (c2 / C::kStages) & 1;
            if (!mbar_wait(empty0 + 8 * s, ph, abort_flag, p.status)) break;
        }
        if (*abort_flag) {  // abandoned waits: give in-flight copies time to land before the CTA retires
            for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        }
        return;
    }

    if (warp == C::kEpilogueWarp) {
        // ============================ epilogue warp ============================
        // It receives each finished item in the consumers' fragment layout
        //   o[n][0..1]: d = 16n + hrow, heads qc, qc+1;  o[n][2..3]: d = 16n + 8 + hrow;
        //   ml = (m, l) of head qc, (m, l) of head qc+1,
        // and keeps partials in global memory in the same layout (one float4 per lane and row), so
        // that the CTA that completes a unit folds the other chunks into registers with coalesced
        // 128-bit loads and stores the result straight from the fragment.
        const int hrow = lane >> 2, qc = (lane & 3) * 2;
        const float kLn2 = 0.6931471805599453f;
        auto store_final = [&](const Item& it, const float (&o)[D / 16][4], const float4& ml) {
            // remainder mode: the Local lse is read by every lane of a head before any lane replaces it
            float l_old2[2] = {0.f, 0.f};
            if (p.mode == 2) {
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (qc + e < G)
                        l_old2[e] = p.lse[((size_t)it.layer * p.batch + it.b) * p.num_q_heads + it.g * G + qc + e] * 1.4426950408889634f;
            }
            __syncwarp();
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int hg = qc + e;
                if (hg >= G) continue;
                float mm = e ? ml.z : ml.x, ll = e ? ml.w : ml.y;
                const int h = it.g * G + hg;
                const size_t idx = (((size_t)it.layer * p.batch + it.b) * p.num_q_heads + h) * D + hrow;
                const size_t lidx = ((size_t)it.layer * p.batch + it.b) * p.num_q_heads + h;
                // remainder mode: out/lse hold the Local result of the same queries; fold it in as
                // one more partial of weight e^lse (value out, already normalised)
                float wa = 0.f, wb = 1.f;
                if (p.mode == 2) {
                    const float l_old = l_old2[e];  // log2 units
                    const float mu = fmaxf(l_old, mm);
                    wa = ex2(l_old - mu);
                    wb = ex2(mm - mu);
                    ll = wa + wb * ll;
                    mm = mu;
                }
                const float inv = 1.f / ll;
                if (p.out_bf16) {
                    __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(p.out) + idx;
#pragma unroll
                    for (int n = 0; n < D / 16; ++n) {
                        const float a0 = p.mode == 2 ? wa * __bfloat162float(ob[n * 16]) : 0.f;
                        const float a1 = p.mode == 2 ? wa * __bfloat162float(ob[n * 16 + 8]) : 0.f;
                        ob[n * 16] = __float2bfloat16_rn((a0 + wb * o[n][e]) * inv);
                        ob[n * 16 + 8] = __float2bfloat16_rn((a1 + wb * o[n][2 + e]) * inv);
                    }
                } else {
                    float* of = reinterpret_cast<float*>(p.out) + idx;
#pragma unroll
                    for (int n = 0; n < D / 16; ++n) {
                        const float a0 = p.mode == 2 ? wa * of[n * 16] : 0.f;
                        const float a1 = p.mode == 2 ? wa * of[n * 16 + 8] : 0.f;
                        of[n * 16] = (a0 + wb * o[n][e]) * inv;
                        of[n * 16 + 8] = (a1 + wb * o[n][2 + e]) * inv;
                    }
                }
                if (p.lse && hrow == 0) p.lse[lidx] = (mm + log2f(ll)) * kLn2;
            }
        };
        for (uint32_t k = 0;; ++k) {
            if (!mbar_wait(efull, k & 1, abort_flag, p.status)) break;
            const EpiMeta m = ctl.meta;
            if (!m.valid) break;
            float o[D / 16][4];
#pragma unroll
            for (int n = 0; n < D / 16; ++n) {
#pragma unroll
                for (int e = 0; e < 4; ++e) o[n][e] = mbuf[(4 * n + e) * 32 + lane];
            }
            const float4 ml = reinterpret_cast<const float4*>(mlbuf)[lane];  // mA, lA, mB, lB
            __syncwarp();
            if (lane == 0) mbar_arrive(efree);  // the consumers may reuse the hand-off buffer
            Item it;
            it.layer = m.layer; it.b = m.b; it.g = m.g; it.chunk = m.chunk; it.nchunks = m.nchunks;
            it.slot_base = m.slot_base;
            if (it.nchunks == 1) {
                store_final(it, o, ml);
            } else {
                float4* slots = reinterpret_cast<float4*>(p.partials) + (size_t)it.slot_base * (kFragSlotFloats / 4);
                float4* mine = slots + (size_t)it.chunk * (kFragSlotFloats / 4);
                // The partial goes out first; while it is on its way, a look at the ticket: if every other
                // chunk of the unit has already arrived (the usual case for the last item of a span: its
                // neighbour finished that unit long ago) this CTA merges straight from its registers and
                // needs neither the fence nor its own ticket (the partial it wrote is then never read).
#pragma unroll
                for (int n = 0; n < D / 16; ++n) __stcg(mine + n * 32 + lane, make_float4(o[n][0], o[n][1], o[n][2], o[n][3]));
                __stcg(mine + 8 * 32 + lane, ml);
                int last = 0;
                // (not in launches whose units are all cut alike: their chunks finish together, the look
                // would only add a round trip)
                if (!kUniform && lane == 0) {
                    int* tk = p.tickets + ((size_t)it.layer * p.max_batch + it.b) * p.num_kv_heads + it.g;
                    int seen;
                    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(tk) : "memory");
                    if (seen == it.nchunks - 1) {
                        *tk = 0;  // ready for the next launch
                        last = 1;
                    }
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (!last) {
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) last = take_ticket(p, it);
                    last = __shfl_sync(0xffffffffu, last, 0);
                }
                if (last) {
                    __threadfence();
                    // fold the chunks in index order (this CTA's own chunk comes from its registers);
                    // the next chunk is in flight while the current one is folded
                    float ro[D / 16][4], no[D / 16][4];
                    float4 rml = make_float4(0.f, 0.f, 0.f, 0.f), nml = rml;
                    auto fetch = [&](int c) {
                        if (c >= it.nchunks) return;
                        if (c == it.chunk) {
#pragma unroll
                            for (int n = 0; n < D / 16; ++n) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) no[n][e] = o[n][e];
                            }
                            nml = ml;
                        } else {
                            const float4* src = slots + (size_t)c * (kFragSlotFloats / 4);
#pragma unroll
                            for (int n = 0; n < D / 16; ++n) {
                                const float4 v = __ldcg(src + n * 32 + lane);
                                no[n][0] = v.x; no[n][1] = v.y; no[n][2] = v.z; no[n][3] = v.w;
                            }
                            nml = __ldcg(src + 8 * 32 + lane);
                        }
                    };
                    fetch(0);
#pragma unroll 1
                    for (int c = 0; c < it.nchunks; ++c) {
                        float co[D / 16][4];
#pragma unroll
                        for (int n = 0; n < D / 16; ++n) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) co[n][e] = no[n][e];
                        }
                        const float4 cml = nml;
                        fetch(c + 1);
                        if (c == 0) {
#pragma unroll
                            for (int n = 0; n < D / 16; ++n) {
#pragma unroll
                                for (int e = 0; e < 4; ++e) ro[n][e] = co[n][e];
                            }
                            rml = cml;
                        } else {
                            const float MA = fmaxf(rml.x, cml.x), MB = fmaxf(rml.z, cml.z);
                            const float muA = (MA == -INFINITY) ? 0.f : MA, muB = (MB == -INFINITY) ? 0.f : MB;
                            const float saA = ex2(rml.x - muA), sbA = ex2(cml.x - muA);
                            const float saB = ex2(rml.z - muB), sbB = ex2(cml.z - muB);
#pragma unroll
                            for (int n = 0; n < D / 16; ++n) {
                                ro[n][0] = ro[n][0] * saA + co[n][0] * sbA;
                                ro[n][1] = ro[n][1] * saB + co[n][1] * sbB;
                                ro[n][2] = ro[n][2] * saA + co[n][2] * sbA;
                                ro[n][3] = ro[n][3] * saB + co[n][3] * sbB;
                            }
                            rml = make_float4(MA, rml.y * saA + cml.y * sbA, MB, rml.w * saB + cml.w * sbB);
                        }
                    }
                    store_final(it, ro, rml);
                }
            }
        }
        return;
    }

    // ================================ consumer warps ================================
    // Transposed GQA tile: tokens in the M rows, the group's query heads in the N columns.
    //   S^T[16 tok x 8 heads] = K[16 tok x D] * Q^T[D x 8 heads]
    //   O^T[D x 8 heads]     += V^T[D x 16 tok] * P^T[16 tok x 8 heads]
    // so every accumulator register is a real (d, head) or (token, head) element.
    const int hrow = lane >> 2;          // B-fragment column: the query head whose q this lane holds
    const int qc = (lane & 3) * 2;       // accumulator columns: heads qc, qc+1; B-fragment k pair
    // ldmatrix row addresses inside one page (relative to the page base), 128-byte swizzle
    const int k_tok = (lane & 7) + (((lane >> 3) & 1) << 3), k_half = lane >> 4;
    const int v_tok = (lane & 7) + ((lane >> 4) << 3), v_sel = (lane >> 3) & 1;
    const int xr = lane & 7;
    uint32_t cnt = 0;    // tiles consumed
    uint32_t ecnt = 0;   // items handed to the epilogue warp
    bool aborted = false;

    int span_pages = 0;
    // calibration: the rate is taken over the first half of the span, while every other CTA is still
    // streaming too (a slow CTA speeds up once the fast ones have left, which would hide part of the
    // difference the weights are meant to remove)
    uint64_t t_first = 0, t_half = 0;
    int pages_done = 0, pages_half = 0;
    {
        int x = 0, x_end = 1;
        if (kUniform && dp.ok == 2) uniform_span(dp, span, x, x_end);
        else if (!dp.ok) span_range(plan, span, x, x_end);
        span_pages = x_end - x;
        while (x < x_end && !aborted) {
            Item it;
            // the item's descriptor and its Q^T fragments come with the item's first tile; heads >= G stay zero
            uint32_t qa[D / 16][2];
            {
                const uint32_t s = cnt % C::kStages, ph = (cnt / C::kStages) & 1;
                if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.status)) { aborted = true; break; }
                it = ctl.items[s];
                x += ctl.item_take[s];
                if (cnt == 0 && p.sm_stats) t_first = globaltimer_ns();
                const uint32_t* qs = reinterpret_cast<const uint32_t*>(qring + s * C::kQSlotBytes) + (hrow * D + qc) / 2;
#pragma unroll
                for (int kc = 0; kc < D / 16; ++kc) {
                    qa[kc][0] = hrow < G ? qs[kc * 8] : 0u;
                    qa[kc][1] = hrow < G ? qs[kc * 8 + 4] : 0u;
                }
            }
            float o[D / 16][4];
#pragma unroll
            for (int n = 0; n < D / 16; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
            float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;  // heads qc and qc+1

            TileWalk tw;
            uint32_t s_last = 0;  // the stage of the item's last tile: kept until the fold below is done with it
            for (tw.start(it); !tw.done();) {
                const uint32_t s = cnt % C::kStages, ph = (cnt / C::kStages) & 1;
                ++cnt;
                if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.status)) { aborted = true; break; }
                if (warp < tw.npages) {
                    const bool sink = tw.v + warp < it.sink_pg1;
                    const int pos0 = item_logical_page(it, tw.v + warp) * kPage;
                    const int vlo = sink ? 0 : it.win_lo, vhi = sink ? it.sink_hi : it.win_hi;
                    const bool edge = pos0 < vlo || pos0 + kPage > vhi;
                    const uint32_t kpage = smem_u32(ring + s * C::kStageBytes + warp * C::kPageBytes);
                    const uint32_t vpage = kpage + C::kTilePages * C::kPageBytes;
                    // ---- S^T = K Q^T for 16 tokens ----
                    float st[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int kc = 0; kc < D / 16; ++kc) {
                        const int chunk = (kc & 3) * 2 + k_half;
                        const uint32_t addr = kpage + (kc >> 2) * 2048 + k_tok * 128 + ((chunk ^ xr) << 4);
                        uint32_t a0, a1, a2, a3;
                        ldsm_x4(addr, a0, a1, a2, a3);
                        mma16816(st, a0, a1, a2, a3, qa[kc][0], qa[kc][1]);
                    }
                    // st[0],st[1]: token hrow, heads qc,qc+1;  st[2],st[3]: token hrow+8
                    float x0s = st[0] * p.scale_log2e, x1s = st[1] * p.scale_log2e;
                    float x2s = st[2] * p.scale_log2e, x3s = st[3] * p.scale_log2e;
                    uint32_t mk0 = 0xffffffffu, mk1 = 0xffffffffu;
                    if (edge) {  // positions outside [vlo, vhi) are not in the set
                        const int ta = pos0 + hrow;
                        const bool va = ta >= vlo && ta < vhi, vb = ta + 8 >= vlo && ta + 8 < vhi;
                        x0s = va ? x0s : -INFINITY; x1s = va ? x1s : -INFINITY;
                        x2s = vb ? x2s : -INFINITY; x3s = vb ? x3s : -INFINITY;
                        // V^T fragments hold tokens qc, qc+1 (and +8) in their 16-bit halves
                        const int t0 = pos0 + qc;
                        const bool v0 = t0 >= vlo && t0 < vhi, v1 = t0 + 1 >= vlo && t0 + 1 < vhi;
                        const bool v2 = t0 + 8 >= vlo && t0 + 8 < vhi, v3 = t0 + 9 >= vlo && t0 + 9 < vhi;
                        mk0 = (v0 ? 0x0000ffffu : 0u) | (v1 ? 0xffff0000u : 0u);
                        mk1 = (v2 ? 0x0000ffffu : 0u) | (v3 ? 0xffff0000u : 0u);
                    }
                    // ---- online softmax over the 16 tokens (fp32, base 2); tokens live across lanes ----
                    float mxA = fmaxf(x0s, x2s), mxB = fmaxf(x1s, x3s);
#pragma unroll
                    for (int off = 4; off < 32; off <<= 1) {
                        mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, off));
                        mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, off));
                    }
                    const float mnA = fmaxf(mA, mxA), mnB = fmaxf(mB, mxB);
                    const float muA = (mnA == -INFINITY) ? 0.f : mnA, muB = (mnB == -INFINITY) ? 0.f : mnB;
                    const float alA = ex2(mA - muA), alB = ex2(mB - muB);
                    const float p0 = ex2(x0s - muA), p1 = ex2(x1s - muB), p2 = ex2(x2s - muA), p3 = ex2(x3s - muB);
                    lA = lA * alA + (p0 + p2);
                    lB = lB * alB + (p1 + p3);
                    mA = mnA;
                    mB = mnB;
                    if (!__all_sync(0xffffffffu, alA == 1.f && alB == 1.f)) {
#pragma unroll
                        for (int n = 0; n < D / 16; ++n) { o[n][0] *= alA; o[n][1] *= alB; o[n][2] *= alA; o[n][3] *= alB; }
                    }
                    // P^T as B fragments: transpose the two 8x8 (token x head) tiles; bf16 high + low parts
                    const uint32_t hi0 = pack_bf16x2(p0, p1), hi1 = pack_bf16x2(p2, p3);
                    const uint32_t lo0 = pack_bf16x2(p0 - __uint_as_float(hi0 << 16), p1 - __uint_as_float(hi0 & 0xffff0000u));
                    const uint32_t lo1 = pack_bf16x2(p2 - __uint_as_float(hi1 << 16), p3 - __uint_as_float(hi1 & 0xffff0000u));
                    const uint32_t bh0 = movmatrix_t(hi0), bh1 = movmatrix_t(hi1);
                    const uint32_t bl0 = movmatrix_t(lo0), bl1 = movmatrix_t(lo1);
                    // ---- O^T += V^T P^T ----
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt) {
                        const int chunk = (mt & 3) * 2 + v_sel;
                        const uint32_t addr = vpage + (mt >> 2) * 2048 + v_tok * 128 + ((chunk ^ xr) << 4);
                        uint32_t a0, a1, a2, a3;
                        ldsm_x4_t(addr, a0, a1, a2, a3);
                        if (edge) {  // slots outside the set may hold anything, NaN bit patterns included
                            a0 &= mk0; a1 &= mk0; a2 &= mk1; a3 &= mk1;
                        }
                        mma16816(o[mt], a0, a1, a2, a3, bh0, bh1);
                        mma16816(o[mt], a0, a1, a2, a3, bl0, bl1);
                    }
                }
                __syncwarp();
                if (p.sm_stats) {
                    pages_done += tw.npages;
                    if (pages_half == 0 && 2 * pages_done >= span_pages) {
                        pages_half = pages_done;
                        t_half = globaltimer_ns();
                    }
                }
                tw.next();
                if (tw.done())
                    s_last = s;
                else if (lane == 0)
                    mbar_arrive(empty0 + 8 * s);
            }
            if (aborted || *abort_flag) { aborted = true; break; }

            // ---- fold the four warps' states and leave the item to the epilogue warp.  Every warp
            //      parks its fragment in its own page slot of the item's last stage (that data is
            //      dead: a warp only ever reads its own page), then each warp finishes a quarter of
            //      the rows from all four fragments, in warp order, into the hand-off buffer. ----
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                lA += __shfl_xor_sync(0xffffffffu, lA, off);
                lB += __shfl_xor_sync(0xffffffffu, lB, off);
            }
            {
                uint8_t* stage = ring + s_last * C::kStageBytes;
                float* fo = reinterpret_cast<float*>(stage + warp * C::kPageBytes);
                float4* fml = reinterpret_cast<float4*>(stage + (C::kTilePages + warp) * C::kPageBytes);
#pragma unroll
                for (int n = 0; n < D / 16; ++n) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) fo[(4 * n + e) * 32 + lane] = o[n][e];
                }
                fml[lane] = make_float4(mA, lA, mB, lB);
            }
            consumer_sync();
            {
                const uint8_t* stage = ring + s_last * C::kStageBytes;
                float4 mlf[C::kConsumerWarps];
#pragma unroll
                for (int f = 0; f < C::kConsumerWarps; ++f)
                    mlf[f] = reinterpret_cast<const float4*>(stage + (C::kTilePages + f) * C::kPageBytes)[lane];
                float MA = mlf[0].x, MB = mlf[0].z;
#pragma unroll
                for (int f = 1; f < C::kConsumerWarps; ++f) { MA = fmaxf(MA, mlf[f].x); MB = fmaxf(MB, mlf[f].z); }
                const float muA = (MA == -INFINITY) ? 0.f : MA, muB = (MB == -INFINITY) ? 0.f : MB;
                float scA[C::kConsumerWarps], scB[C::kConsumerWarps];
                float lAf = 0.f, lBf = 0.f;
#pragma unroll
                for (int f = 0; f < C::kConsumerWarps; ++f) {
                    scA[f] = ex2(mlf[f].x - muA);
                    scB[f] = ex2(mlf[f].z - muB);
                    lAf = fmaf(mlf[f].y, scA[f], lAf);
                    lBf = fmaf(mlf[f].w, scB[f], lBf);
                }
                constexpr int kRows = (D / 16) / C::kConsumerWarps;  // fragment rows this warp finishes
                float fin[kRows][4];
#pragma unroll
                for (int r = 0; r < kRows; ++r) {
                    const int n = warp * kRows + r;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float a = 0.f;
#pragma unroll
                        for (int f = 0; f < C::kConsumerWarps; ++f) {
                            const float v = reinterpret_cast<const float*>(stage + f * C::kPageBytes)[(4 * n + e) * 32 + lane];
                            a = fmaf(v, (e & 1) ? scB[f] : scA[f], a);
                        }
                        fin[r][e] = a;
                    }
                }
                // the hand-off buffer is free once the epilogue warp has taken the previous item out of it
                if (!mbar_wait(efree, (ecnt & 1) ^ 1, abort_flag, p.status)) { aborted = true; break; }
#pragma unroll
                for (int r = 0; r < kRows; ++r) {
                    const int n = warp * kRows + r;
#pragma unroll
                    for (int e = 0; e < 4; ++e) mbuf[(4 * n + e) * 32 + lane] = fin[r][e];
                }
                if (warp == 0) {
                    reinterpret_cast<float4*>(mlbuf)[lane] = make_float4(MA, lAf, MB, lBf);
                    if (lane == 0) {
                        EpiMeta m;
                        m.layer = it.layer; m.b = it.b; m.g = it.g; m.chunk = it.chunk; m.nchunks = it.nchunks;
                        m.slot_base = it.slot_base; m.valid = 1; m.pad = 0;
                        ctl.meta = m;
                    }
                }
            }
            // generic-proxy writes into the stage are ordered before the copies that will refill it
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            consumer_sync();
            if (lane == 0) {
                mbar_arrive(empty0 + 8 * s_last);
                if (warp == 0) mbar_arrive(efull);
            }
            ++ecnt;
        }
    }
    // calibration run: how long this SM took to stream how many pages
    if (p.sm_stats && tid == 0 && !aborted && pages_half > 0 && plan.nseg == (int)gridDim.x) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        if ((int)smid < p.num_sms) {
            atomicAdd(p.sm_stats + 2 * smid, (unsigned long long)pages_half);
            atomicAdd(p.sm_stats + 2 * smid + 1, (unsigned long long)(t_half - t_first));
        }
    }
    // end marker for the epilogue warp (also on the abort path, where its own waits are bounded)
    if (warp == 0) {
        if (mbar_wait(efree, (ecnt & 1) ^ 1, abort_flag, p.status)) {
            if (lane == 0) {
                ctl.meta.valid = 0;
                mbar_arrive(efull);
            }
        }
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            (void)cudaGetLastError();
    }
    return fn;
}

bool tma_variant_supported(int head_dim, int64_t layer_stride, int64_t block_stride, int num_layers_phys)
{
    if (head_dim != 64 && head_dim != 128) return false;
    if (num_layers_phys > 1 && (block_stride == 0 || layer_stride % block_stride != 0)) return false;
    return true;
}

// 5-D view of a paged cache: (d within a 64-wide slab, slot, slab, kv head, block); one box = one
// page of one head.  The block extent is a loose bound: the kernel only reads blocks that the
// block table names.
bool encode_kv_map(void* out_map, const void* base, int head_dim, int num_kv_heads, int64_t token_stride,
                   int64_t head_stride, int64_t block_stride, int64_t num_blocks_bound)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[5] = {64, (cuuint64_t)kPage, (cuuint64_t)(head_dim / 64), (cuuint64_t)num_kv_heads,
                          (cuuint64_t)num_blocks_bound};
    cuuint64_t strides[4] = {(cuuint64_t)token_stride * 2, 128, (cuuint64_t)head_stride * 2,
                             (cuuint64_t)block_stride * 2};
    cuuint32_t box[5] = {64, (cuuint32_t)kPage, (cuuint32_t)(head_dim / 64), 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(reinterpret_cast<CUtensorMap*>(out_map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5,
                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int D, int G>
static cudaError_t launch_tma_t(const AttnParams& p, const void* kmap, const void* vmap, int blocks_per_layer,
                                int grid, cudaStream_t st, bool pdl)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(splitkv_tma_kernel<D, G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             TmaCfg<D>::kSmemBytes);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(splitkv_tma_kernel<D, G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     TmaCfg<D>::kSmemBytes);
        if (e != cudaSuccess) return e;
        (void)cudaFuncSetAttribute(splitkv_tma_kernel<D, G, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                   cudaSharedmemCarveoutMaxShared);
        (void)cudaFuncSetAttribute(splitkv_tma_kernel<D, G, true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                   cudaSharedmemCarveoutMaxShared);
        attr_set = true;
    }
    if (p.uniform_hint && !p.direct_hint)
        return launch_ex(splitkv_tma_kernel<D, G, true>, dim3(grid), dim3(TmaCfg<D>::kThreads), TmaCfg<D>::kSmemBytes, st,
                         pdl, p, *reinterpret_cast<const CUtensorMap*>(kmap), *reinterpret_cast<const CUtensorMap*>(vmap),
                         blocks_per_layer);
    return launch_ex(splitkv_tma_kernel<D, G, false>, dim3(grid), dim3(TmaCfg<D>::kThreads), TmaCfg<D>::kSmemBytes, st, pdl,
                     p, *reinterpret_cast<const CUtensorMap*>(kmap), *reinterpret_cast<const CUtensorMap*>(vmap),
                     blocks_per_layer);
}

template <int D, int G>
static int occupancy_tma_t()
{
    int n = 0;
    if (cudaFuncSetAttribute(splitkv_tma_kernel<D, G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TmaCfg<D>::kSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    (void)cudaFuncSetAttribute(splitkv_tma_kernel<D, G, false>, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, splitkv_tma_kernel<D, G, false>, TmaCfg<D>::kThreads,
                                                  TmaCfg<D>::kSmemBytes);
    return n;
}

#define ODA_DISPATCH_DG(D_, G_, EXPR)                                                  \
    do {                                                                               \
        if (D_ == 128) {                                                               \
            if (G_ == 1) { constexpr int DD = 128, GG = 1; EXPR; }                     \
            else if (G_ == 2) { constexpr int DD = 128, GG = 2; EXPR; }                \
            else if (G_ == 4) { constexpr int DD = 128, GG = 4; EXPR; }                \
            else if (G_ == 8) { constexpr int DD = 128, GG = 8; EXPR; }                \
        } else if (D_ == 64) {                                                         \
            if (G_ == 1) { constexpr int DD = 64, GG = 1; EXPR; }                      \
            else if (G_ == 2) { constexpr int DD = 64, GG = 2; EXPR; }                 \
            else if (G_ == 4) { constexpr int DD = 64, GG = 4; EXPR; }                 \
            else if (G_ == 8) { constexpr int DD = 64, GG = 8; EXPR; }                 \
        }                                                                              \
    } while (0)

cudaError_t launch_splitkv_tma(const AttnParams& p, const void* kmap, const void* vmap, int blocks_per_layer,
                               int head_dim, int group, int grid, cudaStream_t st, bool pdl)
{
    cudaError_t e = cudaErrorInvalidValue;
    ODA_DISPATCH_DG(head_dim, group, e = (launch_tma_t<DD, GG>(p, kmap, vmap, blocks_per_layer, grid, st, pdl)));
    return e;
}

int tma_partial_slot_floats() { return kFragSlotFloats; }

int occupancy_splitkv_tma(int head_dim, int group)
{
    int n = 0;
    ODA_DISPATCH_DG(head_dim, group, n = (occupancy_tma_t<DD, GG>()));
    return n;
}

}  // namespace oda
