// Split-KV paged decode attention, TMA + tensor-core variant for sm_100a.
//
// One producer warp streams KV pages from the paged cache into a shared-memory ring with
// tiled TMA copies (cp.async.bulk.tensor, 128-byte swizzle, completion on mbarriers); four
// consumer warps each take one 16-token page of a tile and run the GQA group tile on the
// tensor cores (mma.sync m16n8k16 bf16, fp32 accumulate): S = Q K^T with the group's query
// heads in the M rows, online softmax in fp32 registers, O += P V with P split into a bf16
// high and low part so that the softmax weights keep ~16 bits.  The work is memory bound:
// the tensor cores are there to take the dot products off the issue slots, not for flops.
// Serves the Local pass (Eq. 1, S^L) and the gated Full pass (S^F) with one code path.
#include <cuda.h>

#include "oda_device.cuh"
#include "oda_launch.h"

namespace oda {

constexpr int kStatusWaitTimeout = 4;

template <int D>
struct TmaCfg {
    static constexpr int kConsumerWarps = 4;
    static constexpr int kThreads = (kConsumerWarps + 1) * 32;
    static constexpr int kTilePages = 4;                    // one page per consumer warp
    static constexpr int kPageBytes = kPage * D * 2;        // one tensor, one kv head
    static constexpr int kSlabs = D / 64;                   // 128-byte-row slabs per page
    static constexpr int kStageBytes = 2 * kTilePages * kPageBytes;  // K and V
    static constexpr int kStages = 98304 / kStageBytes;     // 96 KiB ring
    static constexpr int kMergeBytes = 2 * 32 * 32 * 4 + 2 * 32 * 2 * 4;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kMergeBytes + (int)sizeof(Plan) + 256;
};

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t globaltimer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after ~2 s, records it in the status word and raises the CTA's abort
// flag, so a lost completion can never hang the GPU.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 1023u) == 0) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > 2000000000ull) {
                *abort_flag = 1;
                atomicOr(status, kStatusWaitTimeout);
                return false;
            }
        }
    }
    return true;
}

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
// D = A(16x16, rows 8..15 zero) * B(16x8) + D, bf16 in, fp32 accumulate
__device__ __forceinline__ void mma_top(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
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
// Both the producer and the consumers walk the same sequence: sink pages first (chunk 0 of a
// two-segment Local set), then the chunk's window / full pages, four pages per tile.
struct TileWalk {
    int seg;       // 0 = sinks, 1 = window/full, 2 = done
    int pg;        // first logical page of the current tile
    int npages;    // pages in the current tile (1..4)
    __device__ __forceinline__ void start(const Item& it)
    {
        seg = it.sink_pg1 > 0 ? 0 : 1;
        pg = seg ? it.win_pg0 : 0;
        settle(it);
    }
    __device__ __forceinline__ void settle(const Item& it)
    {
        int end = seg == 0 ? it.sink_pg1 : it.win_pg1;
        if (seg == 0 && pg >= end) { seg = 1; pg = it.win_pg0; end = it.win_pg1; }
        if (seg == 1 && pg >= end) { seg = 2; npages = 0; return; }
        npages = min(4, end - pg);
    }
    __device__ __forceinline__ void next(const Item& it) { pg += 4; settle(it); }
    __device__ __forceinline__ bool done() const { return seg == 2; }
};

template <int D, int G>
__global__ void __maxnreg__(200)
splitkv_tma_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap kmap,
                   const __grid_constant__ CUtensorMap vmap, const int blocks_per_layer)
{
    using C = TmaCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* ring = smem;                                           // kStages * kStageBytes
    float* mbuf = reinterpret_cast<float*>(ring + C::kStages * C::kStageBytes);   // [2][32][32]
    float* mlbuf = mbuf + 2 * 32 * 32;                              // [2][32][2]
    Plan& plan = *reinterpret_cast<Plan*>(mlbuf + 2 * 32 * 2);
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(&plan) + ((sizeof(Plan) + 15) & ~size_t(15)));
    int* s_flags = reinterpret_cast<int*>(bars + 2 * C::kStages);   // [0] abort, [1] is_last
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + C::kStages);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, C::kConsumerWarps);
        }
        s_flags[0] = 0;
        s_flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    build_plan(p, plan);  // ends with __syncthreads()
    volatile int* abort_flag = s_flags;
    const int total = plan.total_items;

    if (warp == C::kConsumerWarps) {
        // ============================ producer warp ============================
        const uint64_t policy = 0x12F0000000000000ull;  // L2 evict-first: the KV stream is read once
        uint32_t cnt = 0;
        int id = blockIdx.x;
        Item it;
        TileWalk tw;
        int blk = 0;
        bool have = id < total;
        if (have) {
            it = decode_item(p, plan, id);
            tw.start(it);
            if (lane < tw.npages) blk = __ldg(p.block_table + (size_t)it.b * p.max_blocks_per_seq + tw.pg + lane);
        }
        while (have) {
            // current tile: (it, tw, blk).  Look up the next tile's pages before blocking.
            const Item cur_it = it;
            const int cur_np = tw.npages, cur_blk = blk;
            const int kv_layer = p.layers[cur_it.layer].kv_index;
            tw.next(it);
            if (tw.done()) {
                id += gridDim.x;
                have = id < total;
                if (have) {
                    it = decode_item(p, plan, id);
                    tw.start(it);
                }
            }
            if (have && lane < tw.npages)
                blk = __ldg(p.block_table + (size_t)it.b * p.max_blocks_per_seq + tw.pg + lane);
            const uint32_t s = cnt % C::kStages, ph = (cnt / C::kStages) & 1;
            if (!mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag, p.status)) break;
            if (lane == 0) mbar_expect_tx(full0 + 8 * s, (uint32_t)cur_np * 2 * C::kPageBytes);
            __syncwarp();
            if (lane < cur_np) {
                const uint32_t kdst = smem_u32(ring + s * C::kStageBytes + lane * C::kPageBytes);
                const uint32_t vdst = kdst + C::kTilePages * C::kPageBytes;
                const int bcoord = kv_layer * blocks_per_layer + cur_blk;
                tma_load_page(kdst, &kmap, full0 + 8 * s, cur_it.g, bcoord, policy);
                tma_load_page(vdst, &vmap, full0 + 8 * s, cur_it.g, bcoord, policy);
            }
            ++cnt;
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

    // ================================ consumer warps ================================
    const int row = lane >> 2;           // query head within the group (M row of the fragment)
    const int qc = (lane & 3) * 2;       // column pair inside an 8-wide fragment
    // ldmatrix row addresses inside one page (relative to the page base), 128-byte swizzle
    const int k_tok = (lane & 7) + ((lane >> 4) << 3), k_half = (lane >> 3) & 1;
    const int v_tok = (lane & 7) + (((lane >> 3) & 1) << 3), v_sel = lane >> 4;
    const int xr = lane & 7;
    uint32_t cnt = 0;

    for (int id = blockIdx.x; id < total; id += gridDim.x) {
        const Item it = decode_item(p, plan, id);
        // Q fragments: rows >= G stay zero
        uint32_t qa[D / 16][2];
        {
            const __nv_bfloat16* qb =
                p.q + (((size_t)it.layer * p.batch + it.b) * p.num_q_heads + (size_t)it.g * G + row) * D + qc;
#pragma unroll
            for (int kc = 0; kc < D / 16; ++kc) {
                qa[kc][0] = row < G ? __ldg(reinterpret_cast<const unsigned int*>(qb + kc * 16)) : 0u;
                qa[kc][1] = row < G ? __ldg(reinterpret_cast<const unsigned int*>(qb + kc * 16 + 8)) : 0u;
            }
        }
        float o[D / 8][4];
#pragma unroll
        for (int n = 0; n < D / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;

        TileWalk tw;
        bool aborted = false;
        for (tw.start(it); !tw.done(); tw.next(it)) {
            const uint32_t s = cnt % C::kStages, ph = (cnt / C::kStages) & 1;
            ++cnt;
            if (!mbar_wait(full0 + 8 * s, ph, abort_flag, p.status)) { aborted = true; break; }
            if (warp < tw.npages) {
                const int pos0 = (tw.pg + warp) * kPage;
                const int vlo = tw.seg ? it.win_lo : 0, vhi = tw.seg ? it.win_hi : it.sink_hi;
                const bool edge = pos0 < vlo || pos0 + kPage > vhi;
                const uint32_t kpage = smem_u32(ring + s * C::kStageBytes + warp * C::kPageBytes);
                const uint32_t vpage = kpage + C::kTilePages * C::kPageBytes;
                // ---- S = Q K^T for 16 tokens: two n-tiles of 8 ----
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int kc = 0; kc < D / 16; ++kc) {
                    const int chunk = (kc & 3) * 2 + k_half;
                    const uint32_t addr = kpage + (kc >> 2) * 2048 + k_tok * 128 + ((chunk ^ xr) << 4);
                    uint32_t r0, r1, r2, r3;
                    ldsm_x4(addr, r0, r1, r2, r3);
                    mma_top(s0, qa[kc][0], qa[kc][1], r0, r1);
                    mma_top(s1, qa[kc][0], qa[kc][1], r2, r3);
                }
                float x0 = s0[0] * p.scale_log2e, x1 = s0[1] * p.scale_log2e;
                float x2 = s1[0] * p.scale_log2e, x3 = s1[1] * p.scale_log2e;
                uint32_t mk0 = 0xffffffffu, mk1 = 0xffffffffu;
                if (edge) {  // positions outside [vlo, vhi) are not in the set
                    const int t0 = pos0 + qc;
                    const bool v0 = t0 >= vlo && t0 < vhi, v1 = t0 + 1 >= vlo && t0 + 1 < vhi;
                    const bool v2 = t0 + 8 >= vlo && t0 + 8 < vhi, v3 = t0 + 9 >= vlo && t0 + 9 < vhi;
                    x0 = v0 ? x0 : -INFINITY; x1 = v1 ? x1 : -INFINITY;
                    x2 = v2 ? x2 : -INFINITY; x3 = v3 ? x3 : -INFINITY;
                    mk0 = (v0 ? 0x0000ffffu : 0u) | (v1 ? 0xffff0000u : 0u);
                    mk1 = (v2 ? 0x0000ffffu : 0u) | (v3 ? 0xffff0000u : 0u);
                }
                // ---- online softmax (fp32, base 2) ----
                float mx = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                const float mu = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = ex2(m_run - mu);
                const float p0 = ex2(x0 - mu), p1 = ex2(x1 - mu), p2 = ex2(x2 - mu), p3 = ex2(x3 - mu);
                l_run = l_run * alpha + ((p0 + p1) + (p2 + p3));
                m_run = m_new;
                if (!__all_sync(0xffffffffu, alpha == 1.f)) {
#pragma unroll
                    for (int n = 0; n < D / 8; ++n) { o[n][0] *= alpha; o[n][1] *= alpha; }
                }
                // P as A fragments, split into bf16 high and low parts
                const uint32_t ph0 = pack_bf16x2(p0, p1), ph1 = pack_bf16x2(p2, p3);
                const uint32_t pl0 = pack_bf16x2(p0 - __uint_as_float(ph0 << 16), p1 - __uint_as_float(ph0 & 0xffff0000u));
                const uint32_t pl1 = pack_bf16x2(p2 - __uint_as_float(ph1 << 16), p3 - __uint_as_float(ph1 & 0xffff0000u));
                // ---- O += P V ----
#pragma unroll
                for (int np = 0; np < D / 16; ++np) {
                    const int chunk = (np & 3) * 2 + v_sel;
                    const uint32_t addr = vpage + (np >> 2) * 2048 + v_tok * 128 + ((chunk ^ xr) << 4);
                    uint32_t r0, r1, r2, r3;
                    ldsm_x4_t(addr, r0, r1, r2, r3);
                    if (edge) {  // slots outside the set may hold anything, NaN bit patterns included
                        r0 &= mk0; r1 &= mk1; r2 &= mk0; r3 &= mk1;
                    }
                    mma_top(o[2 * np], ph0, ph1, r0, r1);
                    mma_top(o[2 * np], pl0, pl1, r0, r1);
                    mma_top(o[2 * np + 1], ph0, ph1, r2, r3);
                    mma_top(o[2 * np + 1], pl0, pl1, r2, r3);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * s);
        }
        if (aborted || *abort_flag) break;

        // ---- merge the four warps' streams pairwise through shared memory (same fragment layout) ----
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
#pragma unroll
        for (int round = 0; round < 2; ++round) {
            const int nsend = round == 0 ? 2 : 1;  // round 0: warps 2,3 -> 0,1; round 1: warp 1 -> 0
            if (warp >= nsend && warp < 2 * nsend) {
                float* dst = mbuf + (warp - nsend) * 32 * 32;
#pragma unroll
                for (int n = 0; n < D / 8; ++n) {
                    dst[(2 * n) * 32 + lane] = o[n][0];
                    dst[(2 * n + 1) * 32 + lane] = o[n][1];
                }
                mlbuf[((warp - nsend) * 32 + lane) * 2] = m_run;
                mlbuf[((warp - nsend) * 32 + lane) * 2 + 1] = l_run;
            }
            consumer_sync();
            if (warp < nsend) {
                const float* src = mbuf + warp * 32 * 32;
                const float m2 = mlbuf[(warp * 32 + lane) * 2], l2 = mlbuf[(warp * 32 + lane) * 2 + 1];
                const float M = fmaxf(m_run, m2);
                const float mu = (M == -INFINITY) ? 0.f : M;
                const float sa = ex2(m_run - mu), sb = ex2(m2 - mu);
#pragma unroll
                for (int n = 0; n < D / 8; ++n) {
                    o[n][0] = o[n][0] * sa + src[(2 * n) * 32 + lane] * sb;
                    o[n][1] = o[n][1] * sa + src[(2 * n + 1) * 32 + lane] * sb;
                }
                l_run = l_run * sa + l2 * sb;
                m_run = M;
            }
            consumer_sync();
        }
        // ---- warp 0 holds the CTA's (m, l, o): store the result or publish the partial ----
        constexpr int W = D + 2;
        const float kLn2 = 0.6931471805599453f;
        if (it.nchunks == 1) {
            if (warp == 0 && row < G) {
                const float inv = 1.f / l_run;
                const int h = it.g * G + row;
                const size_t idx = (((size_t)it.layer * p.batch + it.b) * p.num_q_heads + h) * D + qc;
                if (p.out_bf16) {
                    uint32_t* ob = reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(p.out) + idx);
#pragma unroll
                    for (int n = 0; n < D / 8; ++n) ob[n * 4] = pack_bf16x2(o[n][0] * inv, o[n][1] * inv);
                } else {
                    float2* of = reinterpret_cast<float2*>(reinterpret_cast<float*>(p.out) + idx);
#pragma unroll
                    for (int n = 0; n < D / 8; ++n) of[n * 4] = make_float2(o[n][0] * inv, o[n][1] * inv);
                }
                if (p.lse && (lane & 3) == 0)
                    p.lse[((size_t)it.layer * p.batch + it.b) * p.num_q_heads + h] = (m_run + log2f(l_run)) * kLn2;
            }
        } else {
            if (warp == 0 && row < G) {
                float* slot = partial_slot(p, it, G, W) + row * W;
                if ((lane & 3) == 0) {
                    __stcg(slot, m_run);
                    __stcg(slot + 1, l_run);
                }
#pragma unroll
                for (int n = 0; n < D / 8; ++n)
                    __stcg(reinterpret_cast<float2*>(slot + 2 + n * 8 + qc), make_float2(o[n][0], o[n][1]));
            }
            __threadfence();
            consumer_sync();
            if (tid == 0) s_flags[1] = take_ticket(p, it);
            consumer_sync();
            if (s_flags[1]) {
                __threadfence();
                merge_chunks<D, G>(p, it, tid, C::kConsumerWarps * 32);
            }
            consumer_sync();  // s_flags[1] is reused by the next item
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
                                int grid, cudaStream_t st)
{
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(splitkv_tma_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             TmaCfg<D>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    splitkv_tma_kernel<D, G><<<grid, TmaCfg<D>::kThreads, TmaCfg<D>::kSmemBytes, st>>>(
        p, *reinterpret_cast<const CUtensorMap*>(kmap), *reinterpret_cast<const CUtensorMap*>(vmap),
        blocks_per_layer);
    return cudaGetLastError();
}

template <int D, int G>
static int occupancy_tma_t()
{
    int n = 0;
    if (cudaFuncSetAttribute(splitkv_tma_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             TmaCfg<D>::kSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, splitkv_tma_kernel<D, G>, TmaCfg<D>::kThreads,
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
                               int head_dim, int group, int grid, cudaStream_t st)
{
    cudaError_t e = cudaErrorInvalidValue;
    ODA_DISPATCH_DG(head_dim, group, e = (launch_tma_t<DD, GG>(p, kmap, vmap, blocks_per_layer, grid, st)));
    return e;
}

int occupancy_splitkv_tma(int head_dim, int group)
{
    int n = 0;
    ODA_DISPATCH_DG(head_dim, group, n = (occupancy_tma_t<DD, GG>()));
    return n;
}

}  // namespace oda
