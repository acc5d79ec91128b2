// The paper's recall head (appendix "Recall-head architecture") as ONE persistent kernel for small
// batches: 28.3 M fp32 parameters = 113 MB are read once per step, so the head is a chain of
// bandwidth-bound GEMVs whose only true dependency is the small activation vector between stages.
// This is the measured ALTERNATIVE to the per-stage launches of recall_head_full.cu (opt-in,
// variant 2); on a B200 it is slower than they are, for the reason given at the end.
//
// One CTA per SM (cooperative launch, so all CTAs are resident).  In every stage a CTA owns a
// contiguous range of output rows, i.e. a contiguous range of the weight matrix:
//   * a producer warp streams the CTA's weights of ALL stages, in order, through a ring of 4 KiB
//     slots (whatever shared memory the stage inputs leave: 44 slots at batch 1, 19 at batch 4)
//     with bulk asynchronous copies completing on mbarriers.  Weights do not depend on
//     activations, so the stream runs ahead across stage boundaries;
//   * seven consumer warps each own a pair of rows of the current round: they multiply ring slots
//     by the stage's whole input held in shared memory (RMSNorm gain applied, the interaction
//     vector materialised once per CTA), reduce with a fixed shuffle tree and apply the epilogue;
//   * between dependent stages the CTAs meet at a grid barrier: one arrival counter, a bounded
//     spin (a timeout sets the status word and a global abort flag, and every CTA drains and
//     leaves), activations re-read from L2.  The last CTA to arrive at the final barrier computes
//     the scalar output and the decision, so nobody waits for it.
// No split over k: every output element is summed by one warp in a fixed order, so the result is
// deterministic and needs no partial-sum scratch.
//
// Why it loses (in-kernel timeline at batch 1, 69 us in all): the five grid barriers cost 2.3-5.9 us
// each (release fence, arrival, polling, and the slowest CTA), staging a stage's input 0.5-5.4 us,
// and each is a chain of dependent round trips through a memory system that the weight stream
// keeps loaded; that consumer-side critical path (about 35 us) does not shrink with a deeper ring,
// and it is what programmatic dependent launch already hides about as well between kernels.
#include <algorithm>

#include "launch_ex.cuh"
#include "mbar.cuh"
#include "oda_launch.h"

namespace oda {

constexpr int kFuWarps = 7;                      // consumer warps (8 warps with the producer: 2 per scheduler, 255 registers each)
constexpr int kFuConsumers = kFuWarps * 32;
constexpr int kFuThreads = kFuConsumers + 32;    // + the producer warp
constexpr int kFuPiece = 1024;                   // floats per ring slot (4 KiB): one row, one k chunk
constexpr int kFuMaxSlots = 48;                  // ring slots: whatever shared memory the stage inputs leave
constexpr int kFuMaxB = kFullHeadFusedMaxBatch;
constexpr int kFuCtlBytes = 1024;
constexpr int kFuSmem = kFullHeadFusedSmem;             // stage input | ring | control block

struct FusedHeadParams {
    int32_t batch, T, F, d_model, n_blocks;
    int32_t x_floats;        // shared-memory floats reserved for a stage's input (multiple of 1024)
    int32_t n_slots;         // ring slots behind it
    float eps;
    const float* params;
    const float* in[3];
    float *abc, *z, *h;      // activations in the caller's scratch: [3][B][T], [B][T], [B][F]
    int32_t* sync;           // [0] barrier arrivals, [1] abort flag; zero at launch
    int32_t* status;         // device status word (nullable)
    float threshold;
    const uint8_t* override_flags;
    float* scores;
    float* logits;
    uint8_t* flags;
    int32_t* counters;
};

#define FU_CLK(v) do { } while (0)
#define FU_ACC(slot, dt) do { } while (0)

enum { kFuTower = 0, kFuFusion = 1, kFuGateUp = 2, kFuDown = 3 };

struct FuStage {
    int type, tower, K, units;
    const float* W;     // row r: W + r*K
    const float* W2;    // gate+up: the up projection (row m: W2 + m*K)
    const float* gain;  // RMSNorm gain of the stage input, or nullptr
    const float* bias;
};

struct FuCtl {
    uint64_t full[kFuMaxSlots], empty[kFuMaxSlots];
    float ssq[3 * kFuMaxB];   // sum of squares of the raw stage input, per (tower,) request
    float red[kFuWarps][2];
    int32_t abort;
    int32_t last;
};
static_assert(sizeof(FuCtl) <= kFuCtlBytes, "control block");

__device__ __forceinline__ float fu_silu(float a) { return a / (1.f + expf(-a)); }

// stages: 0-2 towers, 3 fusion, then (gate+up, down) per block
__device__ __forceinline__ FuStage fu_stage(const FusedHeadParams& p, int s)
{
    FuStage d;
    const long long tower_stride = (long long)p.d_model + (long long)p.T * p.d_model + p.T;
    d.W2 = nullptr;
    d.tower = 0;
    d.bias = nullptr;
    d.gain = nullptr;
    if (s < 3) {
        const float* base = p.params + s * tower_stride;
        d.type = kFuTower; d.tower = s; d.K = p.d_model; d.units = p.T;
        d.gain = base; d.W = base + p.d_model; d.bias = base + p.d_model + (long long)p.T * p.d_model;
        return d;
    }
    const float* cur = p.params + 3 * tower_stride;
    if (s == 3) {
        d.type = kFuFusion; d.K = 9 * p.T; d.units = p.T; d.W = cur; d.bias = cur + (long long)p.T * 9 * p.T;
        return d;
    }
    cur += (long long)p.T * 9 * p.T + p.T;
    cur += (long long)((s - 4) >> 1) * ((long long)p.T + 3ll * p.F * p.T);
    if (((s - 4) & 1) == 0) {
        d.type = kFuGateUp; d.K = p.T; d.units = p.F;
        d.gain = cur; d.W = cur + p.T; d.W2 = d.W + (long long)p.F * p.T;
    } else {
        d.type = kFuDown; d.K = p.F; d.units = p.T; d.W = cur + p.T + 2ll * p.F * p.T;
    }
    return d;
}

// A CTA's share of a stage: units [u0, u1).  A consumer warp works on a PAIR of rows at a time so
// that each value of the stage input read from shared memory feeds two dot products: pair i of a
// gate+up stage is (gate row, up row) of hidden unit u0+i, pair i of any other stage is rows
// u0+2i, u0+2i+1 (the second may not exist).  Rounds of 8 pairs, one per warp.
struct FuShare {
    int u0, n, npairs, rounds, nkc;
};
__device__ __forceinline__ FuShare fu_share(const FuStage& d, int c, int G)
{
    FuShare sh;
    sh.u0 = (int)((long long)c * d.units / G);
    sh.n = (int)((long long)(c + 1) * d.units / G) - sh.u0;
    sh.npairs = d.type == kFuGateUp ? sh.n : (sh.n + 1) / 2;
    sh.rounds = (sh.npairs + kFuWarps - 1) / kFuWarps;
    sh.nkc = (d.K + kFuPiece - 1) / kFuPiece;
    return sh;
}
// rows with weights in round rd (ring pieces per k chunk): rank 2w+sub exists iff rank < count
__device__ __forceinline__ int fu_round_rows(const FuStage& d, const FuShare& sh, int rd)
{
    const int left = (d.type == kFuGateUp ? 2 * sh.n : sh.n) - rd * 2 * kFuWarps;
    return min(2 * kFuWarps, left);
}
__device__ __forceinline__ const float* fu_row_ptr(const FuStage& d, const FuShare& sh, int rd, int rank)
{
    const int pair = rd * kFuWarps + (rank >> 1), sub = rank & 1;
    if (d.type == kFuGateUp) return (sub ? d.W2 : d.W) + (size_t)(sh.u0 + pair) * d.K;
    return d.W + (size_t)(sh.u0 + 2 * pair + sub) * d.K;
}

// Producer-side wait with back-off: the ring is full most of the time, and a lane that polls an
// mbarrier back to back competes with the consumers' shared-memory loads for the same pipe.
__device__ __forceinline__ bool fu_wait_backoff(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        __nanosleep(64);
        if ((++spins & 255u) == 0) {
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

__device__ __forceinline__ void fu_consumer_sync()
{
    asm volatile("bar.sync 1, %0;" ::"n"(kFuConsumers) : "memory");
}

__device__ __forceinline__ void fu_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}

// Arrival + bounded spin of consumer thread 0 at grid barrier number `index` (0-based); the
// other consumer threads wait at the named barrier around it.  Returns false after an abort.
__device__ __forceinline__ bool fu_grid_barrier(const FusedHeadParams& p, FuCtl* ctl, int index, int tid)
{
    fu_consumer_sync();  // every warp's outputs of the stage are written
    if (tid == 0) {
        asm volatile("fence.acq_rel.gpu;" ::: "memory");
        asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p.sync), "r"(1) : "memory");
        const int target = (index + 1) * (int)gridDim.x;
        const uint64_t t0 = globaltimer_ns();
        uint32_t spins = 0;
        for (;;) {
            int v;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p.sync) : "memory");
            if (v >= target) break;
            if ((++spins & 63u) == 0) {
                int ab;
                asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(ab) : "l"(p.sync + 1) : "memory");
                if (ab || ctl->abort) { ctl->abort = 1; break; }
                if (globaltimer_ns() - t0 > 1000000000ull) {  // a CTA never arrived: give up everywhere
                    ctl->abort = 1;
                    atomicExch(p.sync + 1, 1);
                    if (p.status) atomicOr(p.status, kStatusWaitTimeout);
                    break;
                }
            }
        }
    }
    fu_consumer_sync();
    return ctl->abort == 0;
}

// One batch of a staged copy: up to eight 128-bit loads per thread are issued before any is stored,
// so a copy of n4 <= 8 * kFuConsumers float4 costs one memory latency.  Sources may have been
// written by other CTAs of this kernel, so they are read through L2 (ld.cg).
struct FuCopy {
    float4 v[8];
    __device__ __forceinline__ void load(const float* src, int n4, int base, int tid)
    {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int idx = base + j * kFuConsumers + tid;
            if (idx < n4) v[j] = __ldcg(reinterpret_cast<const float4*>(src) + idx);
        }
    }
    __device__ __forceinline__ void store(float* dst, int n4, int base, int tid) const
    {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int idx = base + j * kFuConsumers + tid;
            if (idx < n4) reinterpret_cast<float4*>(dst)[idx] = v[j];
        }
    }
};
__device__ __forceinline__ void fu_copy_in(float* dst, const float* src, int n4, int tid)
{
    for (int base = 0; base < n4; base += kFuConsumers * 8) {
        FuCopy c;
        c.load(src, n4, base, tid);
        c.store(dst, n4, base, tid);
    }
}

// RMSNorm preparation in shared memory: rows [nrows][K] hold raw inputs and gains [.][K] their
// gains (row r uses gains[r / rows_per_gain]); writes the sum of squares of row r to ssq[r] and
// multiplies the row by its gain in place.  One warp per row, four elements in flight per lane.
__device__ __forceinline__ void fu_norm_rows(float* x, int nrows, int K, const float* gains, int rows_per_gain,
                                             float* ssq, int warp, int lane)
{
    for (int r = warp; r < nrows; r += kFuWarps) {
        float4* row = reinterpret_cast<float4*>(x + (size_t)r * K);
        const float4* g4 = reinterpret_cast<const float4*>(gains + (size_t)(r / rows_per_gain) * K);
        float ss = 0.f;
        const int n4 = K >> 2;
        for (int q0 = 0; q0 < n4; q0 += 128) {
            float4 v[4], g[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int q = q0 + i * 32 + lane;
                if (q < n4) { v[i] = row[q]; g[i] = g4[q]; }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int q = q0 + i * 32 + lane;
                if (q < n4) {
                    ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
                    row[q] = make_float4(v[i].x * g[i].x, v[i].y * g[i].y, v[i].z * g[i].z, v[i].w * g[i].w);
                }
            }
        }
        for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) ssq[r] = ss;
    }
}

// One round of a stage for one consumer warp and NB requests: the warp's pair of rows, all k
// chunks, then the epilogue.  `base` counts the ring pieces issued before the current chunk (the
// producer's numbering) and advances for every warp alike.
template <int NB>
__device__ __forceinline__ void fu_round(const FusedHeadParams& p, const FuStage& d, const FuShare& sh, int rd,
                                         const float* ring, const float* x, const FuCtl* ctl, uint32_t full0,
                                         uint32_t empty0, volatile int* abort_flag, int* wait_status, uint32_t& base,
                                         bool& aborted, int warp, int lane)
{
    const int cnt = fu_round_rows(d, sh, rd);
    const uint32_t kFuSlots = (uint32_t)p.n_slots;
    const bool v0 = 2 * warp < cnt, v1 = 2 * warp + 1 < cnt;
    if (!v0) {
        base += (uint32_t)(cnt * sh.nkc);
        return;
    }
    float acc0[NB], acc1[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc0[b] = acc1[b] = 0.f;
    const int ld4 = d.K >> 2;
    constexpr int ST = NB <= 2 ? 4 : 2;   // warp-wide steps per batch (registers: ST * (2 + NB) float4)
    for (int kc = 0; kc < sh.nkc; ++kc, base += cnt) {
        const int nv = min(kFuPiece, d.K - kc * kFuPiece) >> 2;
        const uint32_t pc0 = base + 2 * warp, pc1 = pc0 + 1;
        const uint32_t s0 = pc0 % kFuSlots, s1 = pc1 % kFuSlots;
        aborted |= (*abort_flag != 0);
        if (!aborted && !mbar_wait(full0 + 8 * s0, (pc0 / kFuSlots) & 1, abort_flag, wait_status)) aborted = true;
        if (v1 && !aborted && !mbar_wait(full0 + 8 * s1, (pc1 / kFuSlots) & 1, abort_flag, wait_status)) aborted = true;
        aborted = __any_sync(0xffffffffu, aborted);   // also reconverges the lanes after the polling loops
        if (aborted) continue;
        const float4* w0p = reinterpret_cast<const float4*>(ring + (size_t)s0 * kFuPiece);
        const float4* w1p = reinterpret_cast<const float4*>(ring + (size_t)s1 * kFuPiece);
        const float4* x4 = reinterpret_cast<const float4*>(x) + kc * (kFuPiece / 4);
        // every shared-memory load of a batch is issued before its arithmetic: a lone warp per
        // scheduler cannot hide load latency any other way
        int q = lane;
        for (; q + 32 * (ST - 1) < nv; q += 32 * ST) {
            float4 w0[ST], w1[ST], xv[NB][ST];
#pragma unroll
            for (int i = 0; i < ST; ++i) {
                w0[i] = w0p[q + 32 * i];
                w1[i] = v1 ? w1p[q + 32 * i] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int b = 0; b < NB; ++b)
#pragma unroll
                for (int i = 0; i < ST; ++i) xv[b][i] = x4[b * ld4 + q + 32 * i];
#pragma unroll
            for (int b = 0; b < NB; ++b)
#pragma unroll
                for (int i = 0; i < ST; ++i) {
                    acc0[b] = fmaf(w0[i].x, xv[b][i].x, acc0[b]); acc1[b] = fmaf(w1[i].x, xv[b][i].x, acc1[b]);
                    acc0[b] = fmaf(w0[i].y, xv[b][i].y, acc0[b]); acc1[b] = fmaf(w1[i].y, xv[b][i].y, acc1[b]);
                    acc0[b] = fmaf(w0[i].z, xv[b][i].z, acc0[b]); acc1[b] = fmaf(w1[i].z, xv[b][i].z, acc1[b]);
                    acc0[b] = fmaf(w0[i].w, xv[b][i].w, acc0[b]); acc1[b] = fmaf(w1[i].w, xv[b][i].w, acc1[b]);
                }
        }
        for (; q < nv; q += 32) {
            const float4 w0 = w0p[q];
            const float4 w1 = v1 ? w1p[q] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const float4 xv = x4[b * ld4 + q];
                acc0[b] = fmaf(w0.x, xv.x, acc0[b]); acc1[b] = fmaf(w1.x, xv.x, acc1[b]);
                acc0[b] = fmaf(w0.y, xv.y, acc0[b]); acc1[b] = fmaf(w1.y, xv.y, acc1[b]);
                acc0[b] = fmaf(w0.z, xv.z, acc0[b]); acc1[b] = fmaf(w1.z, xv.z, acc1[b]);
                acc0[b] = fmaf(w0.w, xv.w, acc0[b]); acc1[b] = fmaf(w1.w, xv.w, acc1[b]);
            }
        }
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(empty0 + 8 * s0);
            if (v1) mbar_arrive(empty0 + 8 * s1);
        }
    }
    if (aborted) return;
    // ---- the pair's epilogue: fixed shuffle tree, then lane 0 finishes and stores
    const int pair = rd * kFuWarps + warp;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        float a0 = acc0[b], a1 = acc1[b];
        for (int o = 16; o; o >>= 1) {
            a0 += __shfl_xor_sync(0xffffffffu, a0, o);
            a1 += __shfl_xor_sync(0xffffffffu, a1, o);
        }
        if (lane == 0) {
            if (d.type == kFuTower) {
                const float rs = rsqrtf(ctl->ssq[d.tower * NB + b] / (float)d.K + p.eps);
                const int r = sh.u0 + 2 * pair;
                float* o = p.abc + ((size_t)d.tower * NB + b) * p.T + r;
                o[0] = fu_silu(a0 * rs + __ldg(d.bias + r));
                if (v1) o[1] = fu_silu(a1 * rs + __ldg(d.bias + r + 1));
            } else if (d.type == kFuFusion) {
                const int r = sh.u0 + 2 * pair;
                const float* a = x + (size_t)b * 9 * p.T + r;   // first three segments of u = a, b, c
                const int plane = p.T;
                float* o = p.z + (size_t)b * p.T + r;
                o[0] = 0.5f * (a[0] + a[plane] + a[2 * plane] + fu_silu(a0 + __ldg(d.bias + r)));
                if (v1) o[1] = 0.5f * (a[1] + a[plane + 1] + a[2 * plane + 1] + fu_silu(a1 + __ldg(d.bias + r + 1)));
            } else if (d.type == kFuGateUp) {
                const float rs = rsqrtf(ctl->ssq[b] / (float)d.K + p.eps);
                p.h[(size_t)b * p.F + sh.u0 + pair] = fu_silu(a0 * rs) * (a1 * rs);
            } else {
                float* o = p.z + (size_t)b * p.T + sh.u0 + 2 * pair;
                o[0] = __ldcg(o) + a0;
                if (v1) o[1] = __ldcg(o + 1) + a1;
            }
        }
    }
}

__global__ void __launch_bounds__(kFuThreads, 1) full_head_fused_kernel(const __grid_constant__ FusedHeadParams p)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    float* xs = reinterpret_cast<float*>(smem);
    float* ring = xs + p.x_floats;
    FuCtl* ctl = reinterpret_cast<FuCtl*>(smem + kFuSmem - kFuCtlBytes);
    const uint32_t kFuSlots = (uint32_t)p.n_slots;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    if (tid == 0) {
        for (int s = 0; s < kFuMaxSlots; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        ctl->abort = 0;
        ctl->last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int* abort_flag = &ctl->abort;
    int* wait_status = p.status ? p.status : p.sync + 1;
    const int n_stages = 4 + 2 * p.n_blocks;
    const int G = gridDim.x, c = blockIdx.x, B = p.batch;

    if (warp == kFuWarps) {
        // ------------------------------------------------------------ producer: the weight stream
        if (lane == 0) {
            uint64_t policy;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
            uint32_t piece = 0;
            bool dead = false;
            for (int s = 0; s < n_stages && !dead; ++s) {
                const FuStage d = fu_stage(p, s);
                const FuShare sh = fu_share(d, c, G);
                for (int rd = 0; rd < sh.rounds && !dead; ++rd) {
                    const int cnt = fu_round_rows(d, sh, rd);
                    for (int kc = 0; kc < sh.nkc && !dead; ++kc) {
                        const int n = min(kFuPiece, d.K - kc * kFuPiece);
                        for (int rank = 0; rank < cnt; ++rank, ++piece) {
                            const uint32_t slot = piece % kFuSlots, ph = (piece / kFuSlots) & 1;
                            if (!fu_wait_backoff(empty0 + 8 * slot, ph ^ 1, abort_flag, wait_status)) {
                                dead = true;
                                break;
                            }
                            mbar_expect_tx(full0 + 8 * slot, (uint32_t)n * 4);
                            fu_bulk_load(smem_u32(ring + (size_t)slot * kFuPiece), fu_row_ptr(d, sh, rd, rank) + (size_t)kc * kFuPiece,
                                         (uint32_t)n * 4, full0 + 8 * slot, policy);
                        }
                    }
                }
            }
            // do not leave while copies may still be landing: wait (bounded) until the consumers
            // have released every slot that was armed
            for (uint32_t k = 0; k < kFuSlots && k < piece; ++k) {
                const uint32_t c2 = piece - 1 - k;
                if (!mbar_wait(empty0 + 8 * (c2 % kFuSlots), (c2 / kFuSlots) & 1, abort_flag, wait_status)) break;
            }
            if (*abort_flag)
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        }
        __syncthreads();
        return;
    }

    // ---------------------------------------------------------------- consumers
    uint32_t base = 0;       // ring pieces issued before the current (round, k chunk)
    bool aborted = false;
    int barrier_index = 0;
    for (int s = 0; s < n_stages; ++s) {
        const FuStage d = fu_stage(p, s);
        const FuShare sh = fu_share(d, c, G);
        // ---- the stage's whole input -> shared memory, as [B][K] (gain applied where the stage
        //      input is RMS-normalised); gains ride behind the inputs so that every load of the
        //      staging is in flight together
        const float* x = xs;
        if (s == 0) {
            const int n4 = B * p.d_model / 4, g4 = p.d_model / 4;
            const long long tower_stride = (long long)p.d_model + (long long)p.T * p.d_model + p.T;
            float* gains = xs + (size_t)3 * B * p.d_model;
            // six source arrays, one contiguous destination [in0 | in1 | in2 | gain0 | gain1 | gain2]
            const int total4 = 3 * n4 + 3 * g4;
            for (int base4 = 0; base4 < total4; base4 += kFuConsumers * 8) {
                float4 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int idx = base4 + j * kFuConsumers + tid;
                    if (idx < total4) {
                        const float* src;
                        int off;
                        if (idx < 3 * n4) {
                            const int i = idx / n4;
                            off = idx - i * n4;
                            src = i == 0 ? p.in[0] : (i == 1 ? p.in[1] : p.in[2]);
                        } else {
                            const int i = (idx - 3 * n4) / g4;
                            off = (idx - 3 * n4) - i * g4;
                            src = p.params + i * tower_stride;
                        }
                        v[j] = __ldg(reinterpret_cast<const float4*>(src) + off);
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int idx = base4 + j * kFuConsumers + tid;
                    if (idx < total4) reinterpret_cast<float4*>(xs)[idx] = v[j];
                }
            }
            fu_consumer_sync();
            fu_norm_rows(xs, 3 * B, p.d_model, gains, B, ctl->ssq, warp, lane);
            fu_consumer_sync();
        } else if (s < 3) {
            x = xs + (size_t)s * B * p.d_model;   // staged with tower 0's
        } else {
            aborted |= !fu_grid_barrier(p, ctl, barrier_index++, tid);  // reads what the previous stage wrote
            if (d.type == kFuFusion) {
                // u = [a; b; c; a.b; |a-b|; a.c; |a-c|; b.c; |b-c|] per request: the towers' outputs go
                // straight to the first three segments, the other six are formed from them
                const int T4 = p.T >> 2, n4 = 3 * B * T4;
                for (int base4 = 0; base4 < n4; base4 += kFuConsumers * 8) {
                    FuCopy cpy;
                    cpy.load(p.abc, n4, base4, tid);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int idx = base4 + j * kFuConsumers + tid;
                        if (idx < n4) {
                            const int i = idx / (B * T4), rem = idx - i * (B * T4), b = rem / T4, j4 = rem - b * T4;
                            reinterpret_cast<float4*>(xs)[(size_t)b * 9 * T4 + i * T4 + j4] = cpy.v[j];
                        }
                    }
                }
                fu_consumer_sync();
                for (int idx = tid; idx < 3 * B * T4; idx += kFuConsumers) {
                    const int pair = idx / (B * T4), rem = idx - pair * (B * T4), b = rem / T4, j4 = rem - b * T4;
                    float4* u = reinterpret_cast<float4*>(xs) + (size_t)b * 9 * T4;
                    const int i0 = pair == 2 ? 1 : 0, i1 = pair == 0 ? 1 : 2;   // (a,b) (a,c) (b,c)
                    const float4 v = u[i0 * T4 + j4], y = u[i1 * T4 + j4];
                    u[(3 + 2 * pair) * T4 + j4] = make_float4(v.x * y.x, v.y * y.y, v.z * y.z, v.w * y.w);
                    u[(4 + 2 * pair) * T4 + j4] = make_float4(fabsf(v.x - y.x), fabsf(v.y - y.y), fabsf(v.z - y.z), fabsf(v.w - y.w));
                }
                fu_consumer_sync();
            } else if (d.type == kFuGateUp) {
                float* gains = xs + (size_t)B * p.T;
                fu_copy_in(xs, p.z, B * p.T / 4, tid);
                fu_copy_in(gains, d.gain, p.T / 4, tid);
                fu_consumer_sync();
                fu_norm_rows(xs, B, p.T, gains, B, ctl->ssq, warp, lane);
                fu_consumer_sync();
            } else {
                fu_copy_in(xs, p.h, B * p.F / 4, tid);
                fu_consumer_sync();
            }
        }
        for (int rd = 0; rd < sh.rounds; ++rd) {
            switch (B) {
            case 1: fu_round<1>(p, d, sh, rd, ring, x, ctl, full0, empty0, abort_flag, wait_status, base, aborted, warp, lane); break;
            case 2: fu_round<2>(p, d, sh, rd, ring, x, ctl, full0, empty0, abort_flag, wait_status, base, aborted, warp, lane); break;
            case 3: fu_round<3>(p, d, sh, rd, ring, x, ctl, full0, empty0, abort_flag, wait_status, base, aborted, warp, lane); break;
            default: fu_round<4>(p, d, sh, rd, ring, x, ctl, full0, empty0, abort_flag, wait_status, base, aborted, warp, lane); break;
            }
        }
    }
    // ---- final barrier is a ticket: the CTA that arrives last computes q = w . RMSNorm(z) + bias
    fu_consumer_sync();
    if (tid == 0) {
        __threadfence();
        const int old = atomicAdd(p.sync, 1);
        ctl->last = (old == (barrier_index + 1) * G - 1) && !*abort_flag;
        __threadfence();
    }
    fu_consumer_sync();
    if (ctl->last) {
        const long long tower_stride = (long long)p.d_model + (long long)p.T * p.d_model + p.T;
        const float* cur = p.params + 3 * tower_stride + (long long)p.T * 9 * p.T + p.T +
                           (long long)p.n_blocks * ((long long)p.T + 3ll * p.F * p.T);
        const float *gain = cur, *w = cur + p.T, *bias = cur + 2 * p.T;
        for (int b = 0; b < B; ++b) {
            float ss = 0.f, dot = 0.f;
            for (int k = tid * 4; k < p.T; k += kFuConsumers * 4) {
                const float4 xv = __ldcg(reinterpret_cast<const float4*>(p.z + (size_t)b * p.T + k));
                const float4 g = __ldg(reinterpret_cast<const float4*>(gain + k));
                const float4 ww = __ldg(reinterpret_cast<const float4*>(w + k));
                ss += xv.x * xv.x + xv.y * xv.y + xv.z * xv.z + xv.w * xv.w;
                dot = fmaf(ww.x, xv.x * g.x, dot);
                dot = fmaf(ww.y, xv.y * g.y, dot);
                dot = fmaf(ww.z, xv.z * g.z, dot);
                dot = fmaf(ww.w, xv.w * g.w, dot);
            }
            for (int o = 16; o; o >>= 1) {
                ss += __shfl_xor_sync(0xffffffffu, ss, o);
                dot += __shfl_xor_sync(0xffffffffu, dot, o);
            }
            if (lane == 0) { ctl->red[warp][0] = ss; ctl->red[warp][1] = dot; }
            fu_consumer_sync();
            if (tid == 0) {
                float s2 = 0.f, d2 = 0.f;
#pragma unroll
                for (int wv = 0; wv < kFuWarps; ++wv) { s2 += ctl->red[wv][0]; d2 += ctl->red[wv][1]; }
                const float zq = d2 * rsqrtf(s2 / (float)p.T + p.eps) + __ldg(bias);
                const float score = 1.f / (1.f + expf(-zq));
                uint8_t f;
                if (p.override_flags)
                    f = p.override_flags[b] ? 1 : 0;
                else
                    f = (!isfinite(zq) || score > p.threshold) ? 1 : 0;
                p.scores[b] = score;
                if (p.logits) p.logits[b] = zq;
                p.flags[b] = f;
                if (p.counters) {
                    p.counters[2 * b] += 1;
                    p.counters[2 * b + 1] += f;
                }
            }
            fu_consumer_sync();
        }
        if (tid == 0) *p.sync = 0;   // the arrival counter is ready for the next launch
    }
    __syncthreads();  // with the producer: shared memory stays alive until its copies have landed
}

// shared-memory floats a stage's whole input needs: towers (inputs + gains), interaction vector, h
long long full_head_fused_x_floats(int batch, int d_model, int T, int F)
{
    return std::max({3ll * d_model * (batch + 1), 9ll * T * batch, (long long)T * (batch + 1), (long long)F * batch});
}

// Grid of the fused head on the current device: one CTA per SM if a cooperative launch can hold
// them all, else 0 (the caller then uses the staged kernels).
int full_head_fused_grid()
{
    static int cached[64];
    static bool known[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (known[dev]) return cached[dev];
    int sms = 0, coop = 0, per_sm = 0;
    int grid = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && coop &&
        cudaFuncSetAttribute(full_head_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFuSmem) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, full_head_fused_kernel, kFuThreads, kFuSmem) == cudaSuccess &&
        per_sm >= 1)
        grid = sms;
    (void)cudaGetLastError();
    cached[dev] = grid;
    known[dev] = true;
    return grid;
}

cudaError_t launch_full_head_fused(int grid, int batch, int d_model, int T, int F, int n_blocks, float eps,
                                   const float* params, const float* h_prev, const float* emb, const float* h_local,
                                   float threshold, const uint8_t* override_flags, float* scores, float* logits,
                                   uint8_t* flags, int32_t* counters, float* abc, float* z, float* h, int32_t* sync,
                                   int32_t* status, cudaStream_t st)
{
    FusedHeadParams p = {};
    p.batch = batch; p.T = T; p.F = F; p.d_model = d_model; p.n_blocks = n_blocks; p.eps = eps;
    const long long need = full_head_fused_x_floats(batch, d_model, T, F);
    p.x_floats = (int32_t)((need + 1023) / 1024 * 1024);
    p.n_slots = std::min(kFuMaxSlots, (kFuSmem - kFuCtlBytes - p.x_floats * 4) / (kFuPiece * 4));
    if (p.n_slots < 8) return cudaErrorNotSupported;
    p.params = params;
    p.in[0] = h_prev; p.in[1] = emb; p.in[2] = h_local;
    p.abc = abc; p.z = z; p.h = h;
    p.sync = sync; p.status = status;
    p.threshold = threshold; p.override_flags = override_flags;
    p.scores = scores; p.logits = logits; p.flags = flags; p.counters = counters;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kFuThreads);
    cfg.dynamicSmemBytes = kFuSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident: the grid barriers cannot starve
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, full_head_fused_kernel, p);
}

}  // namespace oda
