// KV-head tensor parallelism: the decision's one exchange fused into the kernel that takes the
// decision.  Every rank holds its share of W1 x (the first layer of the recall head split by input
// columns, see recall_head.cu).  One CTA per rank
//   1. stores that share into slot [rank] of EVERY rank's receive buffer (plain peer stores over
//      NVLink; its own buffer included),
//   2. makes the stores visible system-wide and raises its arrival flag in every rank's flag array
//      (the flag carries the step's epoch, so nothing is ever reset),
//   3. waits, with a time limit, until all ranks' flags in its OWN array show the epoch,
//   4. adds the shares in rank order from its own buffer and applies bias, SiLU, the second layer
//      and the decision rule.  All ranks add the same numbers in the same order, so they take the
//      same decision bit for bit and no flag has to be sent around.
// Receive buffers are double-buffered by epoch parity: a rank can run at most one exchange ahead
// of the slowest one (it needs that rank's flag to get past step 3), so the buffer it writes at
// epoch e+2 has been read by everybody at epoch e.
//
// No collective library call, no switch-side replication, no load from a peer: only stores to peers and loads
// from local memory.  On one GPU the same kernel is checked by giving each "rank" a CTA of ONE
// cooperative launch (the CTAs wait on one another, so they must be co-resident) and separate
// buffers.  A wait that runs out sets bit 2 of the status word, leaves the outputs untouched and
// returns.
#include "launch_ex.cuh"
#include "mbar.cuh"
#include "oda_device.cuh"
#include "oda_launch.h"

namespace oda {

__device__ __forceinline__ void st_release_sys(uint32_t* p, uint32_t v)
{
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_sys(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void __launch_bounds__(kExchangeThreads) recall_exchange_kernel(const __grid_constant__ ExchangeParams p)
{
    __shared__ int s_ok;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = blockIdx.x;              // which of the ranks run by this launch
    const int rank = p.rank_base + slot;
    const ExchangeRank& me = p.ranks[slot];
    const int n = p.batch * p.d_hidden;       // floats per share
    const size_t parity_off = (size_t)(p.epoch & 1u) * p.world * n;
    // 1. this rank's share -> slot [rank] of every rank's receive buffer
    for (int peer = 0; peer < p.world; ++peer) {
        float* dst = p.recv[peer] + parity_off + (size_t)rank * n;
        if ((n & 3) == 0) {
            for (int i = tid; i < n / 4; i += kExchangeThreads)
                reinterpret_cast<float4*>(dst)[i] = reinterpret_cast<const float4*>(me.pre_local)[i];
        } else {
            for (int i = tid; i < n; i += kExchangeThreads) dst[i] = me.pre_local[i];
        }
    }
    // 2. visible everywhere, then the arrival flags
    __threadfence_system();
    __syncthreads();
    if (tid < p.world) st_release_sys(p.arrived[tid] + rank, p.epoch);
    // 3. bounded wait for every rank's flag in this rank's own array
    if (tid == 0) s_ok = 1;
    __syncthreads();
    if (tid < p.world) {
        const uint32_t* f = p.arrived[rank] + tid;
        const uint64_t t0 = globaltimer_ns();
        uint32_t spins = 0;
        while ((int32_t)(ld_acquire_sys(f) - p.epoch) < 0) {  // a rank that is already one exchange ahead has arrived too
            if ((++spins & 63u) == 0 && globaltimer_ns() - t0 > p.timeout_ns) {
                s_ok = 0;
                break;
            }
        }
    }
    __syncthreads();
    if (!s_ok) {
        if (tid == 0 && p.status) atomicOr(p.status, kStatusWaitTimeout);
        return;
    }
    // 4. shares added in rank order, then the second layer: one warp per request, lanes take hidden
    //    units 32 apart, fixed shuffle tree
    const float* mine = p.recv[rank] + parity_off;
    for (int b = warp; b < p.batch; b += kExchangeThreads / 32) {
        float zp = 0.f;
        for (int j = lane; j < p.d_hidden; j += 32) {
            float a = 0.f;
            for (int r = 0; r < p.world; ++r) a += __ldcg(mine + (size_t)r * n + (size_t)b * p.d_hidden + j);
            a += __ldg(p.b1 + j);
            zp += __ldg(p.w2 + j) * (a / (1.f + expf(-a)));
        }
        for (int o = 16; o; o >>= 1) zp += __shfl_xor_sync(0xffffffffu, zp, o);
        if (lane == 0) {
            const float z = __ldg(p.b2) + zp;
            const float score = 1.f / (1.f + expf(-z));
            uint8_t f;
            if (p.override_flags)
                f = p.override_flags[b] ? 1 : 0;
            else
                f = (!isfinite(z) || score > p.threshold) ? 1 : 0;
            me.scores[b] = score;
            if (me.logits) me.logits[b] = z;
            me.flags[b] = f;
            if (me.counters) {
                me.counters[2 * b] += 1;
                me.counters[2 * b + 1] += f;
            }
        }
    }
}

cudaError_t launch_recall_exchange(const ExchangeParams& p, int n_local, cudaStream_t st, bool pdl)
{
    if (n_local == 1) return launch_ex(recall_exchange_kernel, dim3(1), dim3(kExchangeThreads), 0, st, pdl, p);
    // several ranks on one GPU (checking the protocol): the CTAs wait on one another, so the launch is
    // cooperative -- it fails instead of starting if they cannot all be resident
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_local);
    cfg.blockDim = dim3(kExchangeThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, recall_exchange_kernel, p);
}

}  // namespace oda

// ---------------------------------------------------------------------------------------------------
// Sequence-sharded Full pass: the exchange of the per-rank (out, lse) rows fused with their
// log-sum-exp combination, by the same protocol.  The rows are cut into kMergeBlocks blocks; CTA c
// of every rank pushes its rows of block c into every rank's receive buffer, raises flag
// [rank][c] everywhere, waits for the other ranks' flag c in its own array and combines block c in
// rank order -- so blocks flow independently and no CTA waits for rows it does not need.
namespace oda {

template <int V>
__global__ void __launch_bounds__(kExchangeThreads) merge_exchange_kernel(const __grid_constant__ MergeExchangeParams p)
{
    __shared__ int s_ok;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int D = V * 32;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.x, slot = blockIdx.y;
    const int rank = p.rank_base + slot;
    const MergeExchangeRank& me = p.ranks[slot];
    const long long all_rows = (long long)p.num_layers * p.batch * p.q_heads;   // rows of a whole [L,B,Hq] array
    const long long rows = (long long)(p.layer_end - p.layer_begin) * p.batch * p.q_heads;
    const long long r0 = rows * c / kMergeBlocks, r1 = rows * (c + 1) / kMergeBlocks;
    const size_t par = (size_t)(p.epoch & 1u) * p.world;
    auto row_of = [&](long long w, int& b, bool& live) {
        const int h = (int)(w % p.q_heads);
        b = (int)((w / p.q_heads) % p.batch);
        const int l = p.layer_begin + (int)(w / ((long long)p.q_heads * p.batch));
        live = p.layers[l].gated && (!me.flags || me.flags[b]);
        return ((long long)l * p.batch + b) * p.q_heads + h;
    };
    // 1. this rank's rows of block c -> slot [rank] of every rank's receive buffers
    for (long long w = r0 + warp; w < r1; w += kExchangeThreads / 32) {
        int b;
        bool live;
        const long long row = row_of(w, b, live);
        if (!live) continue;
        const float lr = (!me.tokens_local || me.tokens_local[b] > 0) ? me.part_lse[row] : -INFINITY;
        float v[V];
        if (lr != -INFINITY) {
#pragma unroll
            for (int e = 0; e < V; ++e) v[e] = me.part_out[row * D + lane * V + e];
        }
        for (int peer = 0; peer < p.world; ++peer) {
            const size_t base = (par + rank) * (size_t)all_rows + (size_t)row;
            if (lane == 0) p.recv_lse[peer][base] = lr;
            if (lr != -INFINITY) {
                float* dst = p.recv_out[peer] + base * D + lane * V;
#pragma unroll
                for (int e = 0; e < V; ++e) dst[e] = v[e];
            }
        }
    }
    // 2. visible everywhere, then flag [rank][c] in every rank's array
    __threadfence_system();
    __syncthreads();
    if (tid < p.world) st_release_sys(p.arrived[tid] + (size_t)rank * kMergeBlocks + c, p.epoch);
    // 3. bounded wait for the other ranks' block c
    if (tid == 0) s_ok = 1;
    __syncthreads();
    if (tid < p.world) {
        const uint32_t* f = p.arrived[rank] + (size_t)tid * kMergeBlocks + c;
        const uint64_t t0 = globaltimer_ns();
        uint32_t spins = 0;
        while ((int32_t)(ld_acquire_sys(f) - p.epoch) < 0) {  // a rank that is already one exchange ahead has arrived too
            if ((++spins & 63u) == 0 && globaltimer_ns() - t0 > p.timeout_ns) {
                s_ok = 0;
                break;
            }
        }
    }
    __syncthreads();
    if (!s_ok) {
        if (tid == 0 && p.status) atomicOr(p.status, kStatusWaitTimeout);
        return;
    }
    // 4. log-sum-exp combination of block c, parts in rank order
    const float* my_lse = p.recv_lse[rank];
    const float* my_out = p.recv_out[rank];
    for (long long w = r0 + warp; w < r1; w += kExchangeThreads / 32) {
        int b;
        bool live;
        const long long row = row_of(w, b, live);
        if (!live) continue;
        float m = -INFINITY;
        for (int r = 0; r < p.world; ++r) m = fmaxf(m, __ldcg(my_lse + (par + r) * (size_t)all_rows + row));
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.f;
        float sum = 0.f;
        if (m > -INFINITY) {
            for (int r = 0; r < p.world; ++r) {
                const size_t base = (par + r) * (size_t)all_rows + row;
                const float lr = __ldcg(my_lse + base);
                if (lr == -INFINITY) continue;
                const float wgt = expf(lr - m);
                sum += wgt;
                const float* src = my_out + base * D + lane * V;
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = fmaf(wgt, __ldcg(src + e), acc[e]);
            }
        }
        const float inv = sum > 0.f ? 1.f / sum : 0.f;
        float* dst = me.out + row * D + lane * V;
#pragma unroll
        for (int e = 0; e < V; ++e) dst[e] = acc[e] * inv;
        if (me.lse && lane == 0) me.lse[row] = sum > 0.f ? m + logf(sum) : -INFINITY;
    }
}

cudaError_t launch_merge_exchange(const MergeExchangeParams& p, int n_local, int head_dim, cudaStream_t st, bool pdl)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kMergeBlocks, n_local);
    cfg.blockDim = dim3(kExchangeThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (n_local > 1) {   // ranks sharing one GPU wait on one another: all CTAs must be resident
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
    } else {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (n_local > 1 || pdl) ? 1 : 0;
    if (head_dim == 128) return cudaLaunchKernelEx(&cfg, merge_exchange_kernel<4>, p);
    return cudaLaunchKernelEx(&cfg, merge_exchange_kernel<2>, p);
}

}  // namespace oda
