// Split-KV paged decode attention, CUDA-core variant: 128-bit coalesced K/V loads straight
// from global memory into registers, fp32 FMA dot products, warp-shuffle reductions, online
// softmax per lane group, then a cross-warp merge and the split merge of oda_device.cuh.
// Serves both the Local pass (Eq. 1, S^L) and the gated Full pass (S^F).
#include "oda_device.cuh"
#include "launch_ex.cuh"
#include "oda_launch.h"

namespace oda {

template <int D, int G>
struct SimtCfg {
    static constexpr int kWarps = 4;
    static constexpr int kThreads = kWarps * 32;
    static constexpr int kLPR = D / 8;            // lanes per token row (8 bf16 each)
    static constexpr int kRPL = 32 / kLPR;        // token rows per warp-wide load
    static constexpr int kLoads = kPage / kRPL;   // loads per page per tensor
    static constexpr int kBatch = (G * kLoads <= 32) ? kLoads : (32 / G);  // rows per softmax update
    static constexpr int kSubs = kWarps * kRPL;   // independent online-softmax streams per CTA
    static constexpr int kW = D + kPartHdr;
};

__device__ __forceinline__ uint4 ldg_stream(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& r, float* f)
{
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
}

template <int D, int G>
__global__ void __launch_bounds__(SimtCfg<D, G>::kThreads)
splitkv_simt_kernel(const __grid_constant__ AttnParams p)
{
    using C = SimtCfg<D, G>;
    __shared__ Plan plan;
    __shared__ float s_sub[C::kSubs][G][C::kW];
    __shared__ float s_part[G][C::kW];
    __shared__ int s_is_last;

    prefetch_block_table(p);
    griddep_wait();
    if (gated_pass_is_empty(p)) {
        griddep_launch_dependents();
        return;
    }
    build_plan(p, plan);
    griddep_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / C::kLPR;               // which row of a warp-wide load this lane reads
    const int dofs = (lane % C::kLPR) * 8;        // this lane's 8 head-dim elements

    const int span = plan.my_span;
    if (span < 0) return;
    {
    int x_begin, x_end;
    span_range(plan, span, x_begin, x_end);
    for (int x = x_begin; x < x_end;) {
        Item it;
        x += decode_item(p, plan, span, x, x_end, it);
        // q for the G heads of this kv head, pre-multiplied by scale * log2(e)
        float qf[G][8];
        {
            const __nv_bfloat16* qb =
                p.q + (((size_t)it.layer * p.batch + it.b) * p.num_q_heads + (size_t)it.g * G) * D + dofs;
#pragma unroll
            for (int h = 0; h < G; ++h) {
                uint4 r = *reinterpret_cast<const uint4*>(qb + (size_t)h * D);
                bf16x8_to_f32(r, qf[h]);
#pragma unroll
                for (int d = 0; d < 8; ++d) qf[h][d] *= p.scale_log2e;
            }
        }
        float m[G], l[G], o[G][8];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m[h] = -INFINITY;
            l[h] = 0.f;
#pragma unroll
            for (int d = 0; d < 8; ++d) o[h][d] = 0.f;
        }
        const size_t kv_base = (size_t)it.kv_layer * p.kv_layer_stride + (size_t)it.g * p.kv_head_stride + dofs;
        const int32_t* bt = p.block_table + (size_t)it.b * p.max_blocks_per_seq;

        // segment 0: sink pages (only chunk 0 of a two-segment Local set), segment 1: window/full pages
#pragma unroll 1
        for (int seg = 0; seg < 2; ++seg) {
            const int pg0 = seg ? it.win_pg0 : 0;
            const int pg1 = seg ? it.win_pg1 : it.sink_pg1;
            const int vlo = seg ? it.win_lo : 0;
            const int vhi = seg ? it.win_hi : it.sink_hi;
#pragma unroll 1
            for (int pg = pg0 + warp; pg < pg1; pg += C::kWarps) {
                const int blk = __ldg(bt + pg);
                const size_t pbase = kv_base + (size_t)blk * p.kv_block_stride;
                uint4 kr[C::kLoads], vr[C::kLoads];
#pragma unroll
                for (int i = 0; i < C::kLoads; ++i)
                    kr[i] = ldg_stream(p.k + pbase + (size_t)(i * C::kRPL + sub) * p.kv_token_stride);
#pragma unroll
                for (int i = 0; i < C::kLoads; ++i)
                    vr[i] = ldg_stream(p.v + pbase + (size_t)(i * C::kRPL + sub) * p.kv_token_stride);
#pragma unroll
                for (int i0 = 0; i0 < C::kLoads; i0 += C::kBatch) {
                    float s[C::kBatch][G];
#pragma unroll
                    for (int i = 0; i < C::kBatch; ++i) {
                        float kf[8];
                        bf16x8_to_f32(kr[i0 + i], kf);
#pragma unroll
                        for (int h = 0; h < G; ++h) {
                            float a = 0.f;
#pragma unroll
                            for (int d = 0; d < 8; ++d) a = fmaf(qf[h][d], kf[d], a);
                            s[i][h] = a;
                        }
                    }
#pragma unroll
                    for (int off = C::kLPR / 2; off; off >>= 1)
#pragma unroll
                        for (int i = 0; i < C::kBatch; ++i)
#pragma unroll
                            for (int h = 0; h < G; ++h)
                                s[i][h] += __shfl_xor_sync(0xffffffffu, s[i][h], off);
                    float mn[G];
#pragma unroll
                    for (int h = 0; h < G; ++h) mn[h] = m[h];
#pragma unroll
                    for (int i = 0; i < C::kBatch; ++i) {
                        const int pos = pg * kPage + (i0 + i) * C::kRPL + sub;
                        const bool ok = pos >= vlo && pos < vhi;
#pragma unroll
                        for (int h = 0; h < G; ++h) {
                            s[i][h] = ok ? s[i][h] : -INFINITY;
                            mn[h] = fmaxf(mn[h], s[i][h]);
                        }
                    }
#pragma unroll
                    for (int h = 0; h < G; ++h) {
                        const float mu = (mn[h] == -INFINITY) ? 0.f : mn[h];
                        const float alpha = ex2(m[h] - mu);  // m = -inf -> 0
                        m[h] = mn[h];
                        l[h] *= alpha;
#pragma unroll
                        for (int d = 0; d < 8; ++d) o[h][d] *= alpha;
#pragma unroll
                        for (int i = 0; i < C::kBatch; ++i) s[i][h] = ex2(s[i][h] - mu);
                    }
#pragma unroll
                    for (int i = 0; i < C::kBatch; ++i) {
                        float vf[8];
                        bf16x8_to_f32(vr[i0 + i], vf);
                        const int pos = pg * kPage + (i0 + i) * C::kRPL + sub;
                        const bool ok = pos >= vlo && pos < vhi;
                        if (!ok) {  // slots outside the set may hold anything, also NaN bit patterns
#pragma unroll
                            for (int d = 0; d < 8; ++d) vf[d] = 0.f;
                        }
#pragma unroll
                        for (int h = 0; h < G; ++h) {
                            l[h] += s[i][h];
#pragma unroll
                            for (int d = 0; d < 8; ++d) o[h][d] = fmaf(s[i][h], vf[d], o[h][d]);
                        }
                    }
                }
            }
        }
        // publish each lane group's stream, then merge the streams of the CTA
        const int sidx = warp * C::kRPL + sub;
#pragma unroll
        for (int h = 0; h < G; ++h) {
            if ((lane % C::kLPR) == 0) {
                s_sub[sidx][h][0] = m[h];
                s_sub[sidx][h][1] = l[h];
                s_sub[sidx][h][2] = 0.f;
                s_sub[sidx][h][3] = 0.f;
            }
#pragma unroll
            for (int d = 0; d < 8; ++d) s_sub[sidx][h][kPartHdr + dofs + d] = o[h][d];
        }
        __syncthreads();
        for (int e = tid; e < G * C::kW; e += C::kThreads) {
            const int h = e / C::kW, j = e - h * C::kW;
            float M = -INFINITY;
#pragma unroll
            for (int u = 0; u < C::kSubs; ++u) M = fmaxf(M, s_sub[u][h][0]);
            if (j == 0) {
                s_part[h][0] = M;
            } else {
                float acc = 0.f;
#pragma unroll
                for (int u = 0; u < C::kSubs; ++u) {
                    const float mu = s_sub[u][h][0];
                    const float sc = (mu == -INFINITY) ? 0.f : ex2(mu - M);
                    acc += s_sub[u][h][j] * sc;
                }
                s_part[h][j] = acc;
            }
        }
        __syncthreads();
        finish_item<D, G>(p, it, &s_part[0][0], &s_is_last);
        __syncthreads();
    }
    }
}

template <int D, int G>
static cudaError_t launch_simt_t(const AttnParams& p, int grid, cudaStream_t st, bool pdl)
{
    return launch_ex(splitkv_simt_kernel<D, G>, dim3(grid), dim3(SimtCfg<D, G>::kThreads), 0, st, pdl, p);
}

template <int D, int G>
static int occupancy_simt_t()
{
    int n = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, splitkv_simt_kernel<D, G>, SimtCfg<D, G>::kThreads, 0);
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

cudaError_t launch_splitkv_simt(const AttnParams& p, int head_dim, int group, int grid, cudaStream_t st, bool pdl)
{
    cudaError_t e = cudaErrorInvalidValue;
    ODA_DISPATCH_DG(head_dim, group, e = (launch_simt_t<DD, GG>(p, grid, st, pdl)));
    return e;
}

int occupancy_splitkv_simt(int head_dim, int group)
{
    int n = 0;
    ODA_DISPATCH_DG(head_dim, group, n = (occupancy_simt_t<DD, GG>()));
    return n;
}

}  // namespace oda
