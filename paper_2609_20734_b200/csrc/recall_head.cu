// Recall head of the benchmark configurations, fused with the decision rule:
//   z = w2 . SiLU(W1 x + b1) + b2,  score = sigmoid(z),
//   flag = override ? override[b] : (!isfinite(z) || score > threshold)     (strict >)
// x = [feat_ext ; flattened Local attention output].  fp32 throughout (the paper's head is
// FP32).  One warp per hidden row; CTAs publish per-request partial sums, and the CTA that
// arrives last (one atomic ticket, no waiting) adds them in CTA order and writes the flags,
// so the result does not depend on scheduling.
#include <cuda_bf16.h>
#include "launch_ex.cuh"
#include "oda_launch.h"

namespace oda {

constexpr int kHeadRows = 8;                  // hidden rows per CTA, one warp each
constexpr int kHeadThreads = kHeadRows * 32;
constexpr int kHeadBT = 16;                   // requests per tile
constexpr int kHeadKT = 512;                  // input features per CTA (split-K)

__device__ __forceinline__ float head_x(const HeadParams& p, int b, int i)
{
    if (i < p.d_ext) return __ldg(p.feat_ext + (size_t)b * p.d_ext + i);
    size_t k = (size_t)b * p.d_attn + (i - p.d_ext);
    if (p.attn_bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.attn_out)[k]);
    return reinterpret_cast<const float*>(p.attn_out)[k];
}

// four consecutive input features of request b starting at feature i (i % 4 == 0, vector path)
__device__ __forceinline__ float4 head_x4(const HeadParams& p, int b, int i)
{
    if (i < p.d_ext) return __ldg(reinterpret_cast<const float4*>(p.feat_ext + (size_t)b * p.d_ext + i));
    const size_t k = (size_t)b * p.d_attn + (i - p.d_ext);
    if (p.attn_bf16) {
        const uint2 r = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p.attn_out) + k);
        return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                           __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
    }
    return *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.attn_out) + k);
}

// Split-K GEMV: CTA (rb, ks) multiplies kHeadRows rows of W1 (HBM, read once, 128-bit loads) by
// one 512-feature tile of the inputs x of up to 16 requests (staged in shared memory), and
// publishes the partial pre-activations.  The last CTA of a row block (atomic ticket, no
// waiting) adds the K slices in order, applies bias, SiLU and w2; the last row block adds the
// row blocks' sums in a fixed tree and writes score, logit, flag and counters.  Every sum has a
// fixed order, so the result does not depend on scheduling.  A head whose inputs fit one K slice
// (d_in <= 512) skips the first level: the row block's sums go from the warps to the CTA's shared
// memory, with no fence, ticket or reload.
template <bool kDirect>
__global__ void __launch_bounds__(kHeadThreads) recall_head_kernel(const __grid_constant__ HeadParams p)
{
    __shared__ __align__(16) float s_x[kHeadBT][kHeadKT];
    __shared__ float s_h[kHeadRows][kMaxHeadBatch];
    __shared__ int s_last;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rb = blockIdx.x, ks = blockIdx.y, n_rb = gridDim.x, n_ks = gridDim.y;
    const int j = rb * kHeadRows + warp;
    const int d_in = p.d_ext + p.d_attn;
    const int k0 = ks * kHeadKT;
    constexpr bool direct = kDirect;   // one K slice: the row block's sums stay in the CTA
    // this lane's 16 weights of row j: features k0 + c*128 + lane*4 + e
    float w[4][4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int i = k0 + c * 128 + lane * 4;
        if (j < p.d_hidden && p.vec4 && i < d_in) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(p.W1 + (size_t)j * p.w1_stride + i));
            w[c][0] = v.x; w[c][1] = v.y; w[c][2] = v.z; w[c][3] = v.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                w[c][e] = (j < p.d_hidden && i + e < d_in) ? __ldg(p.W1 + (size_t)j * p.w1_stride + i + e) : 0.f;
        }
    }
    // the weights above are parameters and are already in flight; the Local output read below comes
    // from the previous kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int b0 = 0; b0 < p.batch; b0 += kHeadBT) {
        if (b0) __syncthreads();
        // stage x[b0 .. b0+16)[k0 .. k0+512): every load of the tile is in flight together
        if (p.vec4) {
#pragma unroll
            for (int t = 0; t < kHeadBT * kHeadKT / 4 / kHeadThreads; ++t) {
                const int idx = tid + t * kHeadThreads;
                const int u = idx / (kHeadKT / 4), q = idx - u * (kHeadKT / 4);
                const bool ok = b0 + u < p.batch && k0 + q * 4 < d_in;
                reinterpret_cast<float4*>(&s_x[u][0])[q] =
                    ok ? head_x4(p, b0 + u, k0 + q * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        } else {
            for (int idx = tid; idx < kHeadBT * kHeadKT; idx += kHeadThreads) {
                const int u = idx / kHeadKT, i = idx - u * kHeadKT;
                s_x[u][i] = (b0 + u < p.batch && k0 + i < d_in) ? head_x(p, b0 + u, k0 + i) : 0.f;
            }
        }
        __syncthreads();
        float acc[kHeadBT];
#pragma unroll
        for (int u = 0; u < kHeadBT; ++u) {
            float a = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float4 x = reinterpret_cast<const float4*>(&s_x[u][0])[c * 32 + lane];
                a = fmaf(w[c][0], x.x, a);
                a = fmaf(w[c][1], x.y, a);
                a = fmaf(w[c][2], x.z, a);
                a = fmaf(w[c][3], x.w, a);
            }
            acc[u] = a;
        }
#pragma unroll
        for (int u = 0; u < kHeadBT; ++u) {
            float a = acc[u];
            for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0 && b0 + u < p.batch && j < p.d_hidden) {
                if (direct)
                    s_h[warp][b0 + u] = a;
                else
                    __stcg(p.pre + ((size_t)ks * p.d_hidden + j) * p.max_batch + b0 + u, a);
            }
        }
    }
    if (!direct) {
        // ---- row block complete?  (last of its n_ks K slices)
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int old = atomicAdd(p.rb_tickets + rb, 1);
            s_last = (old == n_ks - 1);
            if (s_last) p.rb_tickets[rb] = 0;
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
    } else {
        __syncthreads();
    }
    if (p.pre_out) {  // column-split head: this rank's share of W1 x, K slices added in order
        for (int e = tid; e < kHeadRows * p.batch; e += kHeadThreads) {
            const int b = e / kHeadRows, jj = rb * kHeadRows + (e - b * kHeadRows);
            if (jj >= p.d_hidden) continue;
            float a = 0.f;
            if (direct)
                a = s_h[e - b * kHeadRows][b];
            else
                for (int s = 0; s < n_ks; ++s) a += __ldcg(p.pre + ((size_t)s * p.d_hidden + jj) * p.max_batch + b);
            p.pre_out[(size_t)b * p.d_hidden + jj] = a;
        }
        return;
    }
    if (direct) {
        for (int e = tid; e < kHeadRows * p.batch; e += kHeadThreads) {
            const int r = e / p.batch, b = e - r * p.batch;
            const int jj = rb * kHeadRows + r;
            float hv = 0.f;
            if (jj < p.d_hidden) {
                const float a = __ldg(p.b1 + jj) + s_h[r][b];
                hv = __ldg(p.w2 + jj) * (a / (1.f + expf(-a)));
            }
            s_h[r][b] = hv;   // each element is read and written by its own thread
        }
    } else {
        for (int e = tid; e < kHeadRows * p.batch; e += kHeadThreads) {
            const int r = e / p.batch, b = e - r * p.batch;
            const int jj = rb * kHeadRows + r;
            float hv = 0.f;
            if (jj < p.d_hidden) {
                float a = __ldg(p.b1 + jj);
                for (int s = 0; s < n_ks; ++s) a += __ldcg(p.pre + ((size_t)s * p.d_hidden + jj) * p.max_batch + b);
                hv = __ldg(p.w2 + jj) * (a / (1.f + expf(-a)));
            }
            s_h[r][b] = hv;
        }
    }
    __syncthreads();
    for (int b = tid; b < p.batch; b += kHeadThreads) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < kHeadRows; ++r) s += s_h[r][b];
        __stcg(p.partial + (size_t)rb * p.max_batch + b, s);
    }
    // ---- head complete?  (last of the n_rb row blocks)
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int old = atomicAdd(p.ticket, 1);
        s_last = (old == n_rb - 1);
        if (s_last) *p.ticket = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // one warp per request: lanes take the row blocks' sums 32 apart, then a fixed shuffle tree
    for (int b = warp; b < p.batch; b += kHeadRows) {
        float zp = 0.f;
        for (int c = lane; c < n_rb; c += 32) zp += __ldcg(p.partial + (size_t)c * p.max_batch + b);
        for (int o = 16; o; o >>= 1) zp += __shfl_xor_sync(0xffffffffu, zp, o);
        if (lane == 0) {
            const float z = __ldg(p.b2) + zp;
            const float score = 1.f / (1.f + expf(-z));
            uint8_t f;
            if (p.override_flags)
                f = p.override_flags[b] ? 1 : 0;
            else
                f = (!isfinite(z) || score > p.threshold) ? 1 : 0;
            p.scores[b] = score;
            if (p.logits) p.logits[b] = z;
            p.flags[b] = f;
            if (p.counters) {
                p.counters[2 * b] += 1;
                p.counters[2 * b + 1] += f;
            }
        }
    }
}

// Second half of a column-split head: pre_sum[b][j] holds W1 x summed over the ranks.  One warp
// per request; lanes take hidden units 32 apart and a fixed shuffle tree adds them, so every
// rank that holds the same pre_sum takes the same decision.
__global__ void __launch_bounds__(kHeadThreads) recall_finalize_kernel(const __grid_constant__ HeadParams p,
                                                                       const float* __restrict__ pre_sum)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * kHeadRows + warp;
    if (b >= p.batch) return;
    float zp = 0.f;
    for (int j = lane; j < p.d_hidden; j += 32) {
        const float a = pre_sum[(size_t)b * p.d_hidden + j] + __ldg(p.b1 + j);
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
        p.scores[b] = score;
        if (p.logits) p.logits[b] = z;
        p.flags[b] = f;
        if (p.counters) {
            p.counters[2 * b] += 1;
            p.counters[2 * b + 1] += f;
        }
    }
}

// no head configured: flags are the override
__global__ void copy_flags_kernel(const uint8_t* __restrict__ ov, uint8_t* __restrict__ flags,
                                  float* scores, float* logits, int32_t* counters, int batch)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < batch; b += gridDim.x * blockDim.x) {
        uint8_t f = ov[b] ? 1 : 0;
        flags[b] = f;
        if (scores) scores[b] = 0.5f;
        if (logits) logits[b] = 0.f;
        if (counters) {
            counters[2 * b] += 1;
            counters[2 * b + 1] += f;
        }
    }
}

__global__ void advance_seq_lens_kernel(int32_t* seq_lens, int batch)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < batch; b += gridDim.x * blockDim.x) seq_lens[b] += 1;
}

int recall_head_grid(int d_hidden) { return (d_hidden + kHeadRows - 1) / kHeadRows; }
int recall_head_ksplits(int d_in) { return d_in > 0 ? (d_in + kHeadKT - 1) / kHeadKT : 1; }

cudaError_t launch_recall_head(const HeadParams& p, cudaStream_t st, bool pdl)
{
    if (p.d_hidden <= 0)
        return launch_ex(copy_flags_kernel, dim3(1), dim3(128), 0, st, pdl, p.override_flags, p.flags, p.scores,
                         p.logits, p.counters, p.batch);
    const int n_ks = recall_head_ksplits(p.d_ext + p.d_attn);
    if (n_ks == 1 && p.batch <= kMaxHeadBatch)
        return launch_ex(recall_head_kernel<true>, dim3(recall_head_grid(p.d_hidden), 1), dim3(kHeadThreads), 0, st, pdl, p);
    return launch_ex(recall_head_kernel<false>, dim3(recall_head_grid(p.d_hidden), n_ks), dim3(kHeadThreads), 0, st, pdl, p);
}

cudaError_t launch_recall_finalize(const HeadParams& p, const float* pre_sum, cudaStream_t st, bool pdl)
{
    return launch_ex(recall_finalize_kernel, dim3((p.batch + kHeadRows - 1) / kHeadRows), dim3(kHeadThreads), 0, st,
                     pdl, p, pre_sum);
}

cudaError_t launch_advance_seq_lens(int32_t* seq_lens, int batch, cudaStream_t st, bool pdl)
{
    return launch_ex(advance_seq_lens_kernel, dim3(1), dim3(128), 0, st, pdl, seq_lens, batch);
}

}  // namespace oda
