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

constexpr int kHeadWarps = 4;
constexpr int kHeadBT = 8;  // requests per register tile

__device__ __forceinline__ float head_x(const HeadParams& p, int b, int i)
{
    if (i < p.d_ext) return __ldg(p.feat_ext + (size_t)b * p.d_ext + i);
    size_t k = (size_t)b * p.d_attn + (i - p.d_ext);
    if (p.attn_bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p.attn_out)[k]);
    return __ldcg(reinterpret_cast<const float*>(p.attn_out) + k);
}

__global__ void __launch_bounds__(kHeadWarps * 32) recall_head_kernel(const __grid_constant__ HeadParams p)
{
    __shared__ float s_h[kHeadWarps][256];
    __shared__ int s_last;
    asm volatile("griddepcontrol.wait;" ::: "memory");  // the Local output it reads comes from the previous kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j = blockIdx.x * kHeadWarps + warp;
    const int d_in = p.d_ext + p.d_attn;
    for (int b0 = 0; b0 < p.batch; b0 += kHeadBT) {
        float acc[kHeadBT];
#pragma unroll
        for (int u = 0; u < kHeadBT; ++u) acc[u] = 0.f;
        if (j < p.d_hidden) {
            const float* wrow = p.W1 + (size_t)j * d_in;
            for (int i = lane; i < d_in; i += 32) {
                const float w = __ldg(wrow + i);
#pragma unroll
                for (int u = 0; u < kHeadBT; ++u)
                    if (b0 + u < p.batch) acc[u] = fmaf(w, head_x(p, b0 + u, i), acc[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kHeadBT; ++u) {
            float a = acc[u];
            for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0 && b0 + u < p.batch) {
                float hv = 0.f;
                if (j < p.d_hidden) {
                    a += __ldg(p.b1 + j);
                    hv = __ldg(p.w2 + j) * (a / (1.f + expf(-a)));
                }
                s_h[warp][b0 + u] = hv;
            }
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < p.batch; b += blockDim.x) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kHeadWarps; ++w) s += s_h[w][b];
        __stcg(p.partial + (size_t)blockIdx.x * p.max_batch + b, s);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        int old = atomicAdd(p.ticket, 1);
        s_last = (old == (int)gridDim.x - 1);
        if (s_last) *p.ticket = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int b = threadIdx.x; b < p.batch; b += blockDim.x) {
        float z = __ldg(p.b2);
        for (int c = 0; c < (int)gridDim.x; ++c) z += __ldcg(p.partial + (size_t)c * p.max_batch + b);
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

int recall_head_grid(int d_hidden) { return (d_hidden + kHeadWarps - 1) / kHeadWarps; }

cudaError_t launch_recall_head(const HeadParams& p, cudaStream_t st, bool pdl)
{
    if (p.d_hidden <= 0)
        return launch_ex(copy_flags_kernel, dim3(1), dim3(128), 0, st, pdl, p.override_flags, p.flags, p.scores,
                         p.logits, p.counters, p.batch);
    return launch_ex(recall_head_kernel, dim3(recall_head_grid(p.d_hidden)), dim3(kHeadWarps * 32), 0, st, pdl, p);
}

cudaError_t launch_advance_seq_lens(int32_t* seq_lens, int batch, cudaStream_t st, bool pdl)
{
    return launch_ex(advance_seq_lens_kernel, dim3(1), dim3(128), 0, st, pdl, seq_lens, batch);
}

}  // namespace oda
