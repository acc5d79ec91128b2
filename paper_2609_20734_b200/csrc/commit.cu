// Selected-state commit (Algorithm 1, line 8): one fused kernel writes the current token's K/V
// of every layer into the paged cache at position seq_len-1 (the paper's "fused commitment"
// across layers), and one selects the per-request hidden rows of the chosen branch.  Both are
// a few hundred KiB of traffic: launch-bound, so they are single launches over all layers.
#include "launch_ex.cuh"
#include "oda_device.cuh"
#include "oda_launch.h"

namespace oda {

__global__ void __launch_bounds__(256)
write_current_kv_kernel(const uint4* __restrict__ k_cur, const uint4* __restrict__ v_cur,
                        const uint8_t* __restrict__ mask, __nv_bfloat16* k_cache, __nv_bfloat16* v_cache,
                        const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                        const LayerInfo* __restrict__ layers, int num_layers, int batch, int num_kv_heads,
                        int head_dim, int max_blocks_per_seq, int64_t layer_stride, int64_t block_stride,
                        int64_t token_stride, int64_t head_stride, int32_t* status)
{
    griddep_wait();
    griddep_launch_dependents();
    const int vec_per_row = head_dim / 8;  // 16-byte pieces of one (layer, request, head) vector
    const long long total = (long long)num_layers * batch * num_kv_heads * vec_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int piece = (int)(i % vec_per_row);
        long long r = i / vec_per_row;
        const int g = (int)(r % num_kv_heads);
        r /= num_kv_heads;
        const int b = (int)(r % batch);
        const int l = (int)(r / batch);
        if (mask && !mask[b]) continue;
        const int t = seq_lens[b];
        if (t < 1 || t > max_blocks_per_seq * kPage) {
            atomicOr(status, kStatusBadSeqLen);
            continue;
        }
        const int blk = block_table[(size_t)b * max_blocks_per_seq + (t - 1) / kPage];
        const size_t dst = (size_t)layers[l].kv_index * layer_stride + (size_t)blk * block_stride +
                           (size_t)((t - 1) % kPage) * token_stride + (size_t)g * head_stride + (size_t)piece * 8;
        *reinterpret_cast<uint4*>(k_cache + dst) = k_cur[i];
        *reinterpret_cast<uint4*>(v_cache + dst) = v_cur[i];
    }
}

__global__ void __launch_bounds__(256)
select_rows_kernel(const uint4* __restrict__ local, const uint4* __restrict__ full, const uint8_t* __restrict__ flags,
                   uint4* __restrict__ out, int batch, int vec_per_row)
{
    griddep_wait();
    griddep_launch_dependents();
    const long long total = (long long)batch * vec_per_row;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int b = (int)(i / vec_per_row);
        out[i] = flags[b] ? full[i] : local[i];
    }
}

// Sequence-sharded Full pass: part r holds softmax attention over rank r's slice of the history
// as (normalised out_r, lse_r).  The whole-history result is the log-sum-exp combination
//   lse = M + ln sum_r e^{lse_r - M},  out = sum_r e^{lse_r - lse} out_r,  M = max_r lse_r,
// parts added in rank order.  A part with part_tokens[r][b] == 0 or lse = -inf (the rank held
// none of the request) adds nothing.  One warp per (layer, request, query head) row; V floats per lane.
template <int V>
__global__ void __launch_bounds__(256)
merge_partials_kernel(const float* __restrict__ parts_out, const float* __restrict__ parts_lse,
                      const int32_t* __restrict__ part_tokens, const uint8_t* __restrict__ flags,
                      const LayerInfo* __restrict__ layers, float* __restrict__ out,
                      float* __restrict__ lse, int n_parts, int layer_begin, int layer_end, int batch, int q_heads,
                      int num_layers, int max_batch_rows)
{
    griddep_wait();
    griddep_launch_dependents();
    constexpr int D = V * 32;
    const int lane = threadIdx.x & 31;
    const long long rows = (long long)(layer_end - layer_begin) * batch * q_heads;
    const long long part_rows = (long long)num_layers * max_batch_rows * q_heads;
    for (long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < rows;
         w += ((long long)gridDim.x * blockDim.x) >> 5) {
        const int h = (int)(w % q_heads);
        const int b = (int)((w / q_heads) % batch);
        const int l = layer_begin + (int)(w / ((long long)q_heads * batch));
        if (!layers[l].gated || (flags && !flags[b])) continue;
        const long long row = ((long long)l * max_batch_rows + b) * q_heads + h;
        float m = -INFINITY;
        unsigned long long have = 0;  // parts that hold some of this request (n_parts <= 64)
        for (int r = 0; r < n_parts; ++r) {
            if (part_tokens && part_tokens[r * batch + b] <= 0) continue;
            const float lr = parts_lse[r * part_rows + row];
            if (lr == -INFINITY) continue;
            have |= 1ull << r;
            m = fmaxf(m, lr);
        }
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.f;
        float sum = 0.f;
        if (have) {
            for (int r = 0; r < n_parts; ++r) {
                if (!((have >> r) & 1)) continue;
                const float lr = parts_lse[r * part_rows + row];
                const float wgt = expf(lr - m);
                sum += wgt;
                const float* src = parts_out + (r * part_rows + row) * D + lane * V;
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = fmaf(wgt, src[e], acc[e]);
            }
        }
        const float inv = sum > 0.f ? 1.f / sum : 0.f;
        float* dst = out + row * D + lane * V;
#pragma unroll
        for (int e = 0; e < V; ++e) dst[e] = acc[e] * inv;
        if (lse && lane == 0) lse[row] = sum > 0.f ? m + logf(sum) : -INFINITY;
    }
}

cudaError_t launch_merge_partials(const float* parts_out, const float* parts_lse, const int32_t* part_tokens,
                                  const uint8_t* flags, const LayerInfo* layers, float* out, float* lse, int n_parts, int layer_begin,
                                  int layer_end, int batch, int q_heads, int head_dim, int num_layers,
                                  cudaStream_t st, bool pdl)
{
    const long long rows = (long long)(layer_end - layer_begin) * batch * q_heads;
    int grid = (int)((rows + 7) / 8);
    if (grid > 1184) grid = 1184;
    if (grid < 1) grid = 1;
    if (head_dim == 128)
        return launch_ex(merge_partials_kernel<4>, dim3(grid), dim3(256), 0, st, pdl, parts_out, parts_lse, part_tokens,
                         flags, layers, out, lse, n_parts, layer_begin, layer_end, batch, q_heads, num_layers, batch);
    return launch_ex(merge_partials_kernel<2>, dim3(grid), dim3(256), 0, st, pdl, parts_out, parts_lse, part_tokens, flags, layers,
                     out, lse, n_parts, layer_begin, layer_end, batch, q_heads, num_layers, batch);
}

__global__ void __launch_bounds__(256) stage_in_kernel(const __grid_constant__ StageIn s)
{
    griddep_wait();
    griddep_launch_dependents();  // the kernels that follow start their own set-up while this one copies
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nth = (long long)gridDim.x * blockDim.x;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const long long n16 = s.bytes[k] >> 4;
        const uint4* src = static_cast<const uint4*>(s.src[k]);
        uint4* dst = static_cast<uint4*>(s.dst[k]);
        for (long long i = tid; i < n16; i += nth) dst[i] = src[i];
        const long long tail = s.bytes[k] & 15;   // fewer than 16 bytes left: byte by byte
        if (tid < tail)
            static_cast<uint8_t*>(s.dst[k])[(n16 << 4) + tid] = static_cast<const uint8_t*>(s.src[k])[(n16 << 4) + tid];
    }
}

cudaError_t launch_stage_in(const StageIn& s, cudaStream_t st, bool pdl)
{
    long long most = 0;
    for (int k = 0; k < 4; ++k) most = most > s.bytes[k] ? most : s.bytes[k];
    int grid = (int)((most / 16 + 255) / 256);   // every 16-byte piece of the largest input in flight at once
    if (grid > 592) grid = 592;
    if (grid < 1) grid = 1;
    return launch_ex(stage_in_kernel, dim3(grid), dim3(256), 0, st, pdl, s);
}

cudaError_t launch_write_current_kv(const void* k_cur, const void* v_cur, const uint8_t* mask, void* k_cache,
                                    void* v_cache, const int32_t* block_table, const int32_t* seq_lens,
                                    const LayerInfo* layers, int num_layers, int batch, int num_kv_heads,
                                    int head_dim, int max_blocks_per_seq, int64_t layer_stride,
                                    int64_t block_stride, int64_t token_stride, int64_t head_stride,
                                    int32_t* status, cudaStream_t st, bool pdl)
{
    const long long total = (long long)num_layers * batch * num_kv_heads * (head_dim / 8);
    int grid = (int)((total + 255) / 256);
    if (grid > 592) grid = 592;
    if (grid < 1) grid = 1;
    return launch_ex(write_current_kv_kernel, dim3(grid), dim3(256), 0, st, pdl,
                     static_cast<const uint4*>(k_cur), static_cast<const uint4*>(v_cur), mask,
                     static_cast<__nv_bfloat16*>(k_cache), static_cast<__nv_bfloat16*>(v_cache), block_table,
                     seq_lens, layers, num_layers, batch, num_kv_heads, head_dim, max_blocks_per_seq,
                     layer_stride, block_stride, token_stride, head_stride, status);
}

cudaError_t launch_select_rows(const void* local, const void* full, const uint8_t* flags, void* out, int batch,
                               size_t row_bytes, cudaStream_t st, bool pdl)
{
    const int vec = (int)(row_bytes / 16);
    const long long total = (long long)batch * vec;
    int grid = (int)((total + 255) / 256);
    if (grid > 592) grid = 592;
    if (grid < 1) grid = 1;
    return launch_ex(select_rows_kernel, dim3(grid), dim3(256), 0, st, pdl, static_cast<const uint4*>(local),
                     static_cast<const uint4*>(full), flags, static_cast<uint4*>(out), batch, vec);
}

}  // namespace oda
