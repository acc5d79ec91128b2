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
