// Host-side launch interface between the C-ABI layer (oda_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace oda {

struct AttnParams;

cudaError_t launch_splitkv_simt(const AttnParams& p, int head_dim, int group, int grid, cudaStream_t st);
int occupancy_splitkv_simt(int head_dim, int group);

struct HeadParams {
    const float* feat_ext;      // [B, d_ext] or nullptr
    const void* attn_out;       // [B, d_attn] fp32 or bf16, or nullptr
    const float *W1, *b1, *w2, *b2;
    const uint8_t* override_flags;
    float* scores;
    float* logits;
    uint8_t* flags;
    int32_t* counters;
    float* partial;             // [grid][max_batch] scratch
    int32_t* ticket;            // one int, zero between launches
    int32_t batch, d_ext, d_attn, d_hidden, attn_bf16, max_batch;
    float threshold;
};

int recall_head_grid(int d_hidden);
cudaError_t launch_recall_head(const HeadParams& p, cudaStream_t st);
cudaError_t launch_advance_seq_lens(int32_t* seq_lens, int batch, cudaStream_t st);

}  // namespace oda
