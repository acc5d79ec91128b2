// Host-side launch interface between the C-ABI layer (oda_api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace oda {

struct AttnParams;

cudaError_t launch_splitkv_simt(const AttnParams& p, int head_dim, int group, int grid, cudaStream_t st,
                                bool pdl = false);
int occupancy_splitkv_simt(int head_dim, int group);

// TMA + tensor-core variant.  kmap / vmap point at 128-byte CUtensorMap objects (host memory).
bool tma_variant_supported(int head_dim, int64_t layer_stride, int64_t block_stride, int num_layers_phys);
bool encode_kv_map(void* out_map, const void* base, int head_dim, int num_kv_heads, int64_t token_stride,
                   int64_t head_stride, int64_t block_stride, int64_t num_blocks_bound);
cudaError_t launch_splitkv_tma(const AttnParams& p, const void* kmap, const void* vmap, int blocks_per_layer,
                               int head_dim, int group, int grid, cudaStream_t st, bool pdl = false);
int occupancy_splitkv_tma(int head_dim, int group);
int tma_partial_slot_floats();


long long full_head_param_count(int d_model, int d_tower, int d_ff, int n_blocks);
size_t full_head_scratch_bytes(int d_model, int d_tower, int d_ff, int batch);
cudaError_t launch_full_head(int batch, int d_model, int d_tower, int d_ff, int n_blocks, float eps,
                             const float* params, const float* h_prev, const float* emb, const float* h_local,
                             float threshold, const uint8_t* override_flags, float* scores, float* logits,
                             uint8_t* flags, int32_t* counters, void* scratch, cudaStream_t st, bool pdl,
                             int* launches, int variant, int32_t* status, int phase = 0);
// the same head as one persistent cooperative kernel (batch <= kFullHeadFusedMaxBatch)
constexpr int kFullHeadFusedMaxBatch = 4;
constexpr int kFullHeadFusedSmem = 230400;    // dynamic shared memory of the fused head (stage input + ring + control)
long long full_head_fused_x_floats(int batch, int d_model, int T, int F);
int full_head_fused_grid();
cudaError_t launch_full_head_fused(int grid, int batch, int d_model, int T, int F, int n_blocks, float eps,
                                   const float* params, const float* h_prev, const float* emb, const float* h_local,
                                   float threshold, const uint8_t* override_flags, float* scores, float* logits,
                                   uint8_t* flags, int32_t* counters, float* abc, float* z, float* h, int32_t* sync,
                                   int32_t* status, cudaStream_t st);

struct LayerInfo;
cudaError_t launch_write_current_kv(const void* k_cur, const void* v_cur, const uint8_t* mask, void* k_cache,
                                    void* v_cache, const int32_t* block_table, const int32_t* seq_lens,
                                    const LayerInfo* layers, int num_layers, int batch, int num_kv_heads,
                                    int head_dim, int max_blocks_per_seq, int64_t layer_stride,
                                    int64_t block_stride, int64_t token_stride, int64_t head_stride,
                                    int32_t* status, cudaStream_t st, bool pdl = false);
// Per-step inputs that live in pinned host memory, pulled into their staging areas by one kernel
// (plain loads over the bus) instead of one copy-engine transfer each.
struct StageIn {
    const void* src[4];   // device views of the host buffers (16-byte aligned where bytes >= 16)
    void* dst[4];
    long long bytes[4];   // 0: unused
};
cudaError_t launch_stage_in(const StageIn& s, cudaStream_t st, bool pdl);

cudaError_t launch_select_rows(const void* local, const void* full, const uint8_t* flags, void* out, int batch,
                               size_t row_bytes, cudaStream_t st, bool pdl = false);

cudaError_t launch_merge_partials(const float* parts_out, const float* parts_lse, const int32_t* part_tokens,
                                  const uint8_t* flags, const LayerInfo* layers, float* out, float* lse, int n_parts, int layer_begin,
                                  int layer_end, int batch, int q_heads, int head_dim, int num_layers,
                                  cudaStream_t st, bool pdl = false);

struct HeadParams {
    const float* feat_ext;      // [B, d_ext] or nullptr
    const void* attn_out;       // [B, d_attn] fp32 or bf16, or nullptr
    const float *W1, *b1, *w2, *b2;
    const uint8_t* override_flags;
    float* scores;
    float* logits;
    uint8_t* flags;
    int32_t* counters;
    float* partial;             // [row blocks][max_batch] scratch
    float* pre;                 // [K slices][d_hidden][max_batch] partial pre-activations
    int32_t* ticket;            // one int, zero between launches
    int32_t* rb_tickets;        // [row blocks], zero between launches
    float* pre_out;             // non-null: stop after W1 x and write [batch][d_hidden] sums (no bias)
    int64_t w1_stride;          // floats between rows of W1 (d_ext + d_attn unless W1 is a column slice)
    int32_t batch, d_ext, d_attn, d_hidden, attn_bf16, max_batch;
    int32_t vec4;               // 128-bit loads are legal: widths multiples of 4, pointers 16-byte aligned
    float threshold;
};

constexpr int kMaxHeadBatch = 128;

// the tensor-parallel decision with its exchange fused in (recall_exchange.cu)
constexpr int kExchangeThreads = 256;
constexpr int kExchangeMaxWorld = 8;
struct ExchangeRank {            // one rank's own buffers
    const float* pre_local;      // [batch][d_hidden] this rank's share of W1 x
    float* scores;
    float* logits;               // nullable
    uint8_t* flags;
    int32_t* counters;           // nullable
};
struct ExchangeParams {
    ExchangeRank ranks[kExchangeMaxWorld];   // the ranks this launch runs: one in production
    float* recv[kExchangeMaxWorld];          // recv[r]: rank r's receive buffer [2][world][batch * d_hidden]
    uint32_t* arrived[kExchangeMaxWorld];    // arrived[r]: rank r's arrival flags [world]
    const float *b1, *w2, *b2;
    const uint8_t* override_flags;
    int32_t* status;
    unsigned long long timeout_ns;
    int32_t batch, d_hidden, world, rank_base;
    uint32_t epoch;
    float threshold;
};
cudaError_t launch_recall_exchange(const ExchangeParams& p, int n_local, cudaStream_t st, bool pdl = false);

// sequence-sharded Full pass: exchange of (out, lse) rows fused with their combination
constexpr int kMergeBlocks = 64;           // row blocks, each with its own arrival flag
struct MergeExchangeRank {
    const float* part_out;       // [L, batch, q_heads, D] this rank's rows
    const float* part_lse;       // [L, batch, q_heads]
    const int32_t* tokens_local; // [batch] positions this rank holds (nullable: all > 0)
    const uint8_t* flags;        // [batch] gate (nullable: all requests)
    float* out;
    float* lse;                  // nullable
};
struct MergeExchangeParams {
    MergeExchangeRank ranks[kExchangeMaxWorld];
    float* recv_out[kExchangeMaxWorld];    // rank r's buffer [2][world][L*batch*q_heads][D]
    float* recv_lse[kExchangeMaxWorld];    // [2][world][L*batch*q_heads]
    uint32_t* arrived[kExchangeMaxWorld];  // [world][kMergeBlocks]
    const LayerInfo* layers;
    int32_t* status;
    unsigned long long timeout_ns;
    int32_t batch, q_heads, num_layers, layer_begin, layer_end, world, rank_base;
    uint32_t epoch;
};
cudaError_t launch_merge_exchange(const MergeExchangeParams& p, int n_local, int head_dim, cudaStream_t st, bool pdl = false);

int recall_head_grid(int d_hidden);
int recall_head_ksplits(int d_in);
cudaError_t launch_recall_head(const HeadParams& p, cudaStream_t st, bool pdl = false);
// z = b2 + w2 . SiLU(pre_sum + b1) and the decision, from summed first-layer products [batch][d_hidden]
cudaError_t launch_recall_finalize(const HeadParams& p, const float* pre_sum, cudaStream_t st, bool pdl = false);
cudaError_t launch_advance_seq_lens(int32_t* seq_lens, int batch, cudaStream_t st, bool pdl = false);

}  // namespace oda
