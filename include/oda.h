/*
 * oda.h -- C ABI of the B200 On-Demand-Attention (ODA) decode library.
 *
 * One decode step of ODA on an attention stack over a block-table paged bf16 KV
 * cache (Algorithm 1, lines 1-7, of the paper "On-Demand Attention"):
 *   1. Local attention for every request over the access set of Eq. 1,
 *        S^L = {first min(s,t) positions} U {last min(w,t) positions},
 *   2. a recall head scores the post-Local state and writes one flag per request,
 *   3. Full attention (S^F = all t positions) is recomputed only for flagged
 *      requests on the gated layers, and replaces their Local output
 *      (selected-state rule of the appendix on selected-state execution).
 * The flag never leaves the device: step 3 reads it there.
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment
 *     says "host".  The library allocates no device memory; its scratch is the
 *     workspace the caller hands to oda_set_workspace().
 *   - All work is enqueued on the stream argument (a cudaStream_t passed as
 *     void*); nothing synchronises except oda_read_device_status() and
 *     oda_step_host().  The device entry points may be stream-captured.
 *   - Positions are 0-based here: request b has t = seq_lens[b] >= 1 positions
 *     0..t-1, the current token's K/V already stored at position t-1.
 *   - KV cache element (layer, block, token slot, kv head, d) of k_cache / v_cache
 *     is at  kv_index(layer)*kv_layer_stride + block*kv_block_stride +
 *     slot*kv_token_stride + head*kv_head_stride + d   (bf16 elements).  The d
 *     values are contiguous, every stride is a multiple of 8 elements and the
 *     base pointers are 16-byte aligned.  block = block_table[b*max_blocks_per_seq
 *     + position/16].  Entries past ceil(t/16) are never read.
 *   - q is [layers, batch, q_heads, head_dim] bf16; query head h reads KV head
 *     h / (q_heads / kv_heads).  out has the same shape in fp32 (or bf16, see
 *     out_dtype), lse is [layers, batch, q_heads] fp32 (natural log of the softmax
 *     denominator, including the maximum).  The layer axis of q/out/lse always
 *     spans all num_layers; a call touches rows layer_begin..layer_end-1.
 *   - Errors a host check can see return a status with nothing enqueued.  Problems
 *     only the device can see (seq_len < 1) set a sticky status word in the
 *     workspace, readable with oda_read_device_status(); the kernels never trap.
 *   - One context must not be used from two streams at once (the workspace is
 *     shared scratch).
 */
#ifndef ODA_H
#define ODA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct oda_ctx oda_ctx_t; /* opaque, host-owned */

typedef enum {
    ODA_OK = 0,
    ODA_ERR_INVALID_ARG = 1,   /* null pointer, bad range, bad shape */
    ODA_ERR_UNSUPPORTED = 2,   /* a shape this build has no kernel for */
    ODA_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or too small */
    ODA_ERR_CUDA = 4,          /* a CUDA runtime call failed */
    ODA_ERR_DEVICE_STATUS = 5  /* the device status word is non-zero */
} oda_status_t;

/* Which attention kernel runs (evidence for the design choice comes from timing both). */
enum {
    ODA_VARIANT_AUTO = 0,
    ODA_VARIANT_SIMT = 1,  /* fp32 CUDA-core math, direct 128-bit global loads, warp-shuffle reductions */
    ODA_VARIANT_TMA_MMA = 2 /* TMA-staged shared-memory ring, bf16 tensor-core GQA tile, fp32 accumulate */
};

typedef struct {
    int32_t num_layers;         /* 1..256 */
    int32_t num_q_heads;        /* multiple of num_kv_heads; group size 1, 2, 4 or 8 */
    int32_t num_kv_heads;
    int32_t head_dim;           /* 64 or 128 */
    int32_t block_size;         /* tokens per KV block: 16 */
    int32_t max_batch;          /* 1..128 */
    int32_t max_blocks_per_seq; /* row length of block_table */
    int32_t out_dtype;          /* 0 = fp32, 1 = bf16 */
    float sm_scale;             /* logit scale; 0 => 1/sqrt(head_dim) */
    int32_t variant;            /* ODA_VARIANT_* */
    /* host arrays [num_layers], copied at create.  Eq. 1: window w >= 1 (includes the
     * current token), sinks s >= 0.  gated: 1 = ODA layer (Local, Full on recall),
     * 0 = fixed-window layer (always Local).  kv_index (nullable => identity): which
     * layer slice of the cache holds this layer's K/V.  A context takes at most four distinct
     * (window, sinks, gated) combinations over its layers (ODA_ERR_UNSUPPORTED beyond that). */
    const int32_t* layer_window;
    const int32_t* layer_sinks;
    const uint8_t* layer_gated;
    const int32_t* layer_kv_index;
    int64_t kv_layer_stride, kv_block_stride, kv_token_stride, kv_head_stride; /* bf16 elements */
    /* Recall head x = [feat_ext (head_d_ext) ; flattened Local output of the last gated layer
     * (q_heads*head_dim, present iff head_use_attn_out)], hidden width head_d_hidden.
     * head_d_hidden = 0: no head (oda_step then needs override_flags). */
    int32_t head_d_ext;
    int32_t head_use_attn_out;
    int32_t head_d_hidden;
    int32_t options;            /* bit 0: launch every kernel fully serialised (no programmatic
                                 * dependent launch between the kernels of a step).
                                 * bit 1: the gated pass reads only the positions Local did not,
                                 * S^F \ S^L = [min(s,t), t-w), and merges them with the Local result
                                 * already in out/lse by log-sum-exp.  That is exact only when the
                                 * Full branch's queries are the Local branch's (an attention-only
                                 * stack, or the first layer of a model): q_full must equal q_local,
                                 * out/lse must hold the Local pass of the same step, lse must not be
                                 * NULL in oda_full_decode_gated.  The paper's runtime recomputes Full
                                 * from scratch; this variant makes a recalled step cost exactly one
                                 * Full pass in bytes.  TMA variant only.
                                 * bit 2: oda_full_decode_gated skips a flagged request whose seq_len is
                                 * 0 (its rows stay untouched) instead of setting the device status:
                                 * for a rank of a sequence-sharded pass that holds none of a short
                                 * request (see oda_merge_partials). */
} oda_config_t;

/* Lifetime.  oda_create validates and copies the config (host only, no device work).
 * Errors: INVALID_ARG, UNSUPPORTED. */
oda_status_t oda_create(const oda_config_t* cfg, oda_ctx_t** out_ctx);
void oda_destroy(oda_ctx_t* ctx);

/* Scratch sizing: bytes the workspace must have for this config on the current device. */
oda_status_t oda_workspace_bytes(const oda_ctx_t* ctx, size_t* bytes);
/* Hands the library its scratch (256-byte aligned, caller-owned, must outlive the ctx's use).
 * Initialises it (tickets, status, layer table) on `stream` and waits for that to finish. */
oda_status_t oda_set_workspace(oda_ctx_t* ctx, void* dev_ptr, size_t bytes, void* stream);

/*
 * Optional: keep part of the Local pass's working set in L2 between steps.  A decode loop reads
 * nearly the same windows step after step; when they are larger than L2 a plain stream evicts
 * every line before its next use.  With a budget set, the Local pass loads the pages of as many
 * leading layers as fit `bytes` (batch x kv heads x (window + sinks) x head_dim x 4 bytes per
 * layer) with an L2 evict-last hint and streams the rest evict-first as before, so that part of
 * the next step's reads hits L2.  About half of the L2 is a good budget; 0 (the default) turns it
 * off.  Host-only call, takes effect at the next launch (captured graphs keep what they were
 * captured with).  The paper has no counterpart (its runtime copies the window into a ring
 * workspace instead).
 */
oda_status_t oda_set_cache_resident_bytes(oda_ctx_t* ctx, size_t bytes);

/*
 * Optional calibration of the split of work across SMs.  HBM bandwidth is not shared evenly among
 * the SMs of a GPU (on a B200, equal spans of KV finish +-10 % apart, in a pattern that is a fixed
 * property of the chip).  Between oda_calibration_begin() and oda_calibration_end() the attention
 * kernels record, per SM, how many pages they streamed in how much time; run one or more large
 * passes in between (e.g. one oda_full_decode_gated with every request flagged: only launches
 * that give every CTA work are counted).  oda_calibration_end() synchronises the stream, and from
 * then on cuts the work of large attention launches in proportion to the measured rate of the SM
 * each CTA runs on, so that all CTAs finish together.  Results stay deterministic (the table is
 * fixed once measured) and agree with the uncalibrated ones up to summation order.  Has no effect
 * for the SIMT variant.  oda_set_workspace() discards the table.  Do not capture these two calls.
 */
oda_status_t oda_calibration_begin(oda_ctx_t* ctx, void* stream);
oda_status_t oda_calibration_end(oda_ctx_t* ctx, void* stream);
/* slowest / fastest SM streaming rate found by the calibration (0 if not calibrated) */
double oda_calibration_spread(const oda_ctx_t* ctx);

/*
 * Local pass (Eq. 1, S^L) for layers [layer_begin, layer_end) and requests 0..batch-1:
 * split-KV partials + log-sum-exp merge.  Writes out/lse rows of those layers.
 * lse may be NULL.  batch = 0 is a no-op.
 */
oda_status_t oda_local_decode(oda_ctx_t* ctx, int32_t layer_begin, int32_t layer_end, int32_t batch,
                              const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* block_table, const int32_t* seq_lens, void* out,
                              float* lse, void* stream);

/*
 * Recall score and decision (Eq. 2 reduced to the benchmark's two-layer head; decision rule
 * of Algorithm 1, line 3):  z = w2 . SiLU(W1 x + b1) + b2, score = sigmoid(z),
 * flag = override_flags[b] if override_flags != NULL, else (z nonfinite) or (score > threshold).
 * feat_ext [batch, head_d_ext] fp32 (NULL iff head_d_ext = 0); attn_out_last [batch, q_heads,
 * head_dim] in out_dtype (NULL iff !head_use_attn_out); W1 [d_hidden, d_in] row-major fp32.
 * Writes scores [batch] fp32, logits [batch] fp32 (nullable), flags [batch] u8 and, if
 * counters != NULL ([batch,2] i32), counters[b] += {1, flag}.
 */
oda_status_t oda_recall_score(oda_ctx_t* ctx, int32_t batch, const float* feat_ext,
                              const void* attn_out_last, const float* W1, const float* b1,
                              const float* w2, const float* b2, float threshold,
                              const uint8_t* override_flags, float* scores, float* logits,
                              uint8_t* flags, int32_t* counters, void* stream);

/*
 * The same head split for KV-head tensor parallelism (the paper runs on one GPU; this is how its
 * Algorithm 1 shards when every rank owns num_kv_heads of the model's KV heads, the query heads
 * of their groups, and the matching columns of W1).  A context is created with the RANK's head
 * counts; head_d_ext is non-zero only on the rank that owns the external features.
 *   oda_recall_preact:   pre_out[b][j] = sum over this rank's input columns of W1[j][col] x[b][col]
 *     (no bias).  W1_cols points at the rank's first column inside row 0 of the full matrix and
 *     w1_row_stride is the full row length in floats.  pre_out [batch, d_hidden] fp32 device.
 *   -- the caller sums pre_out over the ranks (one all-reduce of batch x d_hidden floats) --
 *   oda_recall_finalize: z = w2 . SiLU(pre_sum + b1) + b2 and the decision rule of
 *     oda_recall_score; every rank that holds the same pre_sum writes the same flags.
 * Summation order differs from oda_recall_score, so scores agree to fp32 rounding, not bitwise.
 * One launch each; neither synchronises.
 */
oda_status_t oda_recall_preact(oda_ctx_t* ctx, int32_t batch, const float* feat_ext,
                               const void* attn_out_last, const float* W1_cols, int64_t w1_row_stride,
                               float* pre_out, void* stream);
oda_status_t oda_recall_finalize(oda_ctx_t* ctx, int32_t batch, const float* pre_sum, const float* b1,
                                 const float* w2, const float* b2, float threshold,
                                 const uint8_t* override_flags, float* scores, float* logits,
                                 uint8_t* flags, int32_t* counters, void* stream);

/*
 * The same decision with the exchange inside the kernel (no collective library call): every rank
 * stores its share of W1 x into slot [rank] of every rank's receive buffer (plain peer stores),
 * raises an arrival flag carrying `epoch` in every rank's flag array, waits -- at most timeout_ns
 * (0 => 1 s) -- for all ranks' flags in its own array, adds the shares in rank order and applies
 * oda_recall_finalize's arithmetic.  All ranks therefore take the same decision bit for bit.
 *   recv [world] (host array of device pointers): recv[r] is rank r's receive buffer,
 *     2 * world * batch_max * d_hidden floats, 16-byte aligned, mapped into this GPU's address
 *     space for every r (peer access / symmetric memory); only recv[own rank] is read;
 *   arrived [world] (host array): arrived[r] is rank r's flag array of `world` u32, zero at set-up;
 *   epoch: 1, 2, 3, ... one more on every call, the same on all ranks (buffers alternate by parity;
 *     a rank can run at most one exchange ahead of the slowest);
 *   ranks [n_local] (host array): the buffers of the ranks THIS launch runs, ranks rank_base ..
 *     rank_base + n_local - 1.  In production n_local = 1 (one process per GPU, one CTA).  n_local
 *     > 1 runs several ranks as the CTAs of one cooperative launch on one GPU (the CTAs wait on one
 *     another, so they must be co-resident): that is how the protocol is checked without several GPUs.
 * A wait that runs out sets bit 2 of the device status word and leaves scores / flags untouched.
 * world <= 8.  The caller makes sure every rank of the group issues the call for the same epoch.
 */
typedef struct {
    const float* pre_local; /* [batch, d_hidden]: oda_recall_preact's output on this rank */
    float* scores;
    float* logits;          /* nullable */
    uint8_t* flags;
    int32_t* counters;      /* nullable */
} oda_exchange_rank_t;
oda_status_t oda_recall_finalize_exchange(oda_ctx_t* ctx, int32_t batch, int32_t world, int32_t rank_base,
                                          int32_t n_local, const oda_exchange_rank_t* ranks,
                                          float* const* recv, uint32_t* const* arrived, uint32_t epoch,
                                          uint64_t timeout_ns, const float* b1, const float* w2,
                                          const float* b2, float threshold, const uint8_t* override_flags,
                                          void* stream);

/*
 * Sequence sharding of the gated Full pass (the paper runs on one GPU; this is how the history of
 * Eq. 1's S^F splits over ranks that each hold a range of positions).  Every rank runs
 * oda_full_decode_gated over its own slice (its block table and lengths) and gets, per row,
 * softmax attention over that slice as (out_r, lse_r); the rows of all ranks are gathered into
 * parts_out [n_parts][L, batch, q_heads, D] fp32 and parts_lse [n_parts][L, batch, q_heads] fp32
 * (natural-log lse), and this call combines them for gated layers in [layer_begin, layer_end) and
 * requests with flags[b] != 0 (all requests if flags == NULL):
 *   lse = M + ln sum_r e^{lse_r - M},  out = sum_r e^{lse_r - lse} out_r,  parts in index order.
 * part_tokens [n_parts][batch] i32 (nullable) gives the number of positions each rank holds of each
 * request: a part with 0 positions, or whose lse is -inf, contributes nothing (its rows are never
 * read as numbers that matter, so they may be uninitialised); if no part contributes, out = 0 and
 * lse = -inf.  Other rows of out/lse are not touched.  lse may be NULL.
 * fp32 contexts only (ODA_ERR_UNSUPPORTED otherwise).  One launch; does not synchronise.
 */
oda_status_t oda_merge_partials(oda_ctx_t* ctx, int32_t n_parts, int32_t layer_begin, int32_t layer_end,
                                int32_t batch, const float* parts_out, const float* parts_lse,
                                const int32_t* part_tokens, const uint8_t* flags, void* out, float* lse,
                                void* stream);

/*
 * oda_merge_partials with the exchange inside the kernel, by the protocol of
 * oda_recall_finalize_exchange: the rows are cut into 64 blocks; CTA c of every rank stores its
 * rows of block c (the rank's part_out / part_lse, lse = -inf where tokens_local[b] = 0) into slot
 * [rank] of every rank's receive buffers, raises flag [rank][c] carrying `epoch` in every rank's
 * flag array, waits -- at most timeout_ns (0 => 1 s) -- for the other ranks' flag c in its own
 * array, and combines block c in rank order into out / lse.
 *   recv_out [world]: rank r's buffer of 2 * world * L * batch * q_heads * head_dim floats;
 *   recv_lse [world]: 2 * world * L * batch * q_heads floats;  arrived [world]: world * 64 u32, zero
 *   at set-up; all mapped into this GPU's address space; epoch and n_local as above.
 * flags (per rank, nullable = all requests) must hold the same values on every rank.
 */
typedef struct {
    const float* part_out;       /* [L, batch, q_heads, head_dim] fp32: this rank's oda_full_decode_gated output */
    const float* part_lse;       /* [L, batch, q_heads] */
    const int32_t* tokens_local; /* [batch] positions this rank holds (NULL: some of every request) */
    const uint8_t* flags;        /* [batch] gate (NULL: all requests) */
    void* out;                   /* [L, batch, q_heads, head_dim] fp32 */
    float* lse;                  /* nullable */
} oda_merge_exchange_rank_t;
oda_status_t oda_merge_partials_exchange(oda_ctx_t* ctx, int32_t world, int32_t rank_base, int32_t n_local,
                                         const oda_merge_exchange_rank_t* ranks, float* const* recv_out,
                                         float* const* recv_lse, uint32_t* const* arrived, uint32_t epoch,
                                         uint64_t timeout_ns, int32_t layer_begin, int32_t layer_end,
                                         int32_t batch, void* stream);

/*
 * The paper's own recall head (appendix "Recall-head architecture"; Eq. 2): three
 * RMSNorm -> Linear(d_model -> d_tower) -> SiLU towers over (h_{t-1}, E(x_t), h_t^L), the interaction
 * vector u = [a;b;c;a.b;|a-b|;a.c;|a-c|;b.c;|b-c|], z0 = (a+b+c+SiLU(W_f u + b_f))/2, n_blocks
 * pre-RMSNorm residual SwiGLU blocks (d_tower -> d_ff -> d_tower, no biases), and
 * q = w . RMSNorm(z) + bias; fp32 weights and arithmetic.  score = sigmoid(q); the decision rule is
 * that of oda_recall_score (override, else nonfinite q or score > threshold; the paper's theta on q
 * corresponds to threshold = sigmoid(theta)).  With d_model 2048, d_tower 1024, d_ff 2048 and two
 * blocks this is the paper's 28,325,889-parameter head.
 * params (device, 16-byte aligned, row-major fp32), in this order:
 *   for i in 0..2: gain_i[d_model], W_i[d_tower][d_model], b_i[d_tower];
 *   W_f[d_tower][9 d_tower], b_f[d_tower];
 *   per block: gain[d_tower], W_gate[d_ff][d_tower], W_up[d_ff][d_tower], W_down[d_tower][d_ff];
 *   gain_out[d_tower], w[d_tower], bias[1].
 * h_prev, emb, h_local: [batch, d_model] fp32 device.  scratch: device, 256-byte aligned, at least
 * oda_full_head_scratch_bytes(head, batch) bytes, used only during the call.  d_model and d_ff
 * must be multiples of 4 and d_tower of 8 (else ODA_ERR_UNSUPPORTED).
 * variant 0 or 1: 3 + 2 n_blocks stage launches after one memset, chained by programmatic dependent
 * launch.  variant 2 (batch <= 4 and stage inputs that fit shared memory, else ODA_ERR_UNSUPPORTED):
 * one persistent kernel after one 256-byte memset: a cooperative launch of one CTA per SM that
 * streams all weights through a shared-memory ring and synchronises the stages with bounded grid
 * barriers (a barrier that times out after ~1 s sets bit 2 of the device status word and the kernel
 * returns).  It is kept as the measured alternative: on a B200 it is slower than the stage launches
 * (80 vs 52 us at batch 1).  Both are deterministic; they differ in summation order only.
 *
 * Two of the head's three inputs exist before the step's Local pass (Eq. 2: q_t = R(h_{t-1}, E(x_t),
 * h_t^L)), so the head can be run in two parts.  oda_recall_score_full_pre computes what needs only
 * h_prev and emb -- towers a and b and the four segments (a, b, a.b, |a-b|) of W_f u -- and leaves
 * it in the scratch; oda_recall_score_full with variant 3 on the same scratch then computes tower c,
 * the remaining five segments, the blocks and the output.  The sum W_f u is then taken in the order
 * (first part) + (second part): scores may differ from variants 0-2 in the last bits.  The first part
 * can run whenever the caller has room for it between two steps -- beside the backbone's other work,
 * on another stream -- and oda_step given a full_head with variant 3 then pays only for the second
 * part after its Local pass.  (Beside a Local pass that already saturates DRAM there is no room: on
 * a B200 the batch-1 benchmark step gets slower when the first part is forked next to it.)
 */
typedef struct {
    int32_t d_model, d_tower, d_ff, n_blocks;
    float eps;      /* RMSNorm epsilon (the paper does not print it; 1e-6 is customary) */
    int32_t variant; /* 0 = auto (= 1), 1 = one launch per stage, 2 = one persistent kernel (batch <= 4),
                        3 = second part only, after oda_recall_score_full_pre on the same scratch */
    const float* params;
} oda_full_head_t;
int64_t oda_full_head_param_count(int32_t d_model, int32_t d_tower, int32_t d_ff, int32_t n_blocks);
size_t oda_full_head_scratch_bytes(const oda_full_head_t* head, int32_t batch);
oda_status_t oda_recall_score_full(oda_ctx_t* ctx, int32_t batch, const oda_full_head_t* head,
                                   const float* h_prev, const float* emb, const float* h_local,
                                   float threshold, const uint8_t* override_flags, float* scores,
                                   float* logits, uint8_t* flags, int32_t* counters, void* scratch,
                                   size_t scratch_bytes, void* stream);
/* First part of the paper's head (see above): needs neither the Local hidden state nor a threshold;
 * writes only into scratch.  Two stage launches after one memset. */
oda_status_t oda_recall_score_full_pre(oda_ctx_t* ctx, int32_t batch, const oda_full_head_t* head,
                                       const float* h_prev, const float* emb, void* scratch,
                                       size_t scratch_bytes, void* stream);

/*
 * Gated Full pass (Eq. 1, S^F; Algorithm 1, line 4): for gated layers in [layer_begin,
 * layer_end) and requests with flags[b] != 0, recomputes attention over all t positions and
 * overwrites those rows of out/lse in place; every other row is left untouched.  The work
 * list is built on the device from flags and seq_lens, so the bytes read scale with the
 * flagged requests; no host read of the flags happens.
 */
oda_status_t oda_full_decode_gated(oda_ctx_t* ctx, int32_t layer_begin, int32_t layer_end,
                                   int32_t batch, const void* q_full, const void* k_cache,
                                   const void* v_cache, const int32_t* block_table,
                                   const int32_t* seq_lens, const uint8_t* flags, void* out,
                                   float* lse, void* stream);

/*
 * Commit of the current token (Algorithm 1, line 8; the fused KV commitment of the appendix on
 * selected-state execution): for every layer and every request with mask[b] != 0 (mask NULL =
 * all), writes k_cur/v_cur[l,b,:,:] ([L,B,Hkv,D] bf16) into the paged cache at position
 * seq_lens[b]-1.  One launch for all layers.  A request with seq_len < 1 or beyond the block
 * table sets the device status word and is skipped.
 */
oda_status_t oda_write_current_kv(oda_ctx_t* ctx, int32_t batch, const void* k_cur, const void* v_cur,
                                  const uint8_t* mask, void* k_cache, void* v_cache,
                                  const int32_t* block_table, const int32_t* seq_lens, void* stream);
/* Position advance on the device (the appendix on the runtime protocol: a replay updates the
 * device-side effective length): seq_lens[b] += 1 for b < batch.  oda_step does this by itself
 * (advance_seq_lens); this call is for steps composed from the separate calls.  One small launch. */
oda_status_t oda_advance_seq_lens(oda_ctx_t* ctx, int32_t batch, int32_t* seq_lens, void* stream);
/* Selected-state rule for per-request rows (h_t = h_t^{b_t}): out[b] = flags[b] ? full[b] : local[b];
 * rows of row_bytes bytes (a multiple of 16), 16-byte aligned device pointers. */
oda_status_t oda_select_rows(oda_ctx_t* ctx, int32_t batch, const void* local, const void* full,
                             const uint8_t* flags, void* out, int64_t row_bytes, void* stream);

typedef struct {
    int32_t batch;
    int32_t advance_seq_lens; /* 1 => seq_lens[b] += 1 on the device at the end of the step */
    const void* q_local;      /* [L,B,Hq,D] bf16 */
    const void* q_full;       /* same shape; NULL => q_local */
    const void* k_cache;
    const void* v_cache;
    const int32_t* block_table;
    int32_t* seq_lens;
    const float* feat_ext;    /* [B, head_d_ext] or NULL */
    const float *W1, *b1, *w2, *b2; /* head parameters; ignored when head_d_hidden = 0 */
    float threshold;
    int32_t pad;
    const uint8_t* override_flags; /* nullable: forced flags; the head still runs */
    void* out;                /* [L,B,Hq,D] out_dtype: selected output */
    float* lse;               /* nullable */
    float* scores;            /* [B] */
    float* logits;            /* [B] nullable */
    uint8_t* flags;           /* [B] */
    int32_t* counters;        /* [B,2] nullable */
    /* Optional selected-state commit (Algorithm 1, line 8).  If k_cur_local/v_cur_local
     * ([L,B,Hkv,D] bf16, the Local branch's K/V of the current token) are given, the step first
     * writes them at position seq_len-1 of every request; if k_cur_full/v_cur_full are given, the
     * Full branch's candidates replace them for the requests that recall, before the Full pass:
     * the cache then holds the selected candidate.  k_cache/v_cache must be writable.  If
     * hidden_out is given, hidden_out[b] = flag ? hidden_full[b] : hidden_local[b]
     * (rows of hidden_row_bytes bytes, a multiple of 16). */
    const void *k_cur_local, *v_cur_local, *k_cur_full, *v_cur_full;
    const void *hidden_local, *hidden_full;
    void* hidden_out;
    int64_t hidden_row_bytes;
    /* Optional: decide with the paper's own recall head (see oda_recall_score_full) instead of the
     * two-layer one.  full_head (HOST pointer) non-NULL => head_h_prev, head_emb, head_h_local
     * ([B, d_model] fp32: h_{t-1}, E(x_t) and the Local branch's h_t^L, which the caller's backbone
     * produces) and head_scratch (>= oda_full_head_scratch_bytes) are required; W1, b1, w2, b2 and
     * feat_ext are ignored; override_flags still only replaces the decision.  oda_step only. */
    const oda_full_head_t* full_head;
    const float *head_h_prev, *head_emb, *head_h_local;
    void* head_scratch;
    size_t head_scratch_bytes;
} oda_step_args_t;

/* One whole step (Algorithm 1, lines 1-7, and line 8 when the commit fields are given): Local on
 * all layers -> recall score on the last gated layer's Local output -> flags -> gated Full ->
 * optional seq_lens advance. */
oda_status_t oda_step(oda_ctx_t* ctx, const oda_step_args_t* args, void* stream);

/*
 * The same step for a caller whose per-step data lives in HOST memory: q_local, q_full,
 * feat_ext, override_flags are host inputs, out, lse, scores, logits, flags host outputs
 * (pinned memory makes the copies asynchronous); the KV cache, block table, seq_lens, head
 * weights and counters stay device pointers (they are state, not per-step input).  Brings
 * the inputs into staging areas of the workspace, runs oda_step, copies the results back and
 * waits for the stream.  Reports the bytes moved each way if the pointers are non-NULL.
 * When every input is pinned (q 16-byte aligned), one kernel pulls them all over the bus
 * instead of one copy-engine transfer each.
 * When no kernel reads the outputs back (no recall head configured, options bit 1 clear) and
 * out, lse, scores, logits, flags are all pinned buffers (out 16-byte, lse / scores / logits
 * 4-byte aligned), the kernels write them in place over the bus and no copy follows the last
 * kernel (d2h_bytes then counts every output element once); with a pageable buffer among them
 * everything goes through the staging copies.
 */
oda_status_t oda_step_host(oda_ctx_t* ctx, const oda_step_args_t* args, void* stream,
                           size_t* h2d_bytes, size_t* d2h_bytes);

/* Reads and clears the sticky device status word (synchronises the stream).
 * code: 0 ok; bit 0 = a request had seq_len < 1; bit 1 = work list overflowed its bound. */
oda_status_t oda_read_device_status(oda_ctx_t* ctx, void* stream, int32_t* code);

/* Kernel launches enqueued by this context since creation (for launch accounting). */
int64_t oda_launch_count(const oda_ctx_t* ctx);
/* The variant AUTO resolved to for this context (ODA_VARIANT_*). */
int32_t oda_resolved_variant(const oda_ctx_t* ctx);
/* Grid size (CTAs) the attention kernels of this context launch with. */
int32_t oda_attention_grid(const oda_ctx_t* ctx);

/*
 * Local pass of ONE attention layer without any workspace.  (The paper has no counterpart:
 * this entry point exists for integration, not for the method.)
 *
 * Some callers of this library cannot allocate device memory at the point where they call
 * it -- a plugin running inside another runtime's execution callback, a process whose memory
 * pool was handed out completely at start-up, code that must not disturb an allocator it
 * does not own -- and so cannot provide the workspace oda_set_workspace() asks for.  For them
 * the split partials, merge tickets and status word of this call live in a fixed array inside
 * the library's device image (about 2.2 MiB, held by every GPU that loads the library until
 * the process exits).  The call performs no device or host allocation.
 *
 * Same result as oda_local_decode() for a one-layer stack: q [batch, q_heads, head_dim] bf16,
 * out [batch, q_heads, head_dim] fp32, lse [batch, q_heads] fp32 (nullable), cache addressed by
 * block*kv_block_stride + slot*kv_token_stride + head*kv_head_stride + d, Eq. 1 with the given
 * window and sinks, sm_scale 0 => 1/sqrt(head_dim).  All pointers are device pointers.
 *
 * Limits: batch <= 16 and batch*kv_heads <= 256; anything larger returns ODA_ERR_UNSUPPORTED
 * with nothing enqueued (the scratch is never used beyond its size).
 * The first call on each device looks up the array's device address (that device must be
 * current) -- make that first call outside any stream capture.
 * Every call on a device uses the same array: a call clears what it needs to start from zero,
 * but two calls that overlap on the GPU (different streams) race.  Serialise them.
 * Problems only the device can see (a request with seq_len < 1: its rows are left untouched;
 * a seq_len beyond max_blocks_per_seq*16: clamped to it) set bits in a status word inside the
 * same array; it keeps them across calls until oda_local_decode_static_status() reads it.
 */
oda_status_t oda_local_decode_static(int32_t batch, int32_t num_q_heads, int32_t num_kv_heads,
                                     int32_t head_dim, int32_t window, int32_t sinks, float sm_scale,
                                     int64_t kv_block_stride, int64_t kv_token_stride,
                                     int64_t kv_head_stride, int32_t max_blocks_per_seq, const void* q,
                                     const void* k_cache, const void* v_cache, const int32_t* block_table,
                                     const int32_t* seq_lens, float* out, float* lse, void* stream);

/* Reads and clears the status word that the oda_local_decode_static() calls on the current
 * device have been setting (same bits as oda_read_device_status; no counterpart in the paper).
 * Allocates nothing; synchronises the stream.  Returns ODA_ERR_DEVICE_STATUS when *code != 0.
 * Like the entry point itself, its first call on a device must come outside stream capture. */
oda_status_t oda_local_decode_static_status(void* stream, int32_t* code);

const char* oda_status_string(oda_status_t s);
const char* oda_last_error(const oda_ctx_t* ctx); /* host string describing the last failure */
const char* oda_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ODA_H */
