/*
 * ODA decode-attention oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what one On-Demand-Attention decode step
 * computes on the attention path.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may use it; the CUDA library shares no code,
 * header, table or helper with this file.
 *
 * What it follows, from the paper:
 *   - Eq. 1 (access sets): Full = {1..t}; Local = {1..min(s,t)} U {max(1,t-w+1)..t},
 *     a set (an index that is both a sink and in the window counts once); the
 *     recent window includes the current token.
 *   - Algorithm 1, lines 1-7 and the selected-state equation of the appendix on
 *     selected-state execution: run Local, score it, take Full when the score
 *     exceeds the threshold or is nonfinite, the selected branch supplies the
 *     output.  Restriction applies only to the layers that natively attend to
 *     the whole history; fixed-window layers keep their own window whatever the
 *     decision is.
 *   - The attention inside each branch is exact softmax attention over the
 *     branch's index set, so it is written here as that definition: logits,
 *     a two-pass softmax (max, then exponentials and their sum), a weighted sum
 *     of values.  No online softmax, no splits, no sharing of work between the
 *     query heads of a group.
 *
 * Readings taken where the paper is silent (they are listed in the design notes
 * of the repository as well): logits are scaled by sm_scale (1/sqrt(D) when 0
 * is passed by the caller of the Python wrapper); query head h reads KV head
 * floor(h / (Hq/Hkv)); q and the cached keys arrive already position-encoded;
 * the current token's K/V is already at index t-1 of the paged cache; the
 * recall head of the benchmark configurations is a two-layer MLP
 * z = w2 . SiLU(W1 x + b1) + b2 with x = [external features ; flattened Local
 * output of the last gated layer], score = sigmoid(z), flag = override if one
 * is given, else (z nonfinite) or (score > threshold), strictly.
 *
 * Algorithm 1, line 8 (commit of the selected candidate) is oda_oracle_write_current_kv +
 * oda_oracle_select_rows, composed into a step by step_with_commit() of the wrapper.
 *
 * The paper's own recall head (appendix "Recall-head architecture", Eq. 2) is
 * oda_oracle_full_head: three RMSNorm -> Linear -> SiLU towers, the 9-way
 * interaction vector, the fusion projection, pre-norm residual SwiGLU blocks and a
 * normalised scalar output, in the paper's order; its parameter count is pinned to
 * the 28,325,889 the paper states, the order of the nine interaction segments by
 * one-hot rows of the fusion matrix read against a hand-made table, and a SwiGLU
 * block, the fusion bias and the placement of eps by values worked out by hand.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py
 * (brute force over literal 1-based sets in extended precision, an independent
 * masked-attention library routine, closed forms, set identities quoted from
 * the paper, gating invariants).  No function is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t num_layers;          /* L: layers in q/out */
    int32_t batch;               /* B */
    int32_t num_q_heads;         /* Hq */
    int32_t num_kv_heads;        /* Hkv */
    int32_t head_dim;            /* D */
    int32_t block_size;          /* P tokens per KV block */
    int32_t max_blocks_per_seq;  /* row length of block_table */
    int32_t reserved;
    int64_t kv_layer_stride;     /* element strides of k_cache / v_cache; D contiguous */
    int64_t kv_block_stride;
    int64_t kv_token_stride;
    int64_t kv_head_stride;
    double sm_scale;
} oracle_shape_t;

static double bf16_to_f64(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Eq. 1, written with the paper's 1-based positions: is position i (1..t) in the set? */
static int in_full_set(int i, int t) { return i >= 1 && i <= t; }

static int in_local_set(int i, int t, int s, int w)
{
    int sink_hi = s < t ? s : t;             /* min(s, t) */
    int win_lo = t - w + 1 > 1 ? t - w + 1 : 1; /* max(1, t-w+1) */
    if (i < 1 || i > t) return 0;
    return (i <= sink_hi) || (i >= win_lo);
}

/* address of element 0 of the D-vector of token position j (0-based) of request b */
static const uint16_t *kv_row(const oracle_shape_t *sh, const uint16_t *cache, int kv_layer,
                              const int32_t *block_table, int b, int j, int kv_head)
{
    int32_t blk = block_table[(int64_t)b * sh->max_blocks_per_seq + j / sh->block_size];
    int slot = j % sh->block_size;
    return cache + (int64_t)kv_layer * sh->kv_layer_stride + (int64_t)blk * sh->kv_block_stride +
           (int64_t)slot * sh->kv_token_stride + (int64_t)kv_head * sh->kv_head_stride;
}

/*
 * Softmax attention of ONE query head over one index set.
 * mode 0 = Local (Eq. 1 with s sinks, window w), mode 1 = Full.
 * out[D], *lse = max + ln(sum of exponentials).  scratch has room for t doubles.
 */
static void attend_one(const oracle_shape_t *sh, int mode, int s, int w, const uint16_t *q_row,
                       const uint16_t *k_cache, const uint16_t *v_cache, int kv_layer,
                       const int32_t *block_table, int b, int t, int kv_head, double *out,
                       double *lse, double *scratch)
{
    const int D = sh->head_dim;
    double zmax = -INFINITY;
    int any = 0;
    /* pass 1: logits of the members, and their maximum */
    for (int i = 1; i <= t; ++i) {
        int member = mode ? in_full_set(i, t) : in_local_set(i, t, s, w);
        if (!member) continue;
        const uint16_t *k = kv_row(sh, k_cache, kv_layer, block_table, b, i - 1, kv_head);
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += bf16_to_f64(q_row[d]) * bf16_to_f64(k[d]);
        double z = sh->sm_scale * dot;
        scratch[i - 1] = z;
        if (!any || z > zmax) zmax = z;
        any = 1;
    }
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (!any) { /* empty set: t < 1 */
        *lse = -INFINITY;
        return;
    }
    /* pass 2: exponentials, their sum, weighted values */
    double denom = 0.0;
    for (int i = 1; i <= t; ++i) {
        int member = mode ? in_full_set(i, t) : in_local_set(i, t, s, w);
        if (!member) continue;
        double e = exp(scratch[i - 1] - zmax);
        const uint16_t *v = kv_row(sh, v_cache, kv_layer, block_table, b, i - 1, kv_head);
        denom += e;
        for (int d = 0; d < D; ++d) out[d] += e * bf16_to_f64(v[d]);
    }
    for (int d = 0; d < D; ++d) out[d] /= denom;
    *lse = zmax + log(denom);
}

/*
 * Attention for layers [layer_begin, layer_end), every request and query head.
 * mode 0: Local sets with the layer's (sinks, window); mode 1: Full set.
 * request_mask (nullable, [B]): rows with 0 are skipped and left untouched.
 * layer_kv_index (nullable, [L]): which layer of the cache holds layer l's K/V.
 * q: [L,B,Hq,D] bf16 bits.  out: [L,B,Hq,D] f64.  lse: [L,B,Hq] f64 (nullable).
 * Returns 0, or -1 on a bad argument.
 */
int oda_oracle_attention(const oracle_shape_t *sh, int mode, const int32_t *layer_window,
                         const int32_t *layer_sinks, const int32_t *layer_kv_index,
                         const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                         const int32_t *block_table, const int32_t *seq_lens,
                         const uint8_t *request_mask, int layer_begin, int layer_end, double *out,
                         double *lse, int nthreads)
{
    if (!sh || !q || !k_cache || !v_cache || !block_table || !seq_lens || !out) return -1;
    if (sh->num_kv_heads <= 0 || sh->num_q_heads % sh->num_kv_heads) return -1;
    if (layer_begin < 0 || layer_end > sh->num_layers || layer_begin > layer_end) return -1;
    const int B = sh->batch, Hq = sh->num_q_heads, D = sh->head_dim;
    const int G = Hq / sh->num_kv_heads;
    int tmax = 1;
    for (int b = 0; b < B; ++b)
        if (seq_lens[b] > tmax) tmax = seq_lens[b];
    const int64_t units = (int64_t)(layer_end - layer_begin) * B * Hq;
    if (nthreads < 1) nthreads = 1;
#ifdef _OPENMP
#pragma omp parallel num_threads(nthreads)
#endif
    {
        double *scratch = (double *)malloc(sizeof(double) * (size_t)tmax);
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
        for (int64_t u = 0; u < units; ++u) {
            int h = (int)(u % Hq);
            int b = (int)((u / Hq) % B);
            int l = layer_begin + (int)(u / ((int64_t)Hq * B));
            if (request_mask && !request_mask[b]) continue;
            int t = seq_lens[b];
            int kv_layer = layer_kv_index ? layer_kv_index[l] : l;
            int64_t row = ((int64_t)l * B + b) * Hq + h;
            double l_se;
            attend_one(sh, mode, layer_sinks ? layer_sinks[l] : 0,
                       layer_window ? layer_window[l] : t, q + row * D, k_cache, v_cache, kv_layer,
                       block_table, b, t, h / G, out + row * D, &l_se, scratch);
            if (lse) lse[row] = l_se;
        }
        free(scratch);
    }
    return 0;
}

static double silu(double a) { return a / (1.0 + exp(-a)); }

/*
 * Recall head of the benchmark configurations: for each request
 *   x = [feat_ext[b] (d_ext values) ; attn_feat[b] (d_attn values)],
 *   z = w2 . SiLU(W1 x + b1) + b2,  score = 1 / (1 + exp(-z)).
 * W1 is [d_hidden, d_ext + d_attn] row-major fp32; arithmetic in fp64 on those values.
 */
int oda_oracle_recall_head(int batch, int d_ext, int d_attn, int d_hidden, const float *feat_ext,
                           const double *attn_feat, const float *W1, const float *b1,
                           const float *w2, const float *b2, double *z_out, double *score_out)
{
    if (batch < 0 || d_ext < 0 || d_attn < 0 || d_hidden < 1 || !W1 || !b1 || !w2 || !b2) return -1;
    if ((d_ext > 0 && !feat_ext) || (d_attn > 0 && !attn_feat)) return -1;
    const int d_in = d_ext + d_attn;
    for (int b = 0; b < batch; ++b) {
        double z = (double)b2[0];
        for (int j = 0; j < d_hidden; ++j) {
            double a = (double)b1[j];
            const float *wrow = W1 + (int64_t)j * d_in;
            for (int i = 0; i < d_ext; ++i) a += (double)wrow[i] * (double)feat_ext[(int64_t)b * d_ext + i];
            for (int i = 0; i < d_attn; ++i) a += (double)wrow[d_ext + i] * attn_feat[(int64_t)b * d_attn + i];
            z += (double)w2[j] * silu(a);
        }
        if (z_out) z_out[b] = z;
        if (score_out) score_out[b] = 1.0 / (1.0 + exp(-z));
    }
    return 0;
}

/* Decision rule: the override if one is given; else Full when z is nonfinite or score > tau. */
int oda_oracle_flags(int batch, const double *z, const double *score, double tau,
                     const uint8_t *override_flags, uint8_t *flags)
{
    if (!flags || (!override_flags && (!z || !score))) return -1;
    for (int b = 0; b < batch; ++b) {
        if (override_flags)
            flags[b] = override_flags[b] ? 1 : 0;
        else
            flags[b] = (!isfinite(z[b]) || score[b] > tau) ? 1 : 0;
    }
    return 0;
}

/*
 * One whole step (Algorithm 1, lines 1-7, on the attention stack):
 *   1. Local attention on every layer                      -> out_local
 *   2. recall head on [feat_ext ; Local output of the last gated layer]
 *   3. flags
 *   4. Full attention on gated layers for flagged requests (q_full, or q_local when NULL)
 *   5. out = flag && gated ? full : local
 * If no layer is gated the head sees d_attn = 0 attention features.  d_hidden = 0 means
 * "no head": an override is then required.
 * out, out_local are caller buffers [L,B,Hq,D]; lse, lse_local [L,B,Hq] (nullable).
 */
int oda_oracle_step(const oracle_shape_t *sh, const int32_t *layer_window,
                    const int32_t *layer_sinks, const uint8_t *layer_gated,
                    const int32_t *layer_kv_index, const uint16_t *q_local, const uint16_t *q_full,
                    const uint16_t *k_cache, const uint16_t *v_cache, const int32_t *block_table,
                    const int32_t *seq_lens, int d_ext, int use_attn_out, int d_hidden,
                    const float *feat_ext, const float *W1, const float *b1, const float *w2,
                    const float *b2, double tau, const uint8_t *override_flags, double *out,
                    double *lse, double *out_local, double *lse_local, double *z_out,
                    double *score_out, uint8_t *flags, int nthreads)
{
    if (!sh || !out || !out_local || !flags || !layer_gated) return -1;
    const int L = sh->num_layers, B = sh->batch, Hq = sh->num_q_heads, D = sh->head_dim;
    const int64_t per_layer = (int64_t)B * Hq * D;
    int rc = oda_oracle_attention(sh, 0, layer_window, layer_sinks, layer_kv_index, q_local, k_cache,
                                  v_cache, block_table, seq_lens, NULL, 0, L, out_local, lse_local,
                                  nthreads);
    if (rc) return rc;
    int last_gated = -1;
    for (int l = 0; l < L; ++l)
        if (layer_gated[l]) last_gated = l;
    int d_attn = (use_attn_out && last_gated >= 0) ? Hq * D : 0;
    double *z = (double *)malloc(sizeof(double) * (size_t)(B > 0 ? B : 1));
    double *score = (double *)malloc(sizeof(double) * (size_t)(B > 0 ? B : 1));
    if (d_hidden > 0) {
        rc = oda_oracle_recall_head(B, d_ext, d_attn, d_hidden, feat_ext,
                                    d_attn ? out_local + last_gated * per_layer : NULL, W1, b1, w2,
                                    b2, z, score);
    } else {
        for (int b = 0; b < B; ++b) { z[b] = 0.0; score[b] = 0.5; }
        if (!override_flags) rc = -1;
    }
    if (!rc) rc = oda_oracle_flags(B, z, score, tau, override_flags, flags);
    if (!rc) {
        memcpy(out, out_local, sizeof(double) * (size_t)(L * per_layer));
        if (lse && lse_local) memcpy(lse, lse_local, sizeof(double) * (size_t)L * B * Hq);
        double *full = (double *)malloc(sizeof(double) * (size_t)(L * per_layer > 0 ? L * per_layer : 1));
        double *lse_f = (double *)malloc(sizeof(double) * (size_t)(L * B * Hq > 0 ? L * B * Hq : 1));
        for (int l = 0; l < L && !rc; ++l) {
            if (!layer_gated[l]) continue; /* fixed-window layers keep Local */
            rc = oda_oracle_attention(sh, 1, layer_window, layer_sinks, layer_kv_index,
                                      q_full ? q_full : q_local, k_cache, v_cache, block_table,
                                      seq_lens, flags, l, l + 1, full, lse_f, nthreads);
            for (int b = 0; b < B && !rc; ++b) {
                if (!flags[b]) continue;
                int64_t off = ((int64_t)l * B + b) * Hq * D;
                memcpy(out + off, full + off, sizeof(double) * (size_t)Hq * D);
                if (lse) memcpy(lse + ((int64_t)l * B + b) * Hq, lse_f + ((int64_t)l * B + b) * Hq,
                                sizeof(double) * (size_t)Hq);
            }
        }
        free(full);
        free(lse_f);
    }
    if (z_out) memcpy(z_out, z, sizeof(double) * (size_t)B);
    if (score_out) memcpy(score_out, score, sizeof(double) * (size_t)B);
    free(z);
    free(score);
    return rc;
}

/*
 * Commit of the current token (Algorithm 1, line 8, C_t = C_{t-1} || dC_t; "fused commitment"
 * paragraph of the appendix on selected-state execution): for every layer and every request
 * with mask[b] != 0 (mask NULL = every request), the K and V vectors of the current token are
 * written into the paged cache at position seq_len - 1.  k_cur, v_cur: [L,B,Hkv,D] bf16 bits.
 * Used twice in a step: the Local candidate for every request before the Local pass, and the
 * Full candidate of the requests that recall before the Full pass (the selected candidate is
 * then the one the cache keeps).
 */
int oda_oracle_write_current_kv(const oracle_shape_t *sh, const int32_t *layer_kv_index,
                                const uint16_t *k_cur, const uint16_t *v_cur, const uint8_t *mask,
                                uint16_t *k_cache, uint16_t *v_cache, const int32_t *block_table,
                                const int32_t *seq_lens)
{
    if (!sh || !k_cur || !v_cur || !k_cache || !v_cache || !block_table || !seq_lens) return -1;
    const int L = sh->num_layers, B = sh->batch, H = sh->num_kv_heads, D = sh->head_dim;
    for (int l = 0; l < L; ++l) {
        const int kvl = layer_kv_index ? layer_kv_index[l] : l;
        for (int b = 0; b < B; ++b) {
            if (mask && !mask[b]) continue;
            const int t = seq_lens[b];
            if (t < 1) return -1;
            for (int g = 0; g < H; ++g) {
                const int64_t src = (((int64_t)l * B + b) * H + g) * D;
                /* same addressing as the reads: position t-1 of request b */
                uint16_t *kd = (uint16_t *)kv_row(sh, k_cache, kvl, block_table, b, t - 1, g);
                uint16_t *vd = (uint16_t *)kv_row(sh, v_cache, kvl, block_table, b, t - 1, g);
                memcpy(kd, k_cur + src, sizeof(uint16_t) * (size_t)D);
                memcpy(vd, v_cur + src, sizeof(uint16_t) * (size_t)D);
            }
        }
    }
    return 0;
}

/* Selected-state rule for a per-request row (h_t = h_t^{b_t}): out[b] = flags[b] ? full[b] : local[b]. */
int oda_oracle_select_rows(int batch, int64_t row_bytes, const uint8_t *local, const uint8_t *full,
                           const uint8_t *flags, uint8_t *out)
{
    if (batch < 0 || row_bytes < 0 || !local || !full || !flags || !out) return -1;
    for (int b = 0; b < batch; ++b)
        memcpy(out + (int64_t)b * row_bytes, (flags[b] ? full : local) + (int64_t)b * row_bytes, (size_t)row_bytes);
    return 0;
}

/*
 * The paper's recall head (appendix "Recall-head architecture"), fp64 on fp32 parameters:
 *   towers   a, b, c = SiLU(W_i RMSNorm_i(x_i) + b_i)            x_i in R^d_model -> R^d_tower, i = 0,1,2
 *            (x_0 = preceding selected hidden h_{t-1}, x_1 = embedding E(x_t), x_2 = Local hidden h_t^L)
 *   u        = [a; b; c; a.b; |a-b|; a.c; |a-c|; b.c; |b-c|]      in R^(9 d_tower)
 *   z0       = 1/2 [a + b + c + SiLU(W_f u + b_f)]
 *   blocks   z <- z + W_down( SiLU(W_gate n) . (W_up n) ),  n = RMSNorm(z)   (n_blocks times, no biases)
 *   q        = w . RMSNorm(z) + bias
 * RMSNorm(x) = x / sqrt(mean(x^2) + eps) . g.  The paper does not print eps (1e-6 is used by the
 * callers here) nor the SwiGLU operand order (SiLU on the gate projection, as in the GLU-variants
 * paper it cites).  Parameter layout in `params`, in this order, all row-major fp32:
 *   for i in 0..2: g_i[d_model], W_i[d_tower][d_model], b_i[d_tower];
 *   W_f[d_tower][9 d_tower], b_f[d_tower];
 *   for k in blocks: g_k[d_tower], W_gate[d_ff][d_tower], W_up[d_ff][d_tower], W_down[d_tower][d_ff];
 *   g_out[d_tower], w[d_tower], bias[1].
 * With d_model 2048, d_tower 1024, d_ff 2048 and 2 blocks this is the 28,325,889 parameters the
 * paper states.
 */
int64_t oda_oracle_full_head_param_count(int d_model, int d_tower, int d_ff, int n_blocks)
{
    int64_t tower = (int64_t)d_model + (int64_t)d_tower * d_model + d_tower;
    int64_t fusion = (int64_t)d_tower * 9 * d_tower + d_tower;
    int64_t block = (int64_t)d_tower + 3ll * d_ff * d_tower;
    return 3 * tower + fusion + n_blocks * block + 2ll * d_tower + 1;
}

static void rmsnorm64(const double *x, const float *g, int n, double eps, double *out)
{
    double ss = 0.0;
    for (int i = 0; i < n; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / n + eps);
    for (int i = 0; i < n; ++i) out[i] = x[i] * r * (double)g[i];
}

int oda_oracle_full_head(int batch, int d_model, int d_tower, int d_ff, int n_blocks, double eps,
                         const float *params, const float *h_prev, const float *emb, const float *h_local,
                         double *q_out, double *score_out)
{
    if (batch < 0 || d_model < 1 || d_tower < 1 || d_ff < 1 || n_blocks < 0 || !params) return -1;
    if (!h_prev || !emb || !h_local) return -1;
    const float *inputs[3] = {h_prev, emb, h_local};
    const int T = d_tower;
    double *x = (double *)malloc(sizeof(double) * (size_t)(d_model > T ? d_model : T));
    double *n = (double *)malloc(sizeof(double) * (size_t)(d_model > T ? d_model : T));
    double *abc = (double *)malloc(sizeof(double) * 3 * (size_t)T);
    double *u = (double *)malloc(sizeof(double) * 9 * (size_t)T);
    double *z = (double *)malloc(sizeof(double) * (size_t)T);
    double *hmid = (double *)malloc(sizeof(double) * (size_t)d_ff);
    for (int b = 0; b < batch; ++b) {
        const float *p = params;
        for (int i = 0; i < 3; ++i) {
            const float *g = p, *W = p + d_model, *bias = W + (int64_t)T * d_model;
            for (int k = 0; k < d_model; ++k) x[k] = (double)inputs[i][(int64_t)b * d_model + k];
            rmsnorm64(x, g, d_model, eps, n);
            for (int j = 0; j < T; ++j) {
                double acc = (double)bias[j];
                for (int k = 0; k < d_model; ++k) acc += (double)W[(int64_t)j * d_model + k] * n[k];
                abc[i * T + j] = silu(acc);
            }
            p = bias + T;
        }
        const double *a = abc, *bb = abc + T, *c = abc + 2 * T;
        for (int j = 0; j < T; ++j) {
            u[0 * T + j] = a[j];
            u[1 * T + j] = bb[j];
            u[2 * T + j] = c[j];
            u[3 * T + j] = a[j] * bb[j];
            u[4 * T + j] = fabs(a[j] - bb[j]);
            u[5 * T + j] = a[j] * c[j];
            u[6 * T + j] = fabs(a[j] - c[j]);
            u[7 * T + j] = bb[j] * c[j];
            u[8 * T + j] = fabs(bb[j] - c[j]);
        }
        {
            const float *Wf = p, *bf = Wf + (int64_t)T * 9 * T;
            for (int j = 0; j < T; ++j) {
                double acc = (double)bf[j];
                for (int k = 0; k < 9 * T; ++k) acc += (double)Wf[(int64_t)j * 9 * T + k] * u[k];
                z[j] = 0.5 * (a[j] + bb[j] + c[j] + silu(acc));
            }
            p = bf + T;
        }
        for (int blk = 0; blk < n_blocks; ++blk) {
            const float *g = p, *Wg = g + T, *Wu = Wg + (int64_t)d_ff * T, *Wd = Wu + (int64_t)d_ff * T;
            rmsnorm64(z, g, T, eps, n);
            for (int m = 0; m < d_ff; ++m) {
                double gate = 0.0, up = 0.0;
                for (int k = 0; k < T; ++k) {
                    gate += (double)Wg[(int64_t)m * T + k] * n[k];
                    up += (double)Wu[(int64_t)m * T + k] * n[k];
                }
                hmid[m] = silu(gate) * up;
            }
            for (int j = 0; j < T; ++j) {
                double acc = 0.0;
                for (int m = 0; m < d_ff; ++m) acc += (double)Wd[(int64_t)j * d_ff + m] * hmid[m];
                x[j] = z[j] + acc;
            }
            for (int j = 0; j < T; ++j) z[j] = x[j];
            p = Wd + (int64_t)T * d_ff;
        }
        {
            const float *g = p, *w = g + T, *bias = w + T;
            rmsnorm64(z, g, T, eps, n);
            double q = (double)bias[0];
            for (int k = 0; k < T; ++k) q += (double)w[k] * n[k];
            if (q_out) q_out[b] = q;
            if (score_out) score_out[b] = 1.0 / (1.0 + exp(-q));
        }
    }
    free(x); free(n); free(abc); free(u); free(z); free(hmid);
    return 0;
}

int oda_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
