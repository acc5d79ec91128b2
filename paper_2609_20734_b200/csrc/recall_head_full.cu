// The paper's recall head (appendix "Recall-head architecture"): three RMSNorm -> Linear -> SiLU
// towers, the 9-way interaction vector, a fusion projection, pre-RMSNorm residual SwiGLU blocks and
// a scalar output; fp32 weights and arithmetic as in the paper.  28.3 M parameters = 113 MB read
// once per step, so every stage is a bandwidth-bound GEMV: one kernel template, launched once per
// stage (towers, fusion, gate+up, down, ..., output), chained by programmatic dependent launch.
//
// A stage is  y[b][n] = epilogue( sum_k W[n][k] * gain[k] * x[b][k] ):  CTA (row block of 8 rows,
// 512-wide slice of k) streams its weights with 128-bit loads, stages x of up to 16 requests in
// shared memory (the interaction vector is formed on the fly from the towers' outputs), publishes
// partial sums and -- where the stage input is RMS-normalised -- the slice's sum of squares; the
// CTA that completes a row block (one atomic ticket, no waiting) adds the slices in order and
// applies the stage's epilogue.  All sums have a fixed order: the result does not depend on
// scheduling.
#include <algorithm>

#include "launch_ex.cuh"
#include "oda_launch.h"

namespace oda {

constexpr int kFRows = 8;
constexpr int kFThreads = kFRows * 32;

enum { kStageTower = 0, kStageFusion = 1, kStageGateUp = 2, kStageDown = 3, kStageOut = 4 };

struct FullStageParams {
    int32_t stage, batch, T, F, d_model;
    int32_t K;                   // reduction length of this stage (fusion: of the segments this launch covers)
    int32_t w_stride;            // floats between consecutive weight rows (fusion: always 9 T)
    int32_t tower_base;          // tower stage: blockIdx.z = 0 is this tower
    int32_t fus_part;            // fusion stage: 0 all nine segments of u; 1 the four that need only a and b
                                 // (a, b, a.b, |a-b|), raw sums to `out`; 2 the five that need c, added to `fpre`
    const float* fpre;           // fus_part 2: the sums of part 1, [B][T]
    int32_t row_blocks;
    float eps;
    const float* W;              // towers: W of tower 0 (+ i * tower_stride); gate+up: W_gate, W_up = W + F*T
    const float* gain;           // RMSNorm gain of the stage input (towers: + i * tower_stride), or nullptr
    const float* bias;           // towers (+ i * tower_stride), fusion, output; or nullptr
    long long tower_stride;
    const float *in0, *in1, *in2;  // towers: the three inputs [B][d_model]; fusion: abc [3][B][T];
                                   // gate+up, output: z [B][T]; down: h [B][F]
    float* out;                  // towers: abc; fusion: z; gate+up: h; down: z (in place)
    float* pre;                  // [k slices][rows][batch]
    float* ssq;                  // [row blocks][k slices][batch]
    int32_t* rb_tickets;         // [row blocks], zero between launches
    // output stage
    float threshold;
    const uint8_t* override_flags;
    float* scores;
    float* logits;
    uint8_t* flags;
    int32_t* counters;
};

__device__ __forceinline__ float silu_f(float a) { return a / (1.f + expf(-a)); }

// Fusion stage over a subset of the nine segments of u: position k of the launch's own numbering
// -> position in u (and in a row of W_f).  Segments are T long and T % 4 == 0, so four consecutive
// positions never straddle two segments.
__device__ __forceinline__ int fusion_k(const FullStageParams& p, int k)
{
    if (p.fus_part == 0) return k;
    const int s = k / p.T, j = k - s * p.T;
    // part 1: a, b, a.b, |a-b| = segments 0, 1, 3, 4;  part 2: c, a.c, |a-c|, b.c, |b-c| = 2, 5, 6, 7, 8
    const int seg = p.fus_part == 1 ? (s < 2 ? s : s + 1) : (s == 0 ? 2 : s + 4);
    return seg * p.T + j;
}

// four consecutive elements k..k+3 (k % 4 == 0) of the stage input of request b
__device__ __forceinline__ float4 stage_x4(const FullStageParams& p, int tower, int b, int k)
{
    if (p.stage == kStageTower) {
        const float* in = tower == 0 ? p.in0 : (tower == 1 ? p.in1 : p.in2);
        return __ldg(reinterpret_cast<const float4*>(in + (size_t)b * p.d_model + k));
    }
    if (p.stage == kStageFusion) {
        // u = [a; b; c; a.b; |a-b|; a.c; |a-c|; b.c; |b-c|]
        k = fusion_k(p, k);
        const int seg = k / p.T, j = k - seg * p.T;
        const float* abc = p.in0;
        const size_t row = (size_t)b * p.T + j, plane = (size_t)p.batch * p.T;
        if (seg < 3) return *reinterpret_cast<const float4*>(abc + seg * plane + row);
        const int pair = (seg - 3) >> 1;  // 0: (a,b)  1: (a,c)  2: (b,c)
        const int i0 = pair == 2 ? 1 : 0, i1 = pair == 0 ? 1 : 2;
        const float4 x = *reinterpret_cast<const float4*>(abc + i0 * plane + row);
        const float4 y = *reinterpret_cast<const float4*>(abc + i1 * plane + row);
        if ((seg - 3) & 1) return make_float4(fabsf(x.x - y.x), fabsf(x.y - y.y), fabsf(x.z - y.z), fabsf(x.w - y.w));
        return make_float4(x.x * y.x, x.y * y.y, x.z * y.z, x.w * y.w);
    }
    return *reinterpret_cast<const float4*>(p.in0 + (size_t)b * p.K + k);  // z [B][T] or h [B][F]
}

// What the epilogue of output element (row r of the stage, request b) reads besides the sums: loaded
// apart from stage_finish so that a caller can have these loads in flight together with the sums'.
struct StageEpi {
    float v[5];
};
__device__ __forceinline__ StageEpi stage_epilogue_operands(const FullStageParams& p, int r, int b)
{
    StageEpi e;
    e.v[0] = e.v[1] = e.v[2] = e.v[3] = e.v[4] = 0.f;
    if (p.stage == kStageTower) {
        const int i = r / p.T, j = r - i * p.T;
        e.v[0] = __ldg(p.bias + i * p.tower_stride + j);
    } else if (p.stage == kStageFusion) {
        const size_t row = (size_t)b * p.T + r, plane = (size_t)p.batch * p.T;
        if (p.fus_part != 1) {
            e.v[0] = p.in0[row];
            e.v[1] = p.in0[plane + row];
            e.v[2] = p.in0[2 * plane + row];
            e.v[3] = __ldg(p.bias + r);
        }
        if (p.fus_part == 2) e.v[4] = p.fpre[row];
    } else if (p.stage == kStageDown) {
        e.v[0] = p.out[(size_t)b * p.T + r];
    } else if (p.stage == kStageOut) {
        e.v[0] = __ldg(p.bias);
    }
    return e;
}

// finishes output element (row r of the stage, request b) from the complete sums
__device__ __forceinline__ void stage_finish(const FullStageParams& p, int r, int b, float acc, float acc_up, float ss,
                                             const StageEpi& e)
{
    const float rs = p.gain ? rsqrtf(ss / (float)p.K + p.eps) : 1.f;
    if (p.stage == kStageTower) {
        const int i = r / p.T, j = r - i * p.T;
        p.out[((size_t)i * p.batch + b) * p.T + j] = silu_f(acc * rs + e.v[0]);
    } else if (p.stage == kStageFusion) {
        const size_t row = (size_t)b * p.T + r;
        if (p.fus_part == 1) {
            p.out[row] = acc;   // the share of W_f u that needs only a and b
        } else {
            if (p.fus_part == 2) acc = e.v[4] + acc;   // fixed order: the earlier share first
            p.out[row] = 0.5f * (e.v[0] + e.v[1] + e.v[2] + silu_f(acc + e.v[3]));
        }
    } else if (p.stage == kStageGateUp) {
        p.out[(size_t)b * p.F + r] = silu_f(acc * rs) * (acc_up * rs);
    } else if (p.stage == kStageDown) {
        p.out[(size_t)b * p.T + r] = e.v[0] + acc;
    } else {
        const float z = acc * rs + e.v[0];
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
__device__ __forceinline__ void stage_finish(const FullStageParams& p, int r, int b, float acc, float acc_up, float ss)
{
    stage_finish(p, r, b, acc, acc_up, ss, stage_epilogue_operands(p, r, b));
}

// Tile shapes (requests x features of x in shared memory, 32 KiB either way): 4 x 2048 for small
// batches -- a lane then has all 64 of its weights in flight at once and, at the paper's sizes,
// only the fusion stage is split over k -- and 16 x 512 for larger batches.
// Grid: x = CTAs that share the row blocks of one (k slice, tower) round-robin, y = k slice,
// z = tower (tower stage only).  A CTA stages its x tile once and then walks its row blocks with
// the next block's weights already in flight.
template <int kFBT, int kFKT>
__global__ void __launch_bounds__(kFThreads, (kFKT >= 2048 ? 1 : 2)) full_head_stage_kernel(const __grid_constant__ FullStageParams p)
{
    constexpr int kWC = kFKT / 128;  // float4 weight loads per lane
    constexpr int kXL = kFBT * kFKT / 4 / kFThreads;  // float4 loads of x per thread
    __shared__ __align__(16) float s_x[kFBT][kFKT];   // x * gain
    __shared__ float s_acc[kFRows][kFBT];
    __shared__ float s_ss[kFRows][kFBT];
    __shared__ unsigned char s_lastv[kFThreads], s_list[kFThreads];
    __shared__ int s_nlast;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ks = blockIdx.y, n_ks = gridDim.y;
    const int tower = p.stage == kStageTower ? p.tower_base + (int)blockIdx.z : 0;
    const int k0 = ks * kFKT;
    const int n_rows = p.stage == kStageTower ? 3 * p.T : (p.stage == kStageGateUp ? 2 * p.F : (p.stage == kStageOut ? 1 : p.T));
    const int out_rows = p.stage == kStageGateUp ? kFRows / 2 : kFRows;
    // row blocks this CTA's group covers, and the group's offset in the stage's row numbering
    const int group_rbs = p.stage == kStageTower ? (p.T + kFRows - 1) / kFRows
                        : (p.stage == kStageGateUp ? (p.F + out_rows - 1) / out_rows
                        : (p.stage == kStageOut ? 1 : (p.T + kFRows - 1) / kFRows));
    const int group_row0 = tower * p.T;
    const float* gain = p.gain ? p.gain + tower * p.tower_stride : nullptr;
    const float* wbase = p.W + tower * p.tower_stride;
    // (row in the stage's numbering, is it a real row) of this warp for row block rb
    auto row_of = [&](int rb, bool& ok) {
        if (p.stage == kStageGateUp) {
            const int m = rb * out_rows + (warp & 3);  // hidden unit; warps 0-3 gate, 4-7 up
            ok = m < p.F;
            return (warp < 4 ? 0 : p.F) + m;
        }
        const int local = rb * kFRows + warp;
        ok = local < (p.stage == kStageTower ? p.T : n_rows);
        return group_row0 + local;
    };
    auto load_w = [&](float4 (&w)[kWC], int rb) {
        bool ok;
        const int n = row_of(rb, ok);
        const float* wrow = wbase + (size_t)(n - group_row0) * p.w_stride;
#pragma unroll
        for (int c = 0; c < kWC; ++c) {
            const int k = k0 + c * 128 + lane * 4;
            const int kw = p.stage == kStageFusion ? fusion_k(p, k) : k;
            w[c] = (ok && k < p.K) ? __ldg(reinterpret_cast<const float4*>(wrow + kw)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    for (int b0 = 0; b0 < p.batch; b0 += kFBT) {
        const bool last_tile = b0 + kFBT >= p.batch;
        float4 w_cur[kWC], w_nxt[kWC];
        int rb = blockIdx.x;
        if (rb < group_rbs) load_w(w_cur, rb);
        // weights are parameters: the first block's loads are in flight before this kernel waits for
        // the stage that produces its input
        if (b0 == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        if (b0) __syncthreads();
        {   // stage x * gain; every load of the tile is in flight together; the sum of squares of
            // the raw x is accumulated on the way
            float4 xr[kXL], gr[kXL];
#pragma unroll
            for (int t = 0; t < kXL; ++t) {
                const int idx = tid + t * kFThreads;
                const int u = idx / (kFKT / 4), q = idx - u * (kFKT / 4);
                const bool ok = b0 + u < p.batch && k0 + q * 4 < p.K;
                xr[t] = ok ? stage_x4(p, tower, b0 + u, k0 + q * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                gr[t] = (ok && gain) ? __ldg(reinterpret_cast<const float4*>(gain + k0 + q * 4)) : make_float4(1.f, 1.f, 1.f, 1.f);
            }
            if (gain) {
#pragma unroll
                for (int u = 0; u < kFBT; ++u) {
                    float ss = 0.f;
#pragma unroll
                    for (int t = 0; t < kXL; ++t) {
                        if ((tid + t * kFThreads) / (kFKT / 4) == u)
                            ss += xr[t].x * xr[t].x + xr[t].y * xr[t].y + xr[t].z * xr[t].z + xr[t].w * xr[t].w;
                    }
                    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                    if (lane == 0) s_ss[warp][u] = ss;
                }
            }
#pragma unroll
            for (int t = 0; t < kXL; ++t) {
                const int idx = tid + t * kFThreads;
                const int u = idx / (kFKT / 4), q = idx - u * (kFKT / 4);
                reinterpret_cast<float4*>(&s_x[u][0])[q] =
                    make_float4(xr[t].x * gr[t].x, xr[t].y * gr[t].y, xr[t].z * gr[t].z, xr[t].w * gr[t].w);
            }
        }
        __syncthreads();
        for (; rb < group_rbs; rb += gridDim.x) {
            const bool more = rb + (int)gridDim.x < group_rbs;
            if (more) load_w(w_nxt, rb + gridDim.x);  // in flight while this block is computed
#pragma unroll
            for (int u = 0; u < kFBT; ++u) {
                if (b0 + u >= p.batch) break;
                float a = 0.f;
#pragma unroll
                for (int c = 0; c < kWC; ++c) {
                    const float4 x = reinterpret_cast<const float4*>(&s_x[u][0])[c * 32 + lane];
                    a = fmaf(w_cur[c].x, x.x, a);
                    a = fmaf(w_cur[c].y, x.y, a);
                    a = fmaf(w_cur[c].z, x.z, a);
                    a = fmaf(w_cur[c].w, x.w, a);
                }
                for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
                if (lane == 0) s_acc[warp][u] = a;
            }
            __syncthreads();
            // ---- the block's results for this tile of requests: finish here when the stage is not
            //      split over k, else publish
            const int grb = (p.stage == kStageTower ? tower * group_rbs : 0) + rb;  // row block id in the scratch
            for (int e = tid; e < out_rows * kFBT; e += kFThreads) {
                const int r = e / kFBT, u = e - r * kFBT;
                if (b0 + u >= p.batch) continue;
                float ss = 0.f;
                if (gain) {
#pragma unroll
                    for (int wv = 0; wv < kFRows; ++wv) ss += s_ss[wv][u];  // fixed order
                }
                if (n_ks == 1) {
                    if (p.stage == kStageGateUp) {
                        const int m = rb * out_rows + r;
                        if (m < p.F) stage_finish(p, m, b0 + u, s_acc[r][u], s_acc[r + 4][u], ss);
                    } else {
                        const int local = rb * kFRows + r;
                        if (local < (p.stage == kStageTower ? p.T : n_rows)) stage_finish(p, group_row0 + local, b0 + u, s_acc[r][u], 0.f, ss);
                    }
                } else {
                    if (gain && r == 0) __stcg(p.ssq + ((size_t)grb * n_ks + ks) * p.batch + b0 + u, ss);
                    for (int rr = r; rr < kFRows; rr += out_rows) {  // gate+up: both halves
                        int nn;
                        bool ok;
                        if (p.stage == kStageGateUp) {
                            const int m = rb * out_rows + (rr & 3);
                            nn = (rr < 4 ? 0 : p.F) + m;
                            ok = m < p.F;
                        } else {
                            const int local = rb * kFRows + rr;
                            nn = group_row0 + local;
                            ok = local < (p.stage == kStageTower ? p.T : n_rows);
                        }
                        if (ok) __stcg(p.pre + ((size_t)ks * n_rows + nn) * p.batch + b0 + u, s_acc[rr][u]);
                    }
                }
            }
            __syncthreads();  // s_acc is reused by the next row block
#pragma unroll
            for (int c = 0; c < kWC; ++c) w_cur[c] = w_nxt[c];
        }
        if (n_ks > 1 && last_tile) {
            // ---- split over k: one fence for everything this CTA published, then one ticket per
            //      row block it worked on; the CTA that completes a row block adds the slices in order
            __threadfence();
            __syncthreads();
            // the tickets of all the row blocks this CTA worked on are taken at once (one thread each: one
            // round trip, not one per block), then the blocks it completed are finished one after another
            const int n_mine = (int)blockIdx.x < group_rbs ? (group_rbs - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
            for (int i0 = 0; i0 < n_mine; i0 += kFThreads) {
                const int i = i0 + tid;
                unsigned char last = 0;
                if (i < n_mine) {
                    const int grb = (p.stage == kStageTower ? tower * group_rbs : 0) + (int)blockIdx.x + i * (int)gridDim.x;
                    const int old = atomicAdd(p.rb_tickets + grb, 1);
                    last = (old == n_ks - 1);
                    if (last) p.rb_tickets[grb] = 0;
                }
                s_lastv[tid] = last;
                __threadfence();
                __syncthreads();
                const int n_here = min(kFThreads, n_mine - i0);
                // the row blocks this CTA completed, in a compact list (their order does not matter: every
                // output element is finished by itself)
                if (tid == 0) s_nlast = 0;
                __syncthreads();
                if (tid < n_here && s_lastv[tid]) s_list[atomicAdd(&s_nlast, 1)] = (unsigned char)tid;
                __syncthreads();
                // One group of G lanes per output element: the lanes fetch the k slices' partial sums (four
                // in flight per lane) and the epilogue's own operands together and add them in a fixed order
                // (per lane, then a shuffle tree); a warp finishes 32 / G elements at a time.  G is as large
                // as the number of elements leaves room for in one pass of the CTA (few elements at batch 1:
                // a group per element, one round trip; many at batch 16: a thread per element), and no
                // larger than the power of two that holds the slices.
                const int per_rb = out_rows * p.batch, total = s_nlast * per_rb;
                int G = 1;
                while (G < 32 && G < n_ks && 2 * G * total <= kFThreads) G <<= 1;
                const int per_warp = 32 / G, sub = lane / G, sl = lane - sub * G;
                for (int item0 = warp * per_warp; item0 < total; item0 += kFRows * per_warp) {
                    const int item = item0 + sub;
                    bool ok = item < total;
                    int row = 0, row_up = -1, b = 0, grb = 0;
                    if (ok) {
                        const int jj = item / per_rb, e = item - jj * per_rb;
                        const int r = e / p.batch;
                        b = e - r * p.batch;
                        const int rb2 = (int)blockIdx.x + (i0 + (int)s_list[jj]) * (int)gridDim.x;
                        grb = (p.stage == kStageTower ? tower * group_rbs : 0) + rb2;
                        if (p.stage == kStageGateUp) {
                            row = rb2 * out_rows + r;
                            row_up = p.F + row;
                            ok = row < p.F;
                        } else {
                            const int local = rb2 * kFRows + r;
                            row = group_row0 + local;
                            ok = local < (p.stage == kStageTower ? p.T : n_rows);
                        }
                    }
                    StageEpi epi;
                    float a = 0.f, a_up = 0.f, ss = 0.f;
                    if (ok) {
                        if (sl == 0) epi = stage_epilogue_operands(p, row, b);  // in flight with the sums below
                        for (int s0 = sl; s0 < n_ks; s0 += 4 * G) {
                            float v[4], vu[4], vs[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int s2 = s0 + q * G;
                                const bool in = s2 < n_ks;
                                v[q] = in ? __ldcg(p.pre + ((size_t)s2 * n_rows + row) * p.batch + b) : 0.f;
                                vu[q] = (in && row_up >= 0) ? __ldcg(p.pre + ((size_t)s2 * n_rows + row_up) * p.batch + b) : 0.f;
                                vs[q] = (in && gain) ? __ldcg(p.ssq + ((size_t)grb * n_ks + s2) * p.batch + b) : 0.f;
                            }
                            a += (v[0] + v[1]) + (v[2] + v[3]);
                            a_up += (vu[0] + vu[1]) + (vu[2] + vu[3]);
                            ss += (vs[0] + vs[1]) + (vs[2] + vs[3]);
                        }
                    }
                    for (int o = G >> 1; o; o >>= 1) {
                        a += __shfl_xor_sync(0xffffffffu, a, o);
                        a_up += __shfl_xor_sync(0xffffffffu, a_up, o);
                        ss += __shfl_xor_sync(0xffffffffu, ss, o);
                    }
                    if (ok && sl == 0) stage_finish(p, row, b, a, a_up, ss, epi);
                }
                __syncthreads();  // s_lastv is reused by the next batch of tickets
            }
        }
    }
}

long long full_head_param_count(int d_model, int T, int F, int n_blocks)
{
    const long long tower = (long long)d_model + (long long)T * d_model + T;
    const long long fusion = (long long)T * 9 * T + T;
    const long long block = (long long)T + 3ll * F * T;
    return 3 * tower + fusion + n_blocks * block + 2ll * T + 1;
}

static int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }
constexpr int kFKT = 512;  // the narrower tile: what the scratch is sized for

// scratch layout (floats unless noted): abc [3][B][T] | z [B][T] | h [B][F] | fpre [B][T] | pre | ssq | tickets (int32)
struct FullScratch {
    size_t abc, z, h, fpre, pre, ssq, tickets, total;
};

static FullScratch full_scratch_layout(int d_model, int T, int F, int batch)
{
    FullScratch s;
    auto al = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t B = batch;
    size_t off = 0;
    s.abc = off; off = al(off + 3 * B * T * 4);
    s.z = off; off = al(off + B * T * 4);
    s.h = off; off = al(off + B * F * 4);
    s.fpre = off; off = al(off + B * T * 4);
    // pre: max over stages of k slices * rows
    const size_t pre_rows = std::max({(size_t)ceil_div(d_model, kFKT) * 3 * T, (size_t)ceil_div(9ll * T, kFKT) * T,
                                      (size_t)ceil_div(T, kFKT) * 2 * F, (size_t)ceil_div(F, kFKT) * T});
    s.pre = off; off = al(off + pre_rows * B * 4);
    const size_t ssq_rows = std::max({(size_t)ceil_div(3ll * T, kFRows) * ceil_div(d_model, kFKT),
                                      (size_t)ceil_div(F, kFRows / 2) * ceil_div(T, kFKT), (size_t)ceil_div(T, kFKT)});
    s.ssq = off; off = al(off + ssq_rows * B * 4);
    const size_t max_rb = std::max({(size_t)ceil_div(3ll * T, kFRows), (size_t)ceil_div(F, kFRows / 2), (size_t)T});
    s.tickets = off; off = al(off + max_rb * 4);
    s.total = off;
    return s;
}

size_t full_head_scratch_bytes(int d_model, int T, int F, int batch)
{
    return full_scratch_layout(d_model, T, F, batch).total;
}

cudaError_t launch_full_head(int batch, int d_model, int T, int F, int n_blocks, float eps, const float* params,
                             const float* h_prev, const float* emb, const float* h_local, float threshold,
                             const uint8_t* override_flags, float* scores, float* logits, uint8_t* flags,
                             int32_t* counters, void* scratch, cudaStream_t st, bool pdl, int* launches, int variant,
                             int32_t* status, int phase)
{
    // phase 0: the whole head.  phase 1: what does not need the Local hidden state -- towers a and b
    // and their four segments of the fusion product -- left in the scratch.  phase 2: the rest, on top
    // of a phase 1 that ran on the same scratch: tower c, the five segments that need c, the blocks, the
    // output.  1 + 2 sum the fusion product in a different (fixed) order than 0: last bits may differ.
    char* sc = static_cast<char*>(scratch);
    const FullScratch L = full_scratch_layout(d_model, T, F, batch);
    // variant 2: the whole chain as one persistent kernel (measured slower than the stage launches, so
    // 0 = auto picks the stage launches; see recall_head_fused.cu)
    const long long x_floats = full_head_fused_x_floats(batch, d_model, T, F);
    if (variant == 2 && phase != 0) return cudaErrorNotSupported;
    const int fused_grid = (variant == 2 && batch <= kFullHeadFusedMaxBatch && x_floats * 4 + 1024 + 8 * 4096 <= kFullHeadFusedSmem)
                               ? full_head_fused_grid() : 0;
    if (variant == 2 && fused_grid == 0) return cudaErrorNotSupported;
    if (fused_grid > 0) {
        cudaError_t fe = cudaMemsetAsync(sc + L.tickets, 0, 256, st);  // arrival counter and abort flag
        if (fe != cudaSuccess) return fe;
        fe = launch_full_head_fused(fused_grid, batch, d_model, T, F, n_blocks, eps, params, h_prev, emb, h_local,
                                    threshold, override_flags, scores, logits, flags, counters,
                                    reinterpret_cast<float*>(sc + L.abc), reinterpret_cast<float*>(sc + L.z),
                                    reinterpret_cast<float*>(sc + L.h), reinterpret_cast<int32_t*>(sc + L.tickets),
                                    status, st);
        if (fe == cudaSuccess && launches) ++*launches;
        return fe;
    }
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        sms = 148;
    float* abc = reinterpret_cast<float*>(sc + L.abc);
    float* z = reinterpret_cast<float*>(sc + L.z);
    float* h = reinterpret_cast<float*>(sc + L.h);
    cudaError_t e = cudaSuccess;
    if (phase != 2) {  // phase 2 finds the tickets as phase 1 left them: every one back at zero
        e = cudaMemsetAsync(sc + L.tickets, 0, L.total - L.tickets, st);
        if (e != cudaSuccess) return e;
    }
    FullStageParams p = {};
    p.batch = batch; p.T = T; p.F = F; p.d_model = d_model; p.eps = eps;
    p.pre = reinterpret_cast<float*>(sc + L.pre);
    p.ssq = reinterpret_cast<float*>(sc + L.ssq);
    p.rb_tickets = reinterpret_cast<int32_t*>(sc + L.tickets);
    int n_towers = 3;
    auto launch = [&](bool dep) {
        // small batches: a 2048-wide k tile (one CTA per SM) where that divides k (towers, down: no
        // split over k), else a 1024-wide one (gate+up fits it whole; the fusion's k = 9 x 1024 splits
        // evenly): two CTAs per SM.  Measured (before the finishing pass
        // of the split-k stages was parallelised): 2048 everywhere 61 us, 1024 everywhere 68 us, mixed 59 us.
        const int kt = batch <= 4 ? ((p.K <= 1024 || p.K % 2048 != 0) ? 1024 : 2048) : 512;
        const int n_ks = ceil_div(p.K, kt);
        const int groups = p.stage == kStageTower ? n_towers : 1;
        const int group_rbs = p.stage == kStageTower ? ceil_div(T, kFRows) : p.row_blocks;
        // about one CTA per SM in total for small batches and two for large ones (narrow tiles, two
        // CTAs fit an SM), each staging its x tile once and walking several row blocks
        // (half as many CTAs, so that the next stage's CTAs could sit beside them and have their first
        // weights in flight when this stage ends, was measured twice -- 1024-wide tiles everywhere, and the
        // tiles below compiled for two CTAs per SM: 58 -> 96 and 58 -> 92 us per call at batch 1.  A stage is
        // bound by how many loads an SM has in flight, and half the CTAs are half the loads.)
        int gx = (kt >= 2048 ? sms : 2 * sms) / (n_ks * groups);
        gx = std::max(1, std::min(gx, group_rbs));
        const dim3 grid(gx, n_ks, groups);
        cudaError_t le = kt == 2048 ? launch_ex(full_head_stage_kernel<4, 2048>, grid, dim3(kFThreads), 0, st, dep, p)
                         : kt == 1024 ? launch_ex(full_head_stage_kernel<4, 1024>, grid, dim3(kFThreads), 0, st, dep, p)
                                      : launch_ex(full_head_stage_kernel<16, 512>, grid, dim3(kFThreads), 0, st, dep, p);
        if (le == cudaSuccess && launches) ++*launches;
        return le;
    };
    const long long tower_stride = (long long)d_model + (long long)T * d_model + T;
    const float* cur = params;
    float* fpre = reinterpret_cast<float*>(sc + L.fpre);
    // towers (one launch for those of this phase)
    n_towers = phase == 0 ? 3 : (phase == 1 ? 2 : 1);
    p.stage = kStageTower; p.K = d_model; p.w_stride = d_model; p.row_blocks = ceil_div(3ll * T, kFRows);
    p.tower_base = phase == 2 ? 2 : 0;
    p.gain = cur; p.W = cur + d_model; p.bias = cur + d_model + (long long)T * d_model; p.tower_stride = tower_stride;
    p.in0 = h_prev; p.in1 = emb; p.in2 = h_local; p.out = abc;
    if ((e = launch(false)) != cudaSuccess) return e;  // follows a memset (phases 0, 1) or a join of two streams (phase 2): ordinary launch
    cur += 3 * tower_stride;
    // fusion
    p.stage = kStageFusion; p.K = (phase == 0 ? 9 : (phase == 1 ? 4 : 5)) * T; p.w_stride = 9 * T; p.row_blocks = ceil_div(T, kFRows);
    p.fus_part = phase; p.fpre = fpre;
    p.gain = nullptr; p.W = cur; p.bias = cur + (long long)T * 9 * T; p.in0 = abc; p.in1 = p.in2 = nullptr;
    p.out = phase == 1 ? fpre : z;
    if ((e = launch(pdl)) != cudaSuccess) return e;
    if (phase == 1) return cudaSuccess;
    p.fus_part = 0;
    cur += (long long)T * 9 * T + T;
    for (int k = 0; k < n_blocks; ++k) {
        p.stage = kStageGateUp; p.K = T; p.w_stride = T; p.row_blocks = ceil_div(F, kFRows / 2);
        p.gain = cur; p.W = cur + T; p.bias = nullptr; p.in0 = z; p.out = h;
        if ((e = launch(pdl)) != cudaSuccess) return e;
        p.stage = kStageDown; p.K = F; p.w_stride = F; p.row_blocks = ceil_div(T, kFRows);
        p.gain = nullptr; p.W = cur + T + 2ll * F * T; p.in0 = h; p.out = z;
        if ((e = launch(pdl)) != cudaSuccess) return e;
        cur += (long long)T + 3ll * F * T;
    }
    p.stage = kStageOut; p.K = T; p.w_stride = T; p.row_blocks = 1;
    p.gain = cur; p.W = cur + T; p.bias = cur + 2 * T; p.in0 = z; p.out = nullptr;
    p.threshold = threshold; p.override_flags = override_flags; p.scores = scores; p.logits = logits;
    p.flags = flags; p.counters = counters;
    return launch(pdl);
}

}  // namespace oda
