// The persistent decode kernel: Algorithm 1 of the paper, one cooperative launch for many steps.
//
// One CTA per SM, ten warps: a weight producer, an activation / KV producer and eight consumers.
// Every CTA walks the same program
//     control | for each layer: QKV | attention | O | gate-up | down | [head, control] ... | final head | control
// with a grid barrier between phases.  The weight producer is not held by those barriers: it
// keeps the TMA ring full with the tiles of the coming phases, so HBM keeps streaming while the
// consumers meet.  All decoding state (sequence, per-layer fill levels, in-flight tokens, row
// residuals, counters) lives in device memory; the control points run in CTA 0, which publishes
// each decision (continue the climb, start the next token, stop) to the other CTAs through a
// sequence-numbered record.  The host launches, waits, and launches again until the call is done.
//
// Token columns: the up-to-eight tokens of a pass (the newest token and the early-predicted
// tokens still in flight, Algorithm 1's P[l] (+) t_i) are the eight columns of the tensor-core
// tile; column = position - base, fixed for the life of a token.  Per-column buffers therefore
// persist across steps: a token that left the climb at layer e finds its residual, its
// normalisation partial sums and its layer-(e+1) GEMM input where its last pass left them.
// Each column's numbers depend only on that column's own inputs (never on which other columns
// ride along), which is what makes the adaptive output bit-identical to plain greedy decoding.
#pragma once

#include "kernels.cuh"
#include "stream.cuh"

namespace ada {
namespace mg {

using namespace st;

constexpr int ACT_CONTINUE = 1, ACT_NEWSTEP = 2, ACT_STOP = 3;
constexpr int CTRL_START = 0, CTRL_HEAD = 1, CTRL_TOP = 2;
constexpr int ATT_PAGE = 64;          // cache positions per attention sub-block (= KV page size on this path)
constexpr int ATT_CHUNK = kAttnChunk; // positions per attention work item (fixed: anchored at position 0)
constexpr int ERR_BAD_STATE = 3;

struct StepDesc {
    int n_cols;                // columns with a token (in flight + newest, over all sequences of the launch)
    int newest_mask;           // columns holding the newest token of their sequence
    int head_mask;             // newest columns that may consult intermediate heads in this step
    int pmax;                  // highest position of the step
    int fresh;                 // columns whose token enters at layer 1 in this step (their embedding is set up by the control point)
    int run_final;             // the step ends with the final head (0: a prompt pass that is not the last)
    int first_layer[MAX_COLS]; // 0-based layer at which the column resumes (INT_MAX: no token, or its sequence has left the step)
    int pos[MAX_COLS];
    int seq_pmax[MAX_COLS];    // per sequence of the launch: position of its newest token (-1: the sequence is not in this step)
};
static_assert(sizeof(StepDesc) <= 32 * sizeof(int), "the step descriptor must fit its shared-memory slot");

struct Pub {                   // what CTA 0 publishes at a control point
    unsigned seq;
    int action;
    StepDesc d;
    int pad[8];
};

struct MegaLayer {
    // wqkv: the fused q | k | v matrix with the rows of every q and k head reordered for the rotation (see the QKV phase);
    // wgu: gate stacked over up, or the gate matrix alone when wup is set (the two lent as separate tensors)
    const CUtensorMap *wqkv, *wo, *wgu, *wup, *wdown, *wT;
    const __nv_bfloat16 *attn_norm, *ffn_norm;
    float head_scale;
    int has_head;
};

struct MegaModel {
    const CUtensorMap *lm_head;
    const __nv_bfloat16 *tok_embed, *final_norm;
    float rope_base;
    int pad;
    MegaLayer layer[ADA_MAX_LAYERS + 1];   // [l] for 0-based layer l; head fields of 1-based layer e live in layer[e]
};

struct MegaArgs {
    Ctx c;
    const MegaModel *mm;
    const int *exit_at;        // [L + 1]: 1 + the index of 1-based layer e among the call's exit layers if the call consults its head, else 0
    __nv_bfloat16 *XA, *XB, *XO, *XH, *XF, *XT;   // GEMM inputs in fragment layout (see stream.cuh)
    float *ssq_a, *ssq_b;      // [d/16][8] partial sums of squares of the residual (per 16-feature tile, per column)
    uint32_t *qfrag;           // [nkv][2][hd/16][32][8]: rotated, scaled queries as tensor-core A fragments (bf16 high parts, then low parts)
    float *attn_part;          // [8 * nq][n_chunks][hd + 4]
    float *head_part;          // [grid][8][4]
    const double *rope_freq;   // [hd/2]: base^(-2i/hd), computed once on the host
    unsigned long long *part;  // [grid][8][256]: tagged partial sums of weight tiles split between two CTAs (null: none)
    unsigned *attn_cnt;        // [nkv]
    unsigned *grid_ctr;
    Pub *pub;                  // [2]
    int *err;
    int step_budget;           // steps this launch may start
    int seq0, nseq;            // the launch decodes sequences seq0 .. seq0 + nseq - 1 of the session together: sequence k of them owns the
                               // token columns [k slots, (k + 1) slots), slots = max_early + 1, nseq slots <= 8; they share every weight stream
    unsigned long long wait_ns;   // a single device-side wait gives up after this long
    int store_logits;
    // Sampled decoding (Eq. 1 with a drawn token, Eq. 2 with its acceptance test and the resampling): off = greedy
    int sampling;
    float inv_temp;            // 1 / temperature: every head's logits are multiplied by it
    const float *uniforms;     // [batch][max_seq][SAMPLE_NU]: the random numbers of the token at each sequence position
    float *q_stage;            // [batch][8][vocab]: logits of the intermediate head that drew the token after position p, slot p % 8
    float4 *qinfo;             // [batch][8]: (max logit, sum of exp, probability of the drawn token) of that head
    Trace trace;               // test hook: event trace of the steps [trace_step0, trace_step1) of this launch
    int trace_step0, trace_step1;
};

// ---------------------------------------------------------------- small helpers

__device__ __forceinline__ float ldcg(const float *p) { return __ldcg(p); }

__device__ __forceinline__ unsigned active_mask(const StepDesc &d, int layer) {
    unsigned m = 0;
#pragma unroll
    for (int c = 0; c < MAX_COLS; ++c) m |= (d.first_layer[c] <= layer ? 1u : 0u) << c;
    return m;
}

// rstd[c] = 1 / sqrt(sum_tiles ssq[tile][c] / d + eps), one warp per column, fixed summation order.
// RMSNorm factors 1/sqrt(mean square + eps) of the eight columns from the per-tile sums of squares
// ssq[tile][column], by the activation producer warp: lane l sums column l%8 over the tiles
// l/8 + 4u in ascending order (32 loads in flight), the four lanes of a column are folded by a
// butterfly.  The order is fixed, so the factor of a column does not depend on the other columns.
__device__ __forceinline__ void rstd_produce(Smem *sm, const float *ssq, int ntiles, int d, float eps, unsigned seq) {
    const int lane = threadIdx.x & 31, col = lane & 7, sub = lane >> 3;
    float s = 0.f;
    for (int t0 = 0; t0 < ntiles; t0 += 128) {
        float v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const int t = t0 + sub + 4 * u;
            v[u] = t < ntiles ? ldcg(ssq + (size_t)t * MAX_COLS + col) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 32; ++u) s += v[u];
    }
    s += __shfl_xor_sync(0xffffffffu, s, 8);
    s += __shfl_xor_sync(0xffffffffu, s, 16);
    if (lane < MAX_COLS) sm->vec[lane] = 1.0f / sqrtf(s / (float)d + eps);
    __threadfence_block();
    __syncwarp();
    if (lane == 0) *(volatile unsigned *)&sm->vec_seq = seq;
}

// Grid barrier as seen by the consumers of a CTA.
__device__ __forceinline__ void barrier_consumers(const Shared &S, unsigned *ctr, unsigned &bar_no, int G, int cls) {
    if (threadIdx.x == 0) trace(S, EV_EPI_END, cls);
    bar_consumers();
    ++bar_no;
    if (threadIdx.x == 0) {
        grid_arrive(ctr);
        trace(S, EV_ARRIVE, cls);
        grid_wait(S, ctr, bar_no * (unsigned)G);
        trace(S, EV_PHASE_BEGIN, cls);
    }
    bar_consumers();
}

// Merge the per-CTA (max, sum exp, argmax) partials of one column, by one whole warp: lane i folds
// CTAs i, i+32, ... in ascending order, then the lanes are folded by a butterfly (the merge is
// symmetric, so every lane ends with the same value).
__device__ __forceinline__ HeadResult merge_head(const float *head_part, int G, int col) {
    const int lane = threadIdx.x & 31;
    Msa a; a.m = -INFINITY; a.s = 0.f; a.i = INT_MAX;
    for (int b0 = lane; b0 < G; b0 += 32 * 8) {   // eight CTAs' partials in flight per lane, merged in ascending order
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int b = b0 + 32 * u;
            v[u] = b < G ? __ldcg(reinterpret_cast<const float4 *>(head_part + ((size_t)b * MAX_COLS + col) * 4)) : make_float4(-INFINITY, 0.f, __int_as_float(INT_MAX), 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (b0 + 32 * u < G) {
                Msa x; x.m = v[u].x; x.s = v[u].y; x.i = __float_as_int(v[u].z);
                a = msa_merge(a, x);
            }
        }
    }
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        Msa o;
        o.m = __shfl_xor_sync(0xffffffffu, a.m, off);
        o.s = __shfl_xor_sync(0xffffffffu, a.s, off);
        o.i = __shfl_xor_sync(0xffffffffu, a.i, off);
        a = msa_merge(a, o);
    }
    HeadResult hr; hr.token = a.i; hr.zmax = a.m; hr.sumexp = a.s; hr.p = 1.0f / a.s;
    return hr;
}

// ---------------------------------------------------------------- sampling (CTA 0, consumer warps)

// Random numbers per sequence position: [0] draw at the last layer, [1] acceptance test of Eq. 2, [2] resampling after a
// rejection, [3 + e] draw at the e-th exit layer of the call.
constexpr int SAMPLE_NU = 8;
constexpr int DRAW_CHUNK = 128;                 // vocabulary entries per partial sum
constexpr int DRAW_OFFSET = 12288;              // the draw's buffers sit in the consumers' scratch behind the control point's copies
constexpr int DRAW_MAX_CHUNKS = (SCRATCH_BYTES - DRAW_OFFSET - 4 * (CONS_THREADS + DRAW_CHUNK + 8)) / 4;
constexpr int DRAW_MAX_VOCAB = DRAW_MAX_CHUNKS * DRAW_CHUNK;

// Weights the draw is made from, in vocabulary order: exp(z - m) (a head's distribution up to its normaliser), or, with
// zq set, the positive part of exp(z - m) / s - exp(zq - mq) / sq (the distribution Eq. 2 resamples from, up to its normaliser).
struct DrawSrc {
    const float *z; float m, inv_s;
    const float *zq; float mq, inv_sq;
    __device__ __forceinline__ float weight_of(float zv, float qv) const {   // from the loaded logits (-inf: outside the vocabulary)
        const float a = __expf(zv - m);
        if (!zq) return a;
        return fmaxf(0.f, a * inv_s - __expf(qv - mq) * inv_sq);
    }
    __device__ __forceinline__ float weight(int v) const { return weight_of(__ldcg(z + v), zq ? __ldcg(zq + v) : 0.f); }
};

// Inverse-CDF draw by the consumer warps of one CTA: the first token, in vocabulary order, whose running sum of weights
// exceeds u x (sum of all weights); the last token of non-zero weight if rounding leaves none.  Returns the token to every
// thread (-1 if all weights are zero), with the sum of all weights and the drawn token's weight.  Partial sums per 128
// entries in a fixed order, so the result does not depend on timing.
__device__ __noinline__ int block_draw(Smem *sm, const DrawSrc &src, int V, float u, float &total, float &w_tok) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float *psum = reinterpret_cast<float *>(sm->scratch + DRAW_OFFSET);   // [CONS_THREADS]
    float *wbuf = psum + CONS_THREADS;                                     // [DRAW_CHUNK]
    float *res = wbuf + DRAW_CHUNK;                                        // token, its weight
    float *csum = res + 8;                                                 // [chunks]
    const int n_chunks = (V + DRAW_CHUNK - 1) / DRAW_CHUNK;
    // pass 1: the sum of every chunk (warp w takes chunks w, w + 8, ...; eight chunks' loads in flight)
    const bool vec = (V & 3) == 0;   // rows start on 16-byte boundaries: one 16-byte load per lane and chunk
    for (int c0 = warp; vec && c0 < n_chunks; c0 += CONS_WARPS * 8) {
        float4 zv[8], qv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int v = (c0 + j * CONS_WARPS) * DRAW_CHUNK + 4 * lane;
            const bool in = v < V;   // V is a multiple of 4: the four entries are inside together
            zv[j] = in ? __ldcg(reinterpret_cast<const float4 *>(src.z + v)) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            qv[j] = (src.zq && in) ? __ldcg(reinterpret_cast<const float4 *>(src.zq + v)) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float a = (src.weight_of(zv[j].x, qv[j].x) + src.weight_of(zv[j].y, qv[j].y)) + (src.weight_of(zv[j].z, qv[j].z) + src.weight_of(zv[j].w, qv[j].w));
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            const int ch = c0 + j * CONS_WARPS;
            if (lane == 0 && ch < n_chunks) csum[ch] = a;
        }
    }
    for (int c0 = warp; !vec && c0 < n_chunks; c0 += CONS_WARPS * 8) {
        // all 32 (or 64) loads of the lane first, then the arithmetic: one round trip to L2 per eight chunks, not one per entry
        float zv[8][DRAW_CHUNK / 32], qv[8][DRAW_CHUNK / 32];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int it = 0; it < DRAW_CHUNK / 32; ++it) {
                const int v = (c0 + j * CONS_WARPS) * DRAW_CHUNK + it * 32 + lane;
                zv[j][it] = v < V ? __ldcg(src.z + v) : -INFINITY;
                qv[j][it] = (src.zq && v < V) ? __ldcg(src.zq + v) : -INFINITY;
            }
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float a = 0.f;
#pragma unroll
            for (int it = 0; it < DRAW_CHUNK / 32; ++it) a += src.weight_of(zv[j][it], qv[j][it]);
            acc[j] = a;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float a = acc[j];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
            const int ch = c0 + j * CONS_WARPS;
            if (lane == 0 && ch < n_chunks) csum[ch] = a;
        }
    }
    bar_consumers();
    const int cpt = (n_chunks + CONS_THREADS - 1) / CONS_THREADS;   // chunks per thread of the second level
    {
        float a = 0.f;
        for (int j = 0; j < cpt; ++j) {
            const int ch = tid * cpt + j;
            a += ch < n_chunks ? csum[ch] : 0.f;
        }
        psum[tid] = a;
    }
    bar_consumers();
    // every thread walks the same two levels to the chunk that holds the crossing
    total = 0.f;
    for (int i = 0; i < CONS_THREADS; ++i) total += psum[i];
    w_tok = 0.f;
    if (!(total > 0.f)) return -1;
    const float target = u * total;
    float base = 0.f;
    int t_at = -1;
    for (int i = 0; i < CONS_THREADS; ++i) {
        if (base + psum[i] > target) { t_at = i; break; }
        base += psum[i];
    }
    int ch_at = -1;
    bool take_last = false;
    if (t_at >= 0) {
        for (int j = 0; j < cpt; ++j) {
            const int ch = t_at * cpt + j;
            if (ch >= n_chunks) break;
            if (base + csum[ch] > target) { ch_at = ch; break; }
            base += csum[ch];
        }
    }
    if (ch_at < 0) {   // rounding left no crossing: the last chunk of non-zero weight, its last such token
        take_last = true;
        for (int ch = n_chunks - 1; ch >= 0; --ch)
            if (csum[ch] > 0.f) { ch_at = ch; break; }
        if (ch_at < 0) return -1;
    }
    // pass 2: locate the token inside the chunk
    if (warp == 0) {
#pragma unroll
        for (int it = 0; it < DRAW_CHUNK / 32; ++it) {
            const int v = ch_at * DRAW_CHUNK + it * 32 + lane;
            wbuf[it * 32 + lane] = v < V ? src.weight(v) : 0.f;
        }
        __syncwarp();
        if (lane == 0) {
            float run = base;
            int tok = -1, last = -1;
            for (int i = 0; i < DRAW_CHUNK; ++i) {
                const float w = wbuf[i];
                if (w > 0.f) last = i;
                run += w;
                if (!take_last && run > target) { tok = i; break; }
            }
            if (tok < 0) tok = last < 0 ? 0 : last;
            res[0] = __int_as_float(ch_at * DRAW_CHUNK + tok);
            res[1] = wbuf[tok];
        }
    }
    bar_consumers();
    const int tok = __float_as_int(res[0]);
    w_tok = res[1];
    bar_consumers();   // the buffers may be rewritten by the next draw
    return tok;
}

// The same draw from a head's distribution exp(z - m), using what the head product already left behind: CTA b of the
// grid has published (max, sum of exp, argmax) of its own rows of the vocabulary, [16 t0(b), 16 t1(b)), a contiguous range in
// CTA order.  The running sum over the CTAs finds the CTA whose range holds the crossing; only that range's logits
// (vocabulary / grid entries) are read again.  Two round trips to L2 instead of a pass over the whole vocabulary by one CTA.
__device__ __noinline__ int block_draw_head(Smem *sm, const float *z, float m, const float *head_part, int col, int G, int V, float u,
                                            float &total, float &w_tok) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    float *psum = reinterpret_cast<float *>(sm->scratch + DRAW_OFFSET);   // second-level sums, then the located range
    float *wbuf = psum + CONS_THREADS;
    float *res = wbuf + DRAW_CHUNK;
    float *csum = res + 8;
    const int T = (V + 15) / 16;
    // (1) running sum over the CTAs' sums, by warp 0: lane l holds CTAs [l per, (l + 1) per)
    if (warp == 0) {
        const int per = (G + 31) / 32;
        float loc = 0.f;
        for (int k = 0; k < per; ++k) {
            const int b = lane * per + k;
            if (b < G) {
                const float4 v = __ldcg(reinterpret_cast<const float4 *>(head_part + ((size_t)b * MAX_COLS + col) * 4));
                loc += (v.x == -INFINITY) ? 0.f : v.y * __expf(v.x - m);
            }
        }
        float inc = loc;   // inclusive scan over the lanes
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float o = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += o;
        }
        const float tot = __shfl_sync(0xffffffffu, inc, 31);
        const float target = u * tot;
        const unsigned hit = __ballot_sync(0xffffffffu, inc > target);
        int l_at = hit ? __ffs(hit) - 1 : -1;
        bool take_last = false;
        if (l_at < 0) {   // rounding left no crossing: the last lane of non-zero sum
            const unsigned pos = __ballot_sync(0xffffffffu, loc > 0.f);
            l_at = pos ? 31 - __clz(pos) : -1;
            take_last = true;
        }
        if (lane == (l_at < 0 ? 0 : l_at)) {
            int b_at = -1;
            float base = inc - loc;
            if (l_at >= 0) {
                float run = base;
                int last_b = -1;
                for (int k = 0; k < per; ++k) {   // the lane walks its CTAs again (the same values, from L2)
                    const int b = lane * per + k;
                    if (b >= G) break;
                    const float4 v = __ldcg(reinterpret_cast<const float4 *>(head_part + ((size_t)b * MAX_COLS + col) * 4));
                    const float wv = (v.x == -INFINITY) ? 0.f : v.y * __expf(v.x - m);
                    if (wv > 0.f) last_b = b;
                    if (!take_last && run + wv > target) { b_at = b; base = run; break; }
                    run += wv;
                }
                if (b_at < 0) { b_at = last_b; take_last = true; base = 0.f; }
            }
            res[0] = __int_as_float(b_at);
            res[1] = base;
            res[2] = tot;
            res[3] = take_last ? 1.f : 0.f;
        }
    }
    bar_consumers();
    const int b_at = __float_as_int(res[0]);
    const float base = res[1];
    total = res[2];
    const bool take_last = res[3] != 0.f;
    w_tok = 0.f;
    if (b_at < 0 || !(total > 0.f)) { bar_consumers(); return -1; }
    const float target = u * total;
    int t0, t1;
    cta_tile_range(T, b_at, G, t0, t1);
    const int v0 = t0 * 16, v1 = min(V, t1 * 16), n_sub = (v1 - v0 + DRAW_CHUNK - 1) / DRAW_CHUNK;
    // (2) sums of the 128-entry pieces of that range (one per warp and turn)
    for (int sub = warp; sub < n_sub; sub += CONS_WARPS) {
        float a = 0.f;
#pragma unroll
        for (int it = 0; it < DRAW_CHUNK / 32; ++it) {
            const int v = v0 + sub * DRAW_CHUNK + it * 32 + lane;
            a += v < v1 ? __expf(__ldcg(z + v) - m) : 0.f;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
        if (lane == 0) csum[sub] = a;
    }
    bar_consumers();
    // (3) the piece that holds the crossing, then the entry inside it (warp 0; entries in vocabulary order)
    if (warp == 0) {
        float run = base;
        int sub_at = -1;
        bool tl = take_last;
        for (int sub = 0; sub < n_sub; ++sub) {
            if (!tl && run + csum[sub] > target) { sub_at = sub; break; }
            run += csum[sub];
        }
        if (sub_at < 0) {
            tl = true;
            for (int sub = n_sub - 1; sub >= 0; --sub)
                if (csum[sub] > 0.f) { sub_at = sub; break; }
        }
        int tok = -1;
        float wt = 0.f;
        if (sub_at >= 0) {
            // lane l holds the entries [4 l, 4 l + 4) of the piece
            float wv[4], loc = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int v = v0 + sub_at * DRAW_CHUNK + 4 * lane + i;
                wv[i] = v < v1 ? __expf(__ldcg(z + v) - m) : 0.f;
                loc += wv[i];
            }
            float inc = loc;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const float o = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += o;
            }
            const float before = run + inc - loc;
            int my = -1;
            float r2 = before;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                r2 += wv[i];
                if (my < 0 && !tl && r2 > target) my = i;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, my >= 0);
            int l_at, i_at;
            if (hit) {
                l_at = __ffs(hit) - 1;
                i_at = __shfl_sync(0xffffffffu, my, l_at);
            } else {   // the last entry of non-zero weight
                int lastp = -1;
#pragma unroll
                for (int i = 0; i < 4; ++i) if (wv[i] > 0.f) lastp = i;
                const unsigned pos = __ballot_sync(0xffffffffu, lastp >= 0);
                l_at = pos ? 31 - __clz(pos) : 0;
                i_at = max(__shfl_sync(0xffffffffu, lastp, l_at), 0);
            }
            float wsel = wv[0];
#pragma unroll
            for (int i = 1; i < 4; ++i) if (i == i_at) wsel = wv[i];
            wt = __shfl_sync(0xffffffffu, wsel, l_at);
            tok = v0 + sub_at * DRAW_CHUNK + 4 * l_at + i_at;
        }
        if (lane == 0) { res[4] = __int_as_float(tok); res[5] = wt; }
    }
    bar_consumers();
    const int tok = __float_as_int(res[4]);
    w_tok = res[5];
    bar_consumers();   // the buffers may be rewritten by the next draw
    return tok;
}

struct SampleArgs {
    const float *uniforms; float *q_stage; float4 *qinfo; const float *logit_stage; HeadResult *head_res; DevState *st;
    int vocab, max_seq, cps, L, seq0, nseq, exit_idx;
    const float *head_part; int G;   // the grid's per-CTA (max, sum of exp, argmax) of the head just evaluated
};

// Sampled decoding at a control point (its own function: its registers must not weigh on the streaming loops).
// After an intermediate head (Eq. 1): the newest token's successor is drawn from the head's distribution q; its
// probability q(t) is what the threshold test sees.  After the final head (Eq. 2): every early-predicted token t, in
// sequence order, is accepted with probability min{1, p*(t) / q(t)} -- the result stands in the column's head result as
// the token itself, so that the comparison of the bookkeeping accepts it -- and the first one that is not is replaced by
// a draw from Normalize(max(0, p* - q)); if all are accepted the next token is drawn from p* of the newest column.
__device__ __noinline__ void sample_stage(SampleArgs a, Smem *sm, bool after_head, const StepDesc *dprev, unsigned head_cols) {
    const int tid = threadIdx.x, V = a.vocab, cps = a.cps;
    HeadResult *hr_s = reinterpret_cast<HeadResult *>(sm->scratch + 8192);
    const int *tok_s = reinterpret_cast<const int *>(sm->scratch + 8192 + sizeof(HeadResult) * MAX_COLS);
    auto unif = [&](int s, int pos, int which) { return a.uniforms[((size_t)s * a.max_seq + pos) * SAMPLE_NU + which]; };
    if (after_head) {
        for (int col = 0; col < MAX_COLS; ++col) {
            if (!((head_cols >> col) & 1u)) continue;
            const int s = a.seq0 + (a.nseq == 1 ? 0 : col / cps), pos = dprev->pos[col], slot = s * MAX_COLS + (pos & 7);
            float total, wt;
            const int tok = block_draw_head(sm, a.q_stage + (size_t)slot * V, hr_s[col].zmax, a.head_part, col, a.G, V, unif(s, pos + 1, 3 + a.exit_idx), total, wt);
            if (tid == 0) {
                hr_s[col].token = max(tok, 0);
                hr_s[col].p = tok < 0 ? 0.f : wt / total;
                a.head_res[col] = hr_s[col];
                a.qinfo[slot] = make_float4(hr_s[col].zmax, total, hr_s[col].p, 0.f);
            }
        }
    } else {
        for (int k = 0; k < a.nseq; ++k) {
            const int s = a.seq0 + k, ln = a.st->len[s], bs = a.st->base[s], nrow = ln - bs, c0 = k * cps;
            if (nrow < 1 || nrow > cps || dprev->first_layer[c0 + nrow - 1] > a.L - 1) continue;
            bool rejected = false;
            for (int r = 0; r + 1 < nrow && !rejected; ++r) {
                const int col = c0 + r, pos_t = bs + r + 1, t = min(max(tok_s[col], 0), V - 1), slot = s * MAX_COLS + ((bs + r) & 7);
                const float *zs = a.logit_stage + (size_t)col * V;
                const float4 qi = a.qinfo[slot];
                const float ps = __expf(__ldcg(zs + t) - hr_s[col].zmax) / hr_s[col].sumexp;
                if (unif(s, pos_t, 1) * qi.z < ps) {   // accepted; every thread evaluates the same numbers
                    if (tid == 0) hr_s[col].token = t;
                    continue;
                }
                rejected = true;
                DrawSrc src{zs, hr_s[col].zmax, 1.f / hr_s[col].sumexp, a.q_stage + (size_t)slot * V, qi.x, 1.f / qi.y};
                float total, wt;
                int tok = block_draw(sm, src, V, unif(s, pos_t, 2), total, wt);
                if (tok < 0) {   // p* nowhere above q (they are equal up to rounding): draw from p*
                    DrawSrc plain{zs, hr_s[col].zmax, 0.f, nullptr, 0.f, 0.f};
                    tok = block_draw(sm, plain, V, unif(s, pos_t, 2), total, wt);
                }
                if (tid == 0) hr_s[col].token = max(tok, 0);
            }
            if (!rejected) {
                const int col = c0 + nrow - 1;
                float total, wt;
                const int tok = block_draw_head(sm, a.logit_stage + (size_t)col * V, hr_s[col].zmax, a.head_part, col, a.G, V, unif(s, ln, 0), total, wt);
                if (tid == 0) hr_s[col].token = max(tok, 0);
            }
        }
    }
    __threadfence_block();
    bar_consumers();
}

// ---------------------------------------------------------------- control point (CTA 0, consumer warps)

// Applies the outcome of the step that just ended (Eq. 1 after a head; verification and rollback,
// Eq. 2 at temperature zero, after the final head), then sets up the next step: its columns, the
// embedding of its newest token, that token's rotary table; finally publishes the action.
__device__ __forceinline__ void control_cta0(const MegaArgs &A, Smem *sm, int kind, int e, unsigned pub_no, const StepDesc &dprev,
                                          int &steps_started) {
    const Ctx &c = A.c;
    DevState *st = c.st;
    const MegaModel &M = *A.mm;
    const int tid = threadIdx.x, G = gridDim.x;
    const int nseq = A.nseq, seq0 = A.seq0, cps = c.slots, L = c.L;   // cps: token columns per sequence
    Pub *pub = A.pub + (pub_no & 1);
    // Shared-memory copies for the bookkeeping thread (fetched by many threads at once: a single
    // thread reading them from global memory one after the other spent 30 us here on round trips to L2):
    // the fill levels, the head results, and the tokens the verification compares with.
    int *fill_s = reinterpret_cast<int *>(sm->scratch);                                          // [nseq][L]
    HeadResult *hr_s = reinterpret_cast<HeadResult *>(sm->scratch + 8192);                       // [MAX_COLS]
    int *tok_s = reinterpret_cast<int *>(sm->scratch + 8192 + sizeof(HeadResult) * MAX_COLS);    // [MAX_COLS]: the token after the column's own
    static_assert(ADA_MAX_LAYERS * MAX_COLS * sizeof(int) <= 8192, "fill levels of a launch's sequences must fit the scratch corner");
    for (int i = tid; i < nseq * L; i += CONS_THREADS) fill_s[i] = c.fill[(size_t)seq0 * L + i];
    if (tid >= CONS_THREADS - MAX_COLS) {
        const int j = tid - (CONS_THREADS - MAX_COLS), k = j / cps;
        int v = -1;
        if (k < nseq) {
            const int at = st->base[seq0 + k] + (j - k * cps) + 1;
            if (at < c.max_seq) v = c.tokens[(size_t)(seq0 + k) * c.max_seq + at];
        }
        tok_s[j] = v;
    }
    // (a) head results of the columns that matter: warp w merges column w
    const unsigned head_cols = kind == CTRL_HEAD ? ((unsigned)dprev.head_mask & active_mask(dprev, e - 1))
                                                 : (kind == CTRL_TOP ? active_mask(dprev, L - 1) : 0u);
    if (kind != CTRL_START) {
        const int w = tid >> 5;
        if ((head_cols >> w) & 1u) {
            const HeadResult hr = merge_head(A.head_part, G, w);
            if ((tid & 31) == 0) { c.head_res[w] = hr; hr_s[w] = hr; }
        }
    }
    __threadfence_block();
    bar_consumers();
    // (a') sampled decoding replaces the tokens and probabilities the bookkeeping below works with
    if (A.sampling && kind != CTRL_START && !(kind == CTRL_TOP && st->pf_end > 0)) {
        SampleArgs sa{A.uniforms, A.q_stage, A.qinfo, c.logit_stage, c.head_res, st, c.vocab, c.max_seq, cps, L, seq0, nseq,
                      kind == CTRL_HEAD ? A.exit_at[e] - 1 : 0, A.head_part, G};
        sample_stage(sa, sm, kind == CTRL_HEAD, &dprev, head_cols);
    }
    // (b) bookkeeping, one thread.  Every scalar it may need is read up front (the loads overlap);
    // counters are bumped by reductions, which do not wait for memory.
    if (tid == 0) {
        auto bump = [](long long *p, long long v) { atomicAdd(reinterpret_cast<unsigned long long *>(p), (unsigned long long)v); };
        const int err0 = *(volatile int *)A.err;
        const int pf_end0 = st->pf_end, pf_pos0 = st->pf_pos, max_early0 = st->max_early;
        const int tape_n0 = st->tape_n, hl_n0 = st->head_log_n;
        int tape_i = st->tape_i, hl_n = hl_n0;
        const float gamma0 = st->gamma;
        const int eos0 = st->eos_id;
        const long long steps0 = __ldcg(&st->st.steps);   // past the L1: the counters are bumped by reductions
        int len[MAX_COLS], base[MAX_COLS], target[MAX_COLS], done[MAX_COLS];
#pragma unroll
        for (int k = 0; k < MAX_COLS; ++k) {
            const bool in = k < nseq;
            len[k] = in ? st->len[seq0 + k] : 0; base[k] = in ? st->base[seq0 + k] : 0;
            target[k] = in ? st->target_len[seq0 + k] : 0; done[k] = in ? st->done[seq0 + k] : 1;
        }
        int action = ACT_NEWSTEP, verified = 0;
        int pf_end = pf_end0, pf_pos = pf_pos0;
        StepDesc nd = dprev;
        if (err0 != 0) action = ACT_STOP;
        // ---- Eq. 1 after an intermediate head: every sequence whose newest token consulted it decides for itself
        if (action != ACT_STOP && kind == CTRL_HEAD) {
            unsigned still = 0;   // sequences that go on climbing in this step
            int n_steps_seen = 0;
            for (int k = 0; k < nseq; ++k) {
                const int s = seq0 + k, col = k * cps + (len[k] - 1 - base[k]);
                if (col < 0 || col >= MAX_COLS || dprev.first_layer[col] > e - 1) continue;   // not in this step any more
                if (!((head_cols >> col) & 1u)) { still |= 1u << k; continue; }                // climbing, but may not exit early
                const HeadResult hr = hr_s[col];
                bool decide = hr.p > gamma0;
                if (s == 0 && tape_i < tape_n0) {
                    const uint8_t t = st->tape[tape_i++];
                    if (t == 0) decide = false;
                    if (t == 1) decide = true;
                }
                bump(&st->st.head_evals, 1);
                if (s == 0 && c.head_log && hl_n < kHeadLogCap) {
                    float *hl = c.head_log + 4 * (size_t)hl_n;
                    hl[0] = (float)(steps0 + n_steps_seen); hl[1] = (float)e; hl[2] = (float)hr.token; hl[3] = hr.p;
                    ++hl_n;
                }
                if (!decide) { still |= 1u << k; continue; }
                long long rl = 0;
                for (int l = 0; l < e; ++l) {
                    rl += len[k] - fill_s[k * L + l];
                    fill_s[k * L + l] = len[k];
                    c.fill[(size_t)s * L + l] = len[k];
                }
                bump(&st->st.row_layers, rl);
                c.tokens[(size_t)s * c.max_seq + len[k]] = min(max(hr.token, 0), c.vocab - 1);
                len[k] += 1;
                st->len[s] = len[k];
                bump(&st->st.early_exits, 1);
                bump(&st->st.exits_at_layer[e], 1);
                bump(&st->st.steps, 1);
                ++n_steps_seen;
                for (int j = 0; j < cps; ++j) nd.first_layer[k * cps + j] = INT_MAX;   // the sequence sits out the rest of the step
                nd.head_mask &= ~(((1 << cps) - 1) << (k * cps));
            }
            if (tape_i != st->tape_i) st->tape_i = tape_i;
            if (hl_n != hl_n0) st->head_log_n = hl_n;
            if (still) action = ACT_CONTINUE;
            else bump(&st->st.layer_passes, e);   // the weights of layers 1..e were streamed once, for all the sequences
        }
        const bool prefilling = pf_end > 0;
        if (action != ACT_STOP && kind == CTRL_TOP && prefilling) {
            // a pass over prompt positions [pf_pos, pf_pos + n) of the launch's one sequence is complete at every layer
            const int s = seq0, n = dprev.n_cols, end = pf_pos + n;
            for (int l = 0; l < L; ++l) { fill_s[l] = end; c.fill[(size_t)s * L + l] = end; }
            pf_pos = end;
            st->pf_pos = end;
            if (end >= pf_end) {   // KV cache <- LM(x) done: the full-depth argmax at the last prompt token is the first generated token
                const int np = pf_end;
                c.tokens[(size_t)s * c.max_seq + np] = min(max(hr_s[n - 1].token, 0), c.vocab - 1);
                len[0] = np + 1; base[0] = np; done[0] = 1; pf_end = 0;
                st->len[s] = np + 1;
                st->base[s] = np;
                st->n_prompt[s] = np;
                st->done[s] = 1;
                st->pf_end = 0;
                st->keep_rows = 1;
                st->keep_row0 = n - 1;
                verified = s == 0;
            }
        }
        // ---- verification (Eq. 2 at temperature zero) of every sequence whose newest token reached the last layer
        if (action != ACT_STOP && kind == CTRL_TOP && !prefilling) {
            for (int k = 0; k < nseq; ++k) {
                const int s = seq0 + k, nrow = len[k] - base[k], c0 = k * cps;
                if (nrow < 1 || nrow > cps || dprev.first_layer[c0 + nrow - 1] > L - 1) continue;   // left the step at an exit layer, or idle
                int32_t *tok = c.tokens + (size_t)s * c.max_seq;
                long long rl = 0;
                for (int l = 0; l < L; ++l) rl += len[k] - fill_s[k * L + l];
                bump(&st->st.row_layers, rl);
                int bad = -1;
                for (int j = 0; j + 1 < nrow; ++j)
                    if (hr_s[c0 + j].token != tok_s[c0 + j]) { bad = j; break; }
                int new_base, keep;
                if (bad < 0) {
                    bump(&st->st.accepted, nrow - 1);
                    tok[len[k]] = min(max(hr_s[c0 + nrow - 1].token, 0), c.vocab - 1);
                    new_base = len[k];
                    keep = nrow;
                } else {
                    bump(&st->st.accepted, bad);
                    bump(&st->st.rejected, 1);
                    bump(&st->st.discarded, nrow - 2 - bad);
                    new_base = base[k] + bad + 1;
                    tok[new_base] = min(max(hr_s[c0 + bad].token, 0), c.vocab - 1);
                    keep = bad + 1;
                }
                // Algorithm 1 runs "while t_i != [EOS]": the verified tokens of this step (positions base + 1 .. new_base,
                // each equal to the full-depth argmax of the row before it) end the sequence at the first end-of-sequence
                // token among them.  An early-predicted end-of-sequence token stops nothing until it is verified here.
                int tgt = target[k];
                if (eos0 >= 0) {
                    for (int j = 0; j < keep; ++j)
                        if (min(max(hr_s[c0 + j].token, 0), c.vocab - 1) == eos0) {
                            if (base[k] + j + 2 <= tgt) { tgt = base[k] + j + 2; st->eos_hit[s] = 1; }
                            break;
                        }
                }
                int new_len = new_base + 1;
                if (new_len > tgt) {
                    bump(&st->st.truncated, new_len - tgt);
                    new_len = tgt;
                    new_base = new_len - 1;
                }
                keep = new_len - 1 - base[k];   // verified tokens that stay: their logit rows are the ones a capture keeps
                for (int l = 0; l < L; ++l) { fill_s[k * L + l] = new_base; c.fill[(size_t)s * L + l] = new_base; }
                len[k] = new_len; base[k] = new_base;
                st->len[s] = new_len;
                st->base[s] = new_base;
                bump(&st->st.verify_steps, 1);
                bump(&st->st.steps, 1);
                if (new_len >= tgt) { done[k] = 1; st->done[s] = 1; }
                if (s == 0) {
                    st->keep_rows = keep;
                    st->keep_row0 = 0;
                    verified = 1;
                }
            }
        }
        if (action != ACT_STOP && kind == CTRL_TOP && !prefilling) bump(&st->st.layer_passes, L);
        if (action == ACT_NEWSTEP) {
            bool all_done = true;
            for (int k = 0; k < nseq; ++k) all_done = all_done && done[k];
            if (all_done) { action = ACT_STOP; st->n_done = 1; }
            else if (steps_started >= A.step_budget) action = ACT_STOP;
        }
        if (action == ACT_NEWSTEP) {
            ++steps_started;
            nd.n_cols = 0; nd.newest_mask = 0; nd.head_mask = 0; nd.pmax = 0; nd.fresh = 0; nd.run_final = 1;
            for (int j = 0; j < MAX_COLS; ++j) { nd.first_layer[j] = INT_MAX; nd.pos[j] = 0; nd.seq_pmax[j] = -1; }
            if (pf_end > 0) {   // next pass over the prompt: up to eight positions, all from layer 1
                const int n = min(MAX_COLS, pf_end - pf_pos);
                nd.n_cols = n;
                nd.newest_mask = 1 << (n - 1);
                nd.pmax = pf_pos + n - 1;
                nd.seq_pmax[0] = nd.pmax;
                nd.fresh = (1 << n) - 1;
                nd.run_final = pf_pos + n >= pf_end;
                if (n < 1 || nd.pmax >= c.max_seq) {
                    atomicCAS(A.err, 0, ERR_BAD_STATE);
                    action = ACT_STOP;
                }
                for (int j = 0; j < n; ++j) { nd.first_layer[j] = 0; nd.pos[j] = pf_pos + j; }
            } else {
                for (int k = 0; k < nseq; ++k) {
                    if (done[k]) continue;   // a sequence that has reached its target idles while the others go on
                    const int nrow = len[k] - base[k], c0 = k * cps;
                    if (nrow < 1 || nrow > cps || c0 + nrow > MAX_COLS || len[k] > c.max_seq || base[k] < 0) {
                        atomicCAS(A.err, 0, ERR_BAD_STATE);
                        action = ACT_STOP;
                        break;
                    }
                    for (int j = 0; j < nrow; ++j) {
                        const int pos = base[k] + j;
                        int fl = 0;
                        for (int l = 0; l < L; ++l) fl += fill_s[k * L + l] > pos;
                        nd.first_layer[c0 + j] = fl;
                        nd.pos[c0 + j] = pos;
                    }
                    const int cn = c0 + nrow - 1;
                    nd.n_cols += nrow;
                    nd.newest_mask |= 1 << cn;
                    nd.fresh |= 1 << cn;
                    if (nrow - 1 < max_early0 && len[k] < target[k]) nd.head_mask |= 1 << cn;
                    nd.seq_pmax[k] = len[k] - 1;
                    nd.pmax = max(nd.pmax, len[k] - 1);
                }
            }
        }
        if (action == ACT_NEWSTEP || action == ACT_CONTINUE) pub->d = nd;
        pub->action = action;
        sm->bcast[0] = action;
        sm->bcast[3] = verified;
    }
    bar_consumers();
    const int action = sm->bcast[0];
    // (c) logits of the verified rows (test hook), then the embedding of the next newest token
    if (kind == CTRL_TOP && c.capture && sm->bcast[3]) {
        const int keep = st->keep_rows, at = st->capture_n;
        for (int j = 0; j < keep && at + j < st->capture_cap; ++j) {
            const float *src = c.logit_stage + (size_t)(st->keep_row0 + j) * c.vocab;
            float *dst = c.capture + (size_t)(at + j) * c.vocab;
            for (int i = tid; i < c.vocab; i += CONS_THREADS) dst[i] = __ldcg(src + i);
        }
        bar_consumers();
        if (tid == 0) st->capture_n = min(st->capture_cap, at + keep);
    }
    if (action == ACT_NEWSTEP) {
        const StepDesc &nd = pub->d;
        const __nv_bfloat16 *g0 = M.layer[0].attn_norm;
        const int half = c.hd / 2;
        for (int col = 0; col < MAX_COLS; ++col) {
            if (!((nd.fresh >> col) & 1)) continue;
            const int pos = nd.pos[col];
            const int tokid = min(max(c.tokens[(size_t)(seq0 + (nseq == 1 ? 0 : col / cps)) * c.max_seq + pos], 0), c.vocab - 1);
            const __nv_bfloat16 *erow = M.tok_embed + (size_t)tokid * c.d;
            for (int n0 = 0; n0 < c.d; n0 += 8 * CONS_THREADS) {   // eight loads of the embedding row and of the gain in flight per thread
                float v[8], gn[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int n = n0 + u * CONS_THREADS + tid;
                    v[u] = n < c.d ? __bfloat162float(erow[n]) : 0.f;
                    gn[u] = n < c.d ? __bfloat162float(g0[n]) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int n = n0 + u * CONS_THREADS + tid;
                    if (n < c.d) {
                        c.resid[(size_t)col * c.d + n] = v[u];
                        xfrag_store(A.XA, n, col, v[u] * gn[u]);
                    }
                    float q = v[u] * v[u];
                    q += __shfl_xor_sync(0xffffffffu, q, 1);
                    q += __shfl_xor_sync(0xffffffffu, q, 2);
                    q += __shfl_xor_sync(0xffffffffu, q, 4);
                    q += __shfl_xor_sync(0xffffffffu, q, 8);
                    if ((tid & 15) == 0 && n < c.d) A.ssq_a[(size_t)(n >> 4) * MAX_COLS + col] = q;
                }
            }
            for (int i = tid; i < half; i += CONS_THREADS) {
                // angle = pos * freq in double, reduced to [-pi, pi] in double, then single-precision sin / cos
                // (double-precision transcendentals with large arguments are slow on this GPU)
                const double a = (double)pos * A.rope_freq[i];
                const double r = a - 6.283185307179586476925 * rint(a * 0.15915494309189533577);
                float sn, cs;
                sincosf((float)r, &sn, &cs);
                c.rope_cs[((size_t)col * half + i) * 2 + 0] = cs;
                c.rope_cs[((size_t)col * half + i) * 2 + 1] = sn;
            }
        }
    }
    __threadfence();
    fence_proxy_async();
    bar_consumers();
    if (tid == 0) {
        __threadfence();
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&pub->seq), "r"(pub_no) : "memory");
    }
}

// Every role of every CTA passes here; returns the action and (for a new step) the descriptor.
template <int ROLE>
__device__ __forceinline__ int control_point(const MegaArgs &A, const Shared &S, int kind, int e, unsigned &pub_no, StepDesc &d,
                                             int &steps_started) {
    Smem *sm = S.sm;
    ++pub_no;
    const Pub *pub = A.pub + (pub_no & 1);
    int action;
    // the new step descriptor is copied into the role's shared copy `d` by one thread (by every lane of a
    // producer warp: same values), and checked before anything is indexed with it
    auto fetch = [&]() -> int {
        int act = aborted(S) ? ACT_STOP : *(volatile const int *)&pub->action;
        if (act == ACT_NEWSTEP || act == ACT_CONTINUE) {   // a step that goes on may have lost the columns of sequences that left it
            const volatile int *src = reinterpret_cast<const volatile int *>(&pub->d);
            int *dst = reinterpret_cast<int *>(&d);
#pragma unroll
            for (int i = 0; i < (int)(sizeof(StepDesc) / 4); ++i) dst[i] = src[i];
            bool bad = d.n_cols < 1 || d.n_cols > MAX_COLS || d.pmax < 0 || d.pmax >= A.c.max_seq;
#pragma unroll
            for (int i = 0; i < MAX_COLS; ++i) bad = bad || d.pos[i] < 0 || d.pos[i] >= A.c.max_seq || d.seq_pmax[i] >= A.c.max_seq;
            if (bad) act = ACT_STOP;   // cannot happen unless memory was corrupted; never index with it
        }
        // The two record slots alternate.  A role that fell two control points behind would find its slot
        // already rewritten for a later one: a record is used only if its number is still the expected one
        // after it has been copied.
        if (!aborted(S) && ld_acquire(&pub->seq) != pub_no) {
            raise_error(S, ERR_BAD_STATE);
            act = ACT_STOP;
        }
        return act;
    };
    if (ROLE == 2) {
        if (blockIdx.x == 0) {
            control_cta0(A, sm, kind, e, pub_no, d, steps_started);
            bar_consumers();   // every thread is done with the old descriptor before thread 0 replaces it
        }
        if (threadIdx.x == 0) {
            grid_wait(S, &pub->seq, pub_no);
            sm->bcast[1] = fetch();
        }
        bar_consumers();
        action = sm->bcast[1];
    } else {
        grid_wait(S, &pub->seq, pub_no);
        action = fetch();
        __syncwarp();
    }
    return action;
}

// ---------------------------------------------------------------- attention phase

// Shared memory of the attention phase, carved from the consumers' scratch.  The query fragments
// are dead once the last score tile of an item is computed; the merge buffers reuse their space.
template <int HD> struct AttnSmem {
    union {
        uint32_t qfrag[2][HD / 16][32][8];   // A fragments of the rotated, scaled queries: hi a0..a3, lo a0..a3
        float o[2][2][16][HD];               // merge buffers [query tile][source]
    };
    float ml[2][2][2][16];                   // [query tile][source][max | sum][row]
};
static_assert(sizeof(AttnSmem<128>) <= SCRATCH_BYTES, "attention buffers exceed the consumers' scratch");

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Attention work items of a launch that holds several sequences: sequence k of the launch (token columns
// [k cps, (k + 1) cps); all eight in a prompt pass, which holds one sequence) contributes n_kv_heads x its
// own number of 128-position chunks, and an item works on that sequence's columns and cache pages only.
__device__ __forceinline__ unsigned seq_cols(const MegaArgs &A, int k) {
    return A.nseq == 1 ? 0xffu : (((1u << A.c.slots) - 1u) << (k * A.c.slots));
}
__device__ __forceinline__ int seq_chunks(const MegaArgs &A, const StepDesc &d, unsigned mask, int k) {
    return ((mask & seq_cols(A, k)) != 0 && d.seq_pmax[k] >= 0) ? d.seq_pmax[k] / ATT_CHUNK + 1 : 0;
}
__device__ __forceinline__ int attn_items(const MegaArgs &A, const StepDesc &d, unsigned mask) {
    int n = 0;
    for (int k = 0; k < A.nseq; ++k) n += A.c.nkv * seq_chunks(A, d, mask, k);
    return n;
}
// item -> (sequence of the launch, kv head, chunk); nchunk = the sequence's chunk count
__device__ __forceinline__ void attn_item(const MegaArgs &A, const StepDesc &d, unsigned mask, int item, int &k, int &kvh, int &j, int &nchunk) {
    k = 0;
    nchunk = seq_chunks(A, d, mask, 0);
    while (k + 1 < A.nseq && item >= A.c.nkv * nchunk) {
        item -= A.c.nkv * nchunk;
        ++k;
        nchunk = seq_chunks(A, d, mask, k);
    }
    nchunk = max(nchunk, 1);
    kvh = min(item / nchunk, A.c.nkv - 1);
    j = item - kvh * nchunk;
}

// Query tiles (16 (column, q head) pairs each) that hold a pair of the columns mk: bit t = tile t.
__device__ __forceinline__ unsigned seq_tiles(const MegaArgs &A, unsigned mk) {
    unsigned t = 0;
#pragma unroll
    for (int cc = 0; cc < MAX_COLS; ++cc)
        if ((mk >> cc) & 1u) t |= (1u << ((cc * A.c.group) >> 4)) | (1u << ((cc * A.c.group + A.c.group - 1) >> 4));
    return t & 3u;
}
// The consumers are two groups of four warps.  Where an item's queries span both tiles, group t works on tile t
// of the same item.  Where every sequence's queries fit one tile (plain decoding; few columns; one q head per kv
// head) the second group would idle: the groups then take DIFFERENT items, two per round, which halves the rounds
// of a CTA that owns several items.  Which warps compute an item never changes what is computed.
__device__ __forceinline__ bool attn_dual(const MegaArgs &A, unsigned mask) {
    bool dual = true;
    for (int k = 0; k < A.nseq; ++k) {
        const unsigned t = seq_tiles(A, mask & seq_cols(A, k));
        dual = dual && t != 3u;
    }
    return dual;
}
// One item of a round as every role sees it.
struct AttnItem {
    int k, kvh, j, nchunk, nsb, p_base, qt;   // sequence of the launch, kv head, chunk, the sequence's chunks, 64-position sub-blocks, first position, query tile
    unsigned mk;                              // the sequence's active columns
    bool have;
};
__device__ __forceinline__ AttnItem attn_item_of(const MegaArgs &A, const StepDesc &d, unsigned mask, int item, int n_items, bool dual, int grp) {
    AttnItem it;
    it.have = item < n_items;
    it.k = it.kvh = it.j = it.nsb = it.p_base = it.qt = 0; it.nchunk = 1; it.mk = 0;
    if (!it.have) return it;
    attn_item(A, d, mask, item, it.k, it.kvh, it.j, it.nchunk);
    it.mk = mask & seq_cols(A, it.k);
    it.p_base = it.j * ATT_CHUNK;
    it.nsb = min(ATT_CHUNK / ATT_PAGE, (d.seq_pmax[it.k] - it.p_base) / ATT_PAGE + 1);
    it.qt = dual ? ((seq_tiles(A, it.mk) & 1u) ? 0 : 1) : grp;
    return it;
}

// K/V producer: for every work item of this CTA, the K and V page blocks of its sub-blocks, in the order the
// consumers walk them: per round (one item, or two in the dual arrangement) sub-block by sub-block, K of every
// item of the round, then V.  The K and V rows of the tokens of this pass were written into the cache by the QKV
// epilogues of other CTAs; an item whose positions include such a row is fetched only once the grid has passed
// the barrier that ends the QKV phase (`bar_target`).  Every other item reads rows of earlier passes only and is
// fetched as soon as ring slots are free, i.e. while the QKV product is still streaming.
__device__ __forceinline__ void attn_produce(const MegaArgs &A, const Shared &S, const StepDesc &d, int layer, unsigned mask, unsigned bar_target,
                                             Rings &r, uint64_t pol) {
    const Ctx &c = A.c;
    Smem *sm = S.sm;
    const int lane = threadIdx.x & 31, cta = blockIdx.x, G = gridDim.x;
    const int n_items = attn_items(A, d, mask);
    const bool dual = attn_dual(A, mask);
    const int per_round = dual ? 2 : 1;
    const uint32_t bytes = (uint32_t)(ATT_PAGE * c.hd * 2);
    const __nv_bfloat16 *pool = reinterpret_cast<const __nv_bfloat16 *>(c.kv_pool);
    bool synced = false;
    if (lane == 0) trace(S, EV_ATT, 8);
    for (int it0 = cta; it0 < n_items; it0 += G * per_round) {
        AttnItem it[2];
        it[0] = attn_item_of(A, d, mask, it0, n_items, dual, 0);
        it[1] = attn_item_of(A, d, mask, dual ? it0 + G : n_items, n_items, dual, 1);
        bool has_new = false;
#pragma unroll
        for (int g = 0; g < 2; ++g)
#pragma unroll
            for (int cc = 0; cc < MAX_COLS; ++cc)
                has_new = has_new || (it[g].have && ((it[g].mk >> cc) & 1u) && d.pos[cc] >= it[g].p_base && d.pos[cc] < it[g].p_base + ATT_CHUNK);
        if (has_new && !synced) {
            grid_wait(S, A.grid_ctr, bar_target);
            fence_proxy_async();
            synced = true;
        }
        const int nsb = max(it[0].nsb, it[1].nsb);
        for (int sb = 0; sb < nsb; ++sb)
            for (int which = 0; which < 2; ++which)
                for (int g = 0; g < per_round; ++g) {
                    if (!it[g].have || sb >= it[g].nsb) continue;
                    const int32_t *pages = c.page_table + (size_t)(A.seq0 + it[g].k) * c.max_pages;
                    const int page = pages[(it[g].p_base + sb * ATT_PAGE) >> c.page_shift];
                    const int slot = r.xi % NX;
                    mbar_wait(S, &sm->x_empty[slot], ((r.xi / NX) & 1) ^ 1);
                    if (lane == 0 && !aborted(S)) {
                        const size_t blk = ((((size_t)page * c.L + layer) * 2 + which) * c.nkv + it[g].kvh) * ((size_t)ATT_PAGE * c.hd);
                        mbar_expect_tx(&sm->x_full[slot], bytes);
                        bulk_g2s(sm->x[slot], pool + blk, bytes, &sm->x_full[slot], pol);
                        trace(S, EV_ATT, 9 + 16 * (2 * sb + which));
                    }
                    ++r.xi;
                }
    }
}

// The producer of a phase in which no CTA owns more than one item (see attn_consume_single).
__device__ __forceinline__ void attn_produce_single(const MegaArgs &A, const Shared &S, const StepDesc &d, int layer, unsigned mask, unsigned bar_target,
                                             Rings &r, uint64_t pol) {
    const Ctx &c = A.c;
    Smem *sm = S.sm;
    const int lane = threadIdx.x & 31, cta = blockIdx.x, G = gridDim.x;
    const int n_items = attn_items(A, d, mask);
    const uint32_t bytes = (uint32_t)(ATT_PAGE * c.hd * 2);
    const __nv_bfloat16 *pool = reinterpret_cast<const __nv_bfloat16 *>(c.kv_pool);
    bool synced = false;
    if (lane == 0) trace(S, EV_ATT, 8);
    for (int item = cta; item < n_items; item += G) {
        int k, kvh, j, nchunk;
        attn_item(A, d, mask, item, k, kvh, j, nchunk);
        const unsigned mk = mask & seq_cols(A, k);
        const int32_t *pages = c.page_table + (size_t)(A.seq0 + k) * c.max_pages;
        const int p_base = j * ATT_CHUNK;
        const int nsb = min(ATT_CHUNK / ATT_PAGE, (d.seq_pmax[k] - p_base) / ATT_PAGE + 1);
        bool has_new = false;
#pragma unroll
        for (int cc = 0; cc < MAX_COLS; ++cc)
            has_new = has_new || (((mk >> cc) & 1u) && d.pos[cc] >= p_base && d.pos[cc] < p_base + ATT_CHUNK);
        if (has_new && !synced) {
            grid_wait(S, A.grid_ctr, bar_target);
            fence_proxy_async();
            synced = true;
        }
        for (int sb = 0; sb < nsb; ++sb) {
            const int page = pages[(p_base + sb * ATT_PAGE) >> c.page_shift];
            for (int which = 0; which < 2; ++which) {
                const int slot = r.xi % NX;
                mbar_wait(S, &sm->x_empty[slot], ((r.xi / NX) & 1) ^ 1);
                if (lane == 0 && !aborted(S)) {
                    const size_t blk = ((((size_t)page * c.L + layer) * 2 + which) * c.nkv + kvh) * ((size_t)ATT_PAGE * c.hd);
                    mbar_expect_tx(&sm->x_full[slot], bytes);
                    bulk_g2s(sm->x[slot], pool + blk, bytes, &sm->x_full[slot], pol);
                    trace(S, EV_ATT, 9 + 16 * (2 * sb + which));
                }
                ++r.xi;
            }
        }
    }
}

// Merge (max, sum, unnormalised output) of another warp, read from shared memory, into this warp's.
template <int NT, int HD>
__device__ __forceinline__ void attn_merge_from(float (&o)[NT][4], float (&m_run)[2], float (&l_run)[2], const float (*so)[HD],
                                                const float (*sml)[16], int lane) {
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
        const int row = (lane >> 2) + 8 * rh;
        const float ms = sml[0][row], ls = sml[1][row];
        const float mn = fmaxf(m_run[rh], ms);
        float a = 1.f, b = 0.f;
        if (mn != -INFINITY) { a = __expf(m_run[rh] - mn); b = __expf(ms - mn); }
        m_run[rh] = mn;
        l_run[rh] = l_run[rh] * a + ls * b;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {   // columns rotated by 8 (row % 8): conflict-free 8-byte accesses
            const float2 v = *reinterpret_cast<const float2 *>(&so[row][(nt * 8 + 2 * (lane & 3) + 8 * (row & 7)) & (HD - 1)]);
            o[nt][2 * rh] = o[nt][2 * rh] * a + v.x * b;
            o[nt][2 * rh + 1] = o[nt][2 * rh + 1] * a + v.y * b;
        }
    }
}
template <int NT, int HD>
__device__ __forceinline__ void attn_merge_to(const float (&o)[NT][4], const float (&m_run)[2], const float (&l_run)[2], float (*so)[HD],
                                              float (*sml)[16], int lane) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            const int row = (lane >> 2) + 8 * rh;
            *reinterpret_cast<float2 *>(&so[row][(nt * 8 + 2 * (lane & 3) + 8 * (row & 7)) & (HD - 1)]) = make_float2(o[nt][2 * rh], o[nt][2 * rh + 1]);
        }
    if ((lane & 3) == 0) {
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            sml[0][(lane >> 2) + 8 * rh] = m_run[rh];
            sml[1][(lane >> 2) + 8 * rh] = l_run[rh];
        }
    }
}

// Consumers: causal attention of every active column over the cache, which by now holds the rows
// of this pass too (the QKV epilogue wrote them).  Work item = (kv head, 128-position chunk).
// Within a 64-position sub-block warp (mt, qr) handles query tile mt (16 of the up to 32 (column,
// q head) pairs of the kv head) and positions [16 qr, 16 qr + 16).  The queries arrive rotated,
// scaled and split into bf16 high / low parts, laid out as the tensor-core A fragments.
// x / group for the q heads per kv head the persistent path admits (1..4) and x < 128, without the
// general integer division (some thirty of those sat on the critical path of every attention item)
__device__ __forceinline__ int div_group(int x, int group) {
    return group == 4 ? x >> 2 : group == 2 ? x >> 1 : group == 1 ? x : (x * 43) >> 7;
}

// The same for a phase in which no CTA owns more than one item (contexts up to about 128 positions x CTAs / kv heads:
// the common case of short and medium contexts): one item, its two query tiles on the two warp groups, merged by
// whichever CTA completes a head last.  Kept as a path of its own: the general form below, with its rounds of two
// items, costs this case 2-4 % of the step.
template <int HD>
__device__ __forceinline__ void attn_consume_single(const MegaArgs &A, const Shared &S, const StepDesc &d, int layer, unsigned mask, Rings &r) {
    const Ctx &c = A.c;
    Smem *sm = S.sm;
    AttnSmem<HD> *as = reinterpret_cast<AttnSmem<HD> *>(sm->scratch);
    constexpr int KSQ = HD / 16, NT = HD / 8;
    constexpr int ATT_STRIDE = HD + 4;                     // floats per chunk partial: output, max, sum, padding (16-byte rows)
    constexpr int QV = 2 * KSQ * 64 / CONS_THREADS;        // 16-byte pieces of a kv head's query fragments per thread
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, cta = blockIdx.x, G = gridDim.x;
    const int group = c.group;
    const int n_items = attn_items(A, d, mask);
    const int mt = warp >> 2, qr = warp & 3;
    (void)layer;
    // Merge of the chunk partials of one kv head into the O-projection's input (by a whole CTA).
    auto merge_chunks = [&](int kvh, unsigned mk) {   // mk: the active columns of the work item's sequence
        // Four features of one (column, q head) per thread and pass; the chunk partials are folded in
        // ascending order, eight at a time with all their loads in flight, by the usual running-max rule.
        const int nqc = MAX_COLS * group;
        for (int idx = tid; idx < nqc * (HD / 4); idx += CONS_THREADS) {
            const int qcol = idx / (HD / 4), dim = (idx - qcol * (HD / 4)) * 4, cc = div_group(qcol, group), g = qcol - cc * group;
            if (!((mk >> cc) & 1u)) continue;
            const int h = kvh * group + g;
            const int nch = d.pos[cc] / ATT_CHUNK + 1;
            const float *part = A.attn_part + (((size_t)cc * c.nq + h) * c.n_chunks) * ATT_STRIDE;
            float Mx = -INFINITY, den = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int k0 = 0; k0 < nch; k0 += 8) {
                float2 ml[8];
                float4 ov[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const bool ok = k0 + u < nch;
                    const float *pk = part + (size_t)(k0 + u) * ATT_STRIDE;
                    ml[u] = ok ? __ldcg(reinterpret_cast<const float2 *>(pk + HD)) : make_float2(-INFINITY, 0.f);
                    ov[u] = ok ? __ldcg(reinterpret_cast<const float4 *>(pk + dim)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float Mn = Mx;
#pragma unroll
                for (int u = 0; u < 8; ++u) Mn = fmaxf(Mn, ml[u].x);
                if (Mn == -INFINITY) continue;
                const float sc = Mx == -INFINITY ? 0.f : __expf(Mx - Mn);
                den *= sc; acc.x *= sc; acc.y *= sc; acc.z *= sc; acc.w *= sc;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (ml[u].x != -INFINITY) {
                        const float w = __expf(ml[u].x - Mn);
                        den += ml[u].y * w;
                        acc.x += ov[u].x * w; acc.y += ov[u].y * w; acc.z += ov[u].z * w; acc.w += ov[u].w * w;
                    }
                }
                Mx = Mn;
            }
            xfrag_store(A.XO, h * HD + dim, cc, acc.x / den);
            xfrag_store(A.XO, h * HD + dim + 1, cc, acc.y / den);
            xfrag_store(A.XO, h * HD + dim + 2, cc, acc.z / den);
            xfrag_store(A.XO, h * HD + dim + 3, cc, acc.w / den);
        }
    };
    // With at most one work item per CTA the CTA that completes a head last merges it at once; with more,
    // designated CTAs do (see below).  Who merges does not change what is computed.
    const bool last_arriver_merges = true;   // at most one item per CTA (the caller's condition)
    for (int item = cta; item < n_items; item += G) {
        int ks_, kvh, j, nchunk;
        attn_item(A, d, mask, item, ks_, kvh, j, nchunk);
        const unsigned mk = mask & seq_cols(A, ks_);   // the item's sequence: its columns only
        const int p_base = j * ATT_CHUNK;
        const int nsb = min(ATT_CHUNK / ATT_PAGE, (d.seq_pmax[ks_] - p_base) / ATT_PAGE + 1);
        // ---- the kv head's query fragments: one round trip to L2, then shared memory
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(A.qfrag) + (size_t)kvh * (2 * KSQ * 64);
            uint4 v[QV];
#pragma unroll
            for (int u = 0; u < QV; ++u) v[u] = __ldcg(src + tid + u * CONS_THREADS);
            bar_consumers();   // the previous item is done with the shared buffers
#pragma unroll
            for (int u = 0; u < QV; ++u) reinterpret_cast<uint4 *>(&as->qfrag[0][0][0][0])[tid + u * CONS_THREADS] = v[u];
        }
        bar_consumers();
        if (tid == 0) trace(S, EV_ATT, 2);   // queries ready
        // ---- per-warp online softmax state: rows (lane/4) and (lane/4)+8 of query tile mt
        int lim[2];
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            const int qcol = mt * 16 + (lane >> 2) + rh * 8, cc = div_group(qcol, group);
            lim[rh] = (cc < MAX_COLS && ((mk >> cc) & 1u)) ? d.pos[cc] : -1;
        }
        // a query tile none of whose 16 (column, q head) pairs is in use does no arithmetic (uniform per warp)
        bool tile_used = false;
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int cc = div_group(mt * 16 + q, group);
            tile_used = tile_used || (cc < MAX_COLS && ((mk >> cc) & 1u));
        }
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
        float o[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[nt][i] = 0.f;
        for (int sb = 0; sb < nsb; ++sb) {
            const int p0 = p_base + sb * ATT_PAGE;
            float s[2][4];
            {   // ---- K block
                const int slot = r.xi % NX;
                mbar_wait(S, &sm->x_full[slot], (r.xi / NX) & 1);
                if (tid == 0) trace(S, EV_ATT, 3 + 16 * sb);   // K block landed
                const unsigned char *kb = sm->x[slot];
                float sh[2][4], sl[2][4];
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) { sh[nt][i] = 0.f; sl[nt][i] = 0.f; }
                const int id = lane >> 3;
                const int pl = 16 * qr + (lane & 7) + 8 * (id >> 1);
                const unsigned char *krow = kb + pl * (HD * 2);
                if (tile_used)
#pragma unroll
                for (int k0 = 0; k0 < KSQ; k0 += 4) {   // four k-steps of loads in flight, then their multiply-adds
                    uint4 qh[4], ql[4];
                    uint32_t kf[4][4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int ks = k0 + u;
                        qh[u] = *reinterpret_cast<const uint4 *>(&as->qfrag[mt][ks][lane][0]);
                        ql[u] = *reinterpret_cast<const uint4 *>(&as->qfrag[mt][ks][lane][4]);
                        ldmatrix_x4(kf[u], krow + ((((2 * ks) | (id & 1)) ^ (pl & 7)) << 4));
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t ah[4] = {qh[u].x, qh[u].y, qh[u].z, qh[u].w}, al[4] = {ql[u].x, ql[u].y, ql[u].z, ql[u].w};
                        mma16816(sh[0], ah, kf[u][0], kf[u][1]);
                        mma16816(sh[1], ah, kf[u][2], kf[u][3]);
                        mma16816(sl[0], al, kf[u][0], kf[u][1]);
                        mma16816(sl[1], al, kf[u][2], kf[u][3]);
                    }
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int pos = p0 + 16 * qr + 8 * nt + 2 * (lane & 3) + (i & 1);
                        s[nt][i] = pos <= lim[i >> 1] ? sh[nt][i] + sl[nt][i] : -INFINITY;
                    }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->x_empty[slot]);
                ++r.xi;
            }
            // ---- online softmax over this warp's 16 positions
            uint32_t ph[4], plo[4];
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                float mx = fmaxf(fmaxf(s[0][2 * rh], s[0][2 * rh + 1]), fmaxf(s[1][2 * rh], s[1][2 * rh + 1]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float mn = fmaxf(m_run[rh], mx);
                float corr = 1.f, p[4] = {0.f, 0.f, 0.f, 0.f};
                if (mn != -INFINITY) {
                    corr = __expf(m_run[rh] - mn);
                    p[0] = __expf(s[0][2 * rh] - mn); p[1] = __expf(s[0][2 * rh + 1] - mn);
                    p[2] = __expf(s[1][2 * rh] - mn); p[3] = __expf(s[1][2 * rh + 1] - mn);
                }
                m_run[rh] = mn;
                l_run[rh] = l_run[rh] * corr + ((p[0] + p[1]) + (p[2] + p[3]));
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) { o[nt][2 * rh] *= corr; o[nt][2 * rh + 1] *= corr; }
                // A fragment of P: a0/a1 = n-tile 0 (rows r / r+8), a2/a3 = n-tile 1
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(p[0], p[1]), h1 = __floats2bfloat162_rn(p[2], p[3]);
                ph[rh] = *reinterpret_cast<const uint32_t *>(&h0);
                ph[2 + rh] = *reinterpret_cast<const uint32_t *>(&h1);
                plo[rh] = pack_bf16(p[0] - __low2float(h0), p[1] - __high2float(h0));
                plo[2 + rh] = pack_bf16(p[2] - __low2float(h1), p[3] - __high2float(h1));
            }
            {   // ---- V block
                const int slot = r.xi % NX;
                mbar_wait(S, &sm->x_full[slot], (r.xi / NX) & 1);
                if (tid == 0) trace(S, EV_ATT, 4 + 16 * sb);   // V block landed
                const unsigned char *vb = sm->x[slot];
                const int id = lane >> 3;
                const int pl = 16 * qr + (lane & 7) + 8 * (id & 1);
                const unsigned char *vrow = vb + pl * (HD * 2);
                if (tile_used)
#pragma unroll
                for (int n0 = 0; n0 < NT / 2; n0 += 4) {
                    uint32_t vf[4][4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) ldmatrix_x4_trans(vf[u], vrow + ((((2 * (n0 + u)) | (id >> 1)) ^ (pl & 7)) << 4));
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int np = n0 + u;
                        mma16816(o[2 * np], ph, vf[u][0], vf[u][1]);
                        mma16816(o[2 * np + 1], ph, vf[u][2], vf[u][3]);
                        mma16816(o[2 * np], plo, vf[u][0], vf[u][1]);
                        mma16816(o[2 * np + 1], plo, vf[u][2], vf[u][3]);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->x_empty[slot]);
                ++r.xi;
            }
        }
        // ---- row sums over the quad, then merge the four position quarters of each query tile:
        //      (q0 + q1) and (q2 + q3), then the two halves
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            l_run[rh] += __shfl_xor_sync(0xffffffffu, l_run[rh], 1);
            l_run[rh] += __shfl_xor_sync(0xffffffffu, l_run[rh], 2);
        }
        if (tid == 0) trace(S, EV_ATT, 5);   // sub-blocks done
        bar_consumers();   // every warp is done with the query fragments, whose space the merge reuses
        // (a query tile without a query in use skips the merge: its warps only keep the barriers)
        if ((qr & 1) && tile_used) attn_merge_to<NT, HD>(o, m_run, l_run, as->o[mt][qr >> 1], as->ml[mt][qr >> 1], lane);
        bar_consumers();
        if (!(qr & 1) && tile_used) attn_merge_from<NT, HD>(o, m_run, l_run, as->o[mt][qr >> 1], as->ml[mt][qr >> 1], lane);
        bar_consumers();
        if (qr == 2 && tile_used) attn_merge_to<NT, HD>(o, m_run, l_run, as->o[mt][0], as->ml[mt][0], lane);
        bar_consumers();
        if (qr == 0) {
            if (tile_used) attn_merge_from<NT, HD>(o, m_run, l_run, as->o[mt][0], as->ml[mt][0], lane);
            // ---- chunk partial (unnormalised output, max, sum) of every valid (column, q head)
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const int qcol = mt * 16 + (lane >> 2) + 8 * rh, cc = div_group(qcol, group), g = qcol - cc * group;
                if (cc < MAX_COLS && ((mk >> cc) & 1u) && d.pos[cc] >= p_base) {
                    float *out = A.attn_part + (((size_t)cc * c.nq + kvh * group + g) * c.n_chunks + j) * ATT_STRIDE;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        *reinterpret_cast<float2 *>(out + nt * 8 + 2 * (lane & 3)) = make_float2(o[nt][2 * rh], o[nt][2 * rh + 1]);
                    if ((lane & 3) == 0) *reinterpret_cast<float2 *>(out + HD) = make_float2(m_run[rh], l_run[rh]);
                }
            }
        }
        // ---- this item's partials are complete: count it (a release that returns nothing, so nobody waits for it)
        if (tid == 0) trace(S, EV_ITEM, item);
        bar_consumers();
        if (last_arriver_merges) {
            if (tid == 0) {   // release this block's partials and acquire the others' in one step
                unsigned old;
                asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(A.attn_cnt + ks_ * c.nkv + kvh) : "memory");
                sm->bcast[2] = (int)old;
            }
            bar_consumers();
            if (sm->bcast[2] == nchunk - 1) {
                merge_chunks(kvh, mk);
                if (tid == 0) { A.attn_cnt[ks_ * c.nkv + kvh] = 0u; trace(S, EV_COMBINE, kvh); }
            }
        } else if (tid == 0) {
            __threadfence();
            red_release_add(A.attn_cnt + ks_ * c.nkv + kvh, 1u);
        }
    }
}

template <int HD>
__device__ __forceinline__ void attn_consume(const MegaArgs &A, const Shared &S, const StepDesc &d, int layer, unsigned mask, Rings &r) {
    const Ctx &c = A.c;
    Smem *sm = S.sm;
    AttnSmem<HD> *as = reinterpret_cast<AttnSmem<HD> *>(sm->scratch);
    constexpr int KSQ = HD / 16, NT = HD / 8;
    constexpr int ATT_STRIDE = HD + 4;                     // floats per chunk partial: output, max, sum, padding (16-byte rows)
    constexpr int QV = KSQ * 64 / (CONS_THREADS / 2);      // 16-byte pieces of one query tile's fragments per thread of a warp group
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, cta = blockIdx.x, G = gridDim.x;
    const int group = c.group;
    const int n_items = attn_items(A, d, mask);
    const int mt = warp >> 2, qr = warp & 3;
    (void)layer;
    // Merge of the chunk partials of one kv head into the O-projection's input (by a whole CTA).
    auto merge_chunks = [&](int kvh, unsigned mk) {   // mk: the active columns of the work item's sequence
        // Four features of one (column, q head) per thread and pass; the chunk partials are folded in
        // ascending order, eight at a time with all their loads in flight, by the usual running-max rule.
        const int nqc = MAX_COLS * group;
        for (int idx = tid; idx < nqc * (HD / 4); idx += CONS_THREADS) {
            const int qcol = idx / (HD / 4), dim = (idx - qcol * (HD / 4)) * 4, cc = div_group(qcol, group), g = qcol - cc * group;
            if (!((mk >> cc) & 1u)) continue;
            const int h = kvh * group + g;
            const int nch = d.pos[cc] / ATT_CHUNK + 1;
            const float *part = A.attn_part + (((size_t)cc * c.nq + h) * c.n_chunks) * ATT_STRIDE;
            float Mx = -INFINITY, den = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int k0 = 0; k0 < nch; k0 += 8) {
                float2 ml[8];
                float4 ov[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const bool ok = k0 + u < nch;
                    const float *pk = part + (size_t)(k0 + u) * ATT_STRIDE;
                    ml[u] = ok ? __ldcg(reinterpret_cast<const float2 *>(pk + HD)) : make_float2(-INFINITY, 0.f);
                    ov[u] = ok ? __ldcg(reinterpret_cast<const float4 *>(pk + dim)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                float Mn = Mx;
#pragma unroll
                for (int u = 0; u < 8; ++u) Mn = fmaxf(Mn, ml[u].x);
                if (Mn == -INFINITY) continue;
                const float sc = Mx == -INFINITY ? 0.f : __expf(Mx - Mn);
                den *= sc; acc.x *= sc; acc.y *= sc; acc.z *= sc; acc.w *= sc;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (ml[u].x != -INFINITY) {
                        const float w = __expf(ml[u].x - Mn);
                        den += ml[u].y * w;
                        acc.x += ov[u].x * w; acc.y += ov[u].y * w; acc.z += ov[u].z * w; acc.w += ov[u].w * w;
                    }
                }
                Mx = Mn;
            }
            xfrag_store(A.XO, h * HD + dim, cc, acc.x / den);
            xfrag_store(A.XO, h * HD + dim + 1, cc, acc.y / den);
            xfrag_store(A.XO, h * HD + dim + 2, cc, acc.z / den);
            xfrag_store(A.XO, h * HD + dim + 3, cc, acc.w / den);
        }
    };
    // With at most one work item per CTA the CTA that completes a head last merges it at once; with more,
    // designated CTAs do (see below).  Who merges does not change what is computed.
    const bool last_arriver_merges = n_items <= G;
    // Rounds: one item whose two query tiles go to the two warp groups, or (every sequence's queries in one tile) two
    // items, one per group.  Every warp walks the ring stages of the whole round in order and releases each of them;
    // it multiplies only those of its own group's item.
    const bool dual = attn_dual(A, mask);
    const int per_round = dual ? 2 : 1;
    for (int it0 = cta; it0 < n_items; it0 += G * per_round) {
        AttnItem itg[2];
        itg[0] = attn_item_of(A, d, mask, it0, n_items, dual, 0);
        itg[1] = attn_item_of(A, d, mask, dual ? it0 + G : it0, n_items, dual, 1);
        const AttnItem me = itg[mt];
        const int kvh = me.kvh, j = me.j, p_base = me.p_base, qt = me.qt;
        const unsigned mk = me.mk;   // the item's sequence: its columns only
        // ---- query tile qt of the item's kv head, by this warp group: one round trip to L2, then shared memory
        {
            const uint4 *src = reinterpret_cast<const uint4 *>(A.qfrag) + (size_t)kvh * (2 * KSQ * 64) + (size_t)qt * (KSQ * 64);
            const int gt = tid & (CONS_THREADS / 2 - 1);
            uint4 v[QV];
#pragma unroll
            for (int u = 0; u < QV; ++u) v[u] = me.have ? __ldcg(src + gt + u * (CONS_THREADS / 2)) : make_uint4(0u, 0u, 0u, 0u);
            bar_consumers();   // the previous round is done with the shared buffers
#pragma unroll
            for (int u = 0; u < QV; ++u) reinterpret_cast<uint4 *>(&as->qfrag[mt][0][0][0])[gt + u * (CONS_THREADS / 2)] = v[u];
        }
        bar_consumers();
        if (tid == 0) trace(S, EV_ATT, 2);   // queries ready
        // ---- per-warp online softmax state: rows (lane/4) and (lane/4)+8 of query tile qt
        int lim[2];
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            const int qcol = qt * 16 + (lane >> 2) + rh * 8, cc = div_group(qcol, group);
            lim[rh] = (me.have && cc < MAX_COLS && ((mk >> cc) & 1u)) ? d.pos[cc] : -1;
        }
        // a query tile none of whose 16 (column, q head) pairs is in use does no arithmetic (uniform per warp)
        bool tile_used = false;
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int cc = div_group(qt * 16 + q, group);
            tile_used = tile_used || (cc < MAX_COLS && ((mk >> cc) & 1u));
        }
        tile_used = tile_used && me.have;
        float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
        float o[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[nt][i] = 0.f;
        const int nsb = max(itg[0].nsb, dual ? itg[1].nsb : 0);
        for (int sb = 0; sb < nsb; ++sb) {
            const int p0 = p_base + sb * ATT_PAGE;
            const bool act = me.have && sb < me.nsb;   // this warp's item has this sub-block
            float s[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) s[nt][i] = -INFINITY;
#pragma unroll 1
            for (int g = 0; g < per_round; ++g) {   // ---- K block(s)
                if (!itg[g].have || sb >= itg[g].nsb) continue;
                const int slot = r.xi % NX;
                mbar_wait(S, &sm->x_full[slot], (r.xi / NX) & 1);
                if (tid == 0) trace(S, EV_ATT, 3 + 16 * sb);   // K block landed
                if (!dual || g == mt) {
                    const unsigned char *kb = sm->x[slot];
                    float sh[2][4], sl[2][4];
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) { sh[nt][i] = 0.f; sl[nt][i] = 0.f; }
                    const int id = lane >> 3;
                    const int pl = 16 * qr + (lane & 7) + 8 * (id >> 1);
                    const unsigned char *krow = kb + pl * (HD * 2);
                    if (tile_used)
#pragma unroll
                    for (int k0 = 0; k0 < KSQ; k0 += 4) {   // four k-steps of loads in flight, then their multiply-adds
                        uint4 qh[4], ql[4];
                        uint32_t kf[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int ks = k0 + u;
                            qh[u] = *reinterpret_cast<const uint4 *>(&as->qfrag[mt][ks][lane][0]);
                            ql[u] = *reinterpret_cast<const uint4 *>(&as->qfrag[mt][ks][lane][4]);
                            ldmatrix_x4(kf[u], krow + ((((2 * ks) | (id & 1)) ^ (pl & 7)) << 4));
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const uint32_t ah[4] = {qh[u].x, qh[u].y, qh[u].z, qh[u].w}, al[4] = {ql[u].x, ql[u].y, ql[u].z, ql[u].w};
                            mma16816(sh[0], ah, kf[u][0], kf[u][1]);
                            mma16816(sh[1], ah, kf[u][2], kf[u][3]);
                            mma16816(sl[0], al, kf[u][0], kf[u][1]);
                            mma16816(sl[1], al, kf[u][2], kf[u][3]);
                        }
                    }
#pragma unroll
                    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int pos = p0 + 16 * qr + 8 * nt + 2 * (lane & 3) + (i & 1);
                            s[nt][i] = pos <= lim[i >> 1] ? sh[nt][i] + sl[nt][i] : -INFINITY;
                        }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->x_empty[slot]);
                ++r.xi;
            }
            // ---- online softmax over this warp's 16 positions
            uint32_t ph[4] = {0u, 0u, 0u, 0u}, plo[4] = {0u, 0u, 0u, 0u};
            if (act) {
#pragma unroll
                for (int rh = 0; rh < 2; ++rh) {
                    float mx = fmaxf(fmaxf(s[0][2 * rh], s[0][2 * rh + 1]), fmaxf(s[1][2 * rh], s[1][2 * rh + 1]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float mn = fmaxf(m_run[rh], mx);
                    float corr = 1.f, p[4] = {0.f, 0.f, 0.f, 0.f};
                    if (mn != -INFINITY) {
                        corr = __expf(m_run[rh] - mn);
                        p[0] = __expf(s[0][2 * rh] - mn); p[1] = __expf(s[0][2 * rh + 1] - mn);
                        p[2] = __expf(s[1][2 * rh] - mn); p[3] = __expf(s[1][2 * rh + 1] - mn);
                    }
                    m_run[rh] = mn;
                    l_run[rh] = l_run[rh] * corr + ((p[0] + p[1]) + (p[2] + p[3]));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) { o[nt][2 * rh] *= corr; o[nt][2 * rh + 1] *= corr; }
                    // A fragment of P: a0/a1 = n-tile 0 (rows r / r+8), a2/a3 = n-tile 1
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(p[0], p[1]), h1 = __floats2bfloat162_rn(p[2], p[3]);
                    ph[rh] = *reinterpret_cast<const uint32_t *>(&h0);
                    ph[2 + rh] = *reinterpret_cast<const uint32_t *>(&h1);
                    plo[rh] = pack_bf16(p[0] - __low2float(h0), p[1] - __high2float(h0));
                    plo[2 + rh] = pack_bf16(p[2] - __low2float(h1), p[3] - __high2float(h1));
                }
            }
#pragma unroll 1
            for (int g = 0; g < per_round; ++g) {   // ---- V block(s)
                if (!itg[g].have || sb >= itg[g].nsb) continue;
                const int slot = r.xi % NX;
                mbar_wait(S, &sm->x_full[slot], (r.xi / NX) & 1);
                if (tid == 0) trace(S, EV_ATT, 4 + 16 * sb);   // V block landed
                if (!dual || g == mt) {
                    const unsigned char *vb = sm->x[slot];
                    const int id = lane >> 3;
                    const int pl = 16 * qr + (lane & 7) + 8 * (id & 1);
                    const unsigned char *vrow = vb + pl * (HD * 2);
                    if (tile_used)
#pragma unroll
                    for (int n0 = 0; n0 < NT / 2; n0 += 4) {
                        uint32_t vf[4][4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) ldmatrix_x4_trans(vf[u], vrow + ((((2 * (n0 + u)) | (id >> 1)) ^ (pl & 7)) << 4));
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int np = n0 + u;
                            mma16816(o[2 * np], ph, vf[u][0], vf[u][1]);
                            mma16816(o[2 * np + 1], ph, vf[u][2], vf[u][3]);
                            mma16816(o[2 * np], plo, vf[u][0], vf[u][1]);
                            mma16816(o[2 * np + 1], plo, vf[u][2], vf[u][3]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->x_empty[slot]);
                ++r.xi;
            }
        }
        // ---- row sums over the quad, then merge the four position quarters of each warp group:
        //      (q0 + q1) and (q2 + q3), then the two halves
#pragma unroll
        for (int rh = 0; rh < 2; ++rh) {
            l_run[rh] += __shfl_xor_sync(0xffffffffu, l_run[rh], 1);
            l_run[rh] += __shfl_xor_sync(0xffffffffu, l_run[rh], 2);
        }
        if (tid == 0) trace(S, EV_ATT, 5);   // sub-blocks done
        bar_consumers();   // every warp is done with the query fragments, whose space the merge reuses
        // (a query tile without a query in use skips the merge: its warps only keep the barriers)
        if ((qr & 1) && tile_used) attn_merge_to<NT, HD>(o, m_run, l_run, as->o[mt][qr >> 1], as->ml[mt][qr >> 1], lane);
        bar_consumers();
        if (!(qr & 1) && tile_used) attn_merge_from<NT, HD>(o, m_run, l_run, as->o[mt][qr >> 1], as->ml[mt][qr >> 1], lane);
        bar_consumers();
        if (qr == 2 && tile_used) attn_merge_to<NT, HD>(o, m_run, l_run, as->o[mt][0], as->ml[mt][0], lane);
        bar_consumers();
        if (qr == 0) {
            if (tile_used) attn_merge_from<NT, HD>(o, m_run, l_run, as->o[mt][0], as->ml[mt][0], lane);
            // ---- chunk partial (unnormalised output, max, sum) of every valid (column, q head)
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const int qcol = qt * 16 + (lane >> 2) + 8 * rh, cc = div_group(qcol, group), g = qcol - cc * group;
                if (me.have && cc < MAX_COLS && ((mk >> cc) & 1u) && d.pos[cc] >= p_base) {
                    float *out = A.attn_part + (((size_t)cc * c.nq + kvh * group + g) * c.n_chunks + j) * ATT_STRIDE;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
                        *reinterpret_cast<float2 *>(out + nt * 8 + 2 * (lane & 3)) = make_float2(o[nt][2 * rh], o[nt][2 * rh + 1]);
                    if ((lane & 3) == 0) *reinterpret_cast<float2 *>(out + HD) = make_float2(m_run[rh], l_run[rh]);
                }
            }
        }
        // ---- the round's partials are complete: count its items (a release that returns nothing, so nobody waits for it)
        if (tid == 0) trace(S, EV_ITEM, it0);
        bar_consumers();
        if (last_arriver_merges) {   // at most one item per CTA: the round holds item it0 alone
            const int cnt = itg[0].k * c.nkv + itg[0].kvh;
            if (tid == 0) {   // release this block's partials and acquire the others' in one step
                unsigned old;
                asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(A.attn_cnt + cnt) : "memory");
                sm->bcast[2] = (int)old;
            }
            bar_consumers();
            if (sm->bcast[2] == itg[0].nchunk - 1) {
                merge_chunks(itg[0].kvh, itg[0].mk);
                if (tid == 0) { A.attn_cnt[cnt] = 0u; trace(S, EV_COMBINE, itg[0].kvh); }
            }
        } else if (tid == 0 || (dual && tid == CONS_THREADS / 2)) {
            const AttnItem &mine = itg[tid == 0 ? 0 : 1];
            if (mine.have) {
                __threadfence();
                red_release_add(A.attn_cnt + mine.k * c.nkv + mine.kvh, 1u);
            }
        }
    }
    if (last_arriver_merges) return;
    // ---- The chunk partials of kv head h are merged by one designated CTA, G - 1 - h (the high CTAs
    // have the fewest work items), once all nchunk items of the head have been counted.  (Letting
    // whichever CTA arrives last do it looks cheaper but piles up at long contexts: the CTA that
    // merges one head is late for its next item, so it is last again for the next head, and ends up
    // merging every head in turn while the rest of the grid waits.)
    for (int hk = G - 1 - cta; hk < A.nseq * c.nkv; hk += G) {   // (sequence of the launch, kv head) pairs of this CTA
        const int ks_ = hk / c.nkv, kvh = hk - ks_ * c.nkv, nchunk = seq_chunks(A, d, mask, ks_);
        if (nchunk == 0) continue;
        if (tid == 0) grid_wait(S, A.attn_cnt + hk, (unsigned)nchunk);
        bar_consumers();
        {
            merge_chunks(kvh, mask & seq_cols(A, ks_));
            if (tid == 0) { A.attn_cnt[hk] = 0u; trace(S, EV_COMBINE, kvh); }
        }
        bar_consumers();   // the next head's wait must not start before every thread is done with this one
    }
}

// ---------------------------------------------------------------- the walker

template <int ROLE, int PAIR, class Epi>
__device__ __forceinline__ void gemm_phase(const Shared &S, const Gemm &g, Rings &r, uint64_t pol, Epi &&epi) {
    const int cta = blockIdx.x, G = gridDim.x;
    if (ROLE == 0) gemm_produce_w(S, g, cta, G, r, pol);
    else if (ROLE == 1) gemm_produce_x(S, g, cta, G, r, pol);
    else gemm_consume<PAIR>(S, g, cta, G, r, epi);
}

struct NoEpi {
    template <class T> __device__ __forceinline__ void operator()(int, T &) const {}
};

// ROLE 0: weight producer warp, 1: activation / KV producer warp, 2: consumer warps.
template <int ROLE, int HD>
__device__ __forceinline__ void run(const MegaArgs &A, Shared &S) {
    const Ctx &c = A.c;
    const MegaModel &M = *A.mm;
    Smem *sm = S.sm;
    const int G = gridDim.x, lane = threadIdx.x & 31;
    const int L = c.L, d_model = c.d, qd = c.nq * c.hd, ntd = d_model / 16;
    const uint64_t pol = ROLE == 0 ? policy_evict_first() : policy_evict_last();
    Rings r{0, 0};
    unsigned bar_no = 0, pub_no = 0;
    int steps_started = 0;
    // CTAs that share the tiles of each kind of GEMM (the rest idle through that phase)
    const int n_qkv = balanced_ctas((c.qkv_rows + 15) / 16, G), n_d = balanced_ctas(ntd, G), n_gu = balanced_ctas(c.dff / 16, G),
              n_head = balanced_ctas((c.vocab + 15) / 16, G);
    // The step descriptor lives in shared memory, one copy per role (the roles pass a control point at
    // different times): indexed by a run-time column it would otherwise sit in local memory, whose
    // cached lines do not survive the acquire of a grid barrier -- every first touch after a barrier
    // then costs a round trip to L2 on the critical path.
    StepDesc &d = *reinterpret_cast<StepDesc *>(sm->desc[ROLE]);
    if (ROLE != 2 || threadIdx.x == 0) {
        d.n_cols = 0; d.newest_mask = 0; d.head_mask = 0; d.pmax = 0; d.fresh = 0; d.run_final = 1;
#pragma unroll
        for (int i = 0; i < MAX_COLS; ++i) { d.first_layer[i] = INT_MAX; d.pos[i] = 0; d.seq_pmax[i] = -1; }
    }
    if (ROLE == 2) bar_consumers(); else __syncwarp();

    // barrier between phases, per role; CTA 0 books the time since the previous one to the phase's class
    unsigned long long t_last = gtime();
    auto phase_barrier = [&](int cls) {
        if (ROLE == 2) {
            barrier_consumers(S, A.grid_ctr, bar_no, G, cls);
            if (blockIdx.x == 0 && threadIdx.x == 0) {
                const unsigned long long t = gtime();
                // reductions, not read-modify-write: thread 0 of CTA 0 must not wait for a load from L2 at every barrier
                atomicAdd(reinterpret_cast<unsigned long long *>(&c.st->st.phase_ns[cls]), t - t_last);
                atomicAdd(reinterpret_cast<unsigned long long *>(&c.st->st.phase_count[cls]), 1ull);
                t_last = t;
            }
        } else ++bar_no;
    };
    auto book_control = [&]() {
        if (ROLE == 2 && blockIdx.x == 0 && threadIdx.x == 0) {
            const unsigned long long t = gtime();
            atomicAdd(reinterpret_cast<unsigned long long *>(&c.st->st.phase_ns[0]), t - t_last);
            atomicAdd(reinterpret_cast<unsigned long long *>(&c.st->st.phase_count[0]), 1ull);
            t_last = t;
        }
    };
    // the activation producer must not fetch a phase's input before the phase that wrote it is complete
    auto x_ready = [&]() {
        if (ROLE == 1) {
            grid_wait(S, A.grid_ctr, bar_no * (unsigned)G);
            fence_proxy_async();
        }
    };
    // head over E* with the fused (max, sum exp, argmax) reduction; X = final-normed residual (or T output)
    auto head_phase = [&](const __nv_bfloat16 *X, const float *ssq, float scale, unsigned cols, bool inter) {
        Gemm g; g.W = M.lm_head; g.X = reinterpret_cast<const uint4 *>(X); g.N = c.vocab; g.K = d_model; g.pair = 1; g.half = 0; g.ctas = n_head; g.part = nullptr; g.phase_id = bar_no + 1; g.columns(cols);
        x_ready();
        const unsigned vseq = bar_no + 1;
        if (ROLE == 2) {
            Msa run[2];
            run[0].m = run[1].m = -INFINITY; run[0].s = run[1].s = 0.f; run[0].i = run[1].i = INT_MAX;
            const int c0 = 2 * (lane & 3);
            // sampled decoding: logits over the temperature; they are kept, the final head's by column, an intermediate
            // head's by the position of its row (the verification of the token drawn from them needs them again)
            if (A.sampling) scale *= A.inv_temp;
            float *zrow[2] = {nullptr, nullptr};
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int col = c0 + q;
                if (!((cols >> col) & 1u)) continue;
                if (A.sampling && inter) zrow[q] = A.q_stage + ((size_t)(A.seq0 + (A.nseq == 1 ? 0 : col / c.slots)) * MAX_COLS + (d.pos[col] & 7)) * c.vocab;
                else if (A.sampling || A.store_logits) zrow[q] = c.logit_stage + (size_t)col * c.vocab;
            }
            float r0 = scale, r1 = scale;
            bool have_r = ssq == nullptr;
            gemm_consume<1>(S, g, blockIdx.x, G, r, [&](int tile, float (&acc)[1][4]) {
                if (!have_r) { vec_wait(S, vseq); r0 = sm->vec[c0] * scale; r1 = sm->vec[c0 + 1] * scale; have_r = true; }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8;
                    if (n < c.vocab) {
                        const float z = acc[0][i] * ((i & 1) ? r1 : r0);
                        if (zrow[i & 1]) zrow[i & 1][n] = z;
                        Msa one; one.m = z; one.s = 1.f; one.i = n;
                        run[i & 1] = msa_merge(run[i & 1], one);
                    }
                }
            });
            // lanes sharing lane%4 hold the same columns: fold them, then the warps, in a fixed order
#pragma unroll
            for (int q = 0; q < 2; ++q) {
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    Msa o;
                    o.m = __shfl_xor_sync(0xffffffffu, run[q].m, off);
                    o.s = __shfl_xor_sync(0xffffffffu, run[q].s, off);
                    o.i = __shfl_xor_sync(0xffffffffu, run[q].i, off);
                    run[q] = msa_merge(run[q], o);
                }
            }
            const int warp = threadIdx.x >> 5;
            float *wp = reinterpret_cast<float *>(sm->scratch);   // [warp][col][4]
            bar_consumers();
            if (lane < 4) {
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    float *o = wp + ((size_t)warp * MAX_COLS + c0 + q) * 4;
                    o[0] = run[q].m; o[1] = run[q].s; o[2] = __int_as_float(run[q].i);
                }
            }
            bar_consumers();
            if (threadIdx.x < MAX_COLS) {
                Msa a; a.m = -INFINITY; a.s = 0.f; a.i = INT_MAX;
                for (int w = 0; w < CONS_WARPS; ++w) {
                    const float *o = wp + ((size_t)w * MAX_COLS + threadIdx.x) * 4;
                    Msa x; x.m = o[0]; x.s = o[1]; x.i = __float_as_int(o[2]);
                    a = msa_merge(a, x);
                }
                float *o = A.head_part + ((size_t)blockIdx.x * MAX_COLS + threadIdx.x) * 4;
                o[0] = a.m; o[1] = a.s; o[2] = __int_as_float(a.i);
            }
        } else if (ROLE == 1) {
            gemm_produce_x(S, g, blockIdx.x, G, r, pol, [&]() { if (ssq) rstd_produce(sm, ssq, ntd, d_model, c.eps, vseq); });
        } else {
            gemm_phase<ROLE, 1>(S, g, r, pol, NoEpi());
        }
        phase_barrier(9);
    };

    int action = control_point<ROLE>(A, S, CTRL_START, 0, pub_no, d, steps_started);
    book_control();
    int step_i = 0;
    while (action == ACT_NEWSTEP) {
        bool restart = false;
        S.tr_on = step_i >= A.trace_step0 && step_i < A.trace_step1;
        ++step_i;
        for (int l = 0; l < L; ++l) {
            const MegaLayer &ly = M.layer[l];
            const unsigned mask = active_mask(d, l);
            // ---- QKV, finished in the epilogue: q rotated, scaled and stored as tensor-core fragments for the
            // attention phase; k rotated, v as it is, both rounded to bf16 and written straight into their cache
            // rows (Algorithm 1: "update KV cache at layer l by processing all tokens in P[l] in parallel").
            // The rows of every q and k head come reordered so that a 16-row tile holds the features
            // [8 t, 8 t + 8) and [hd/2 + 8 t, hd/2 + 8 t + 8): the two partners (i, i + hd/2) of a rotation
            // are then rows r and r + 8 of one tile, which one thread holds for its two columns.
            {
                Gemm g; g.W = ly.wqkv; g.X = reinterpret_cast<const uint4 *>(A.XA); g.N = c.qkv_rows; g.K = d_model; g.pair = 1; g.half = 0; g.ctas = n_qkv; g.part = nullptr; g.phase_id = bar_no + 1; g.columns(mask);
                x_ready();
                const unsigned vseq = bar_no + 1;
                if (ROLE == 2) {
                    constexpr int HALF = HD / 2, KSQ = HD / 16;
                    const int c0 = 2 * (lane & 3), rq = lane >> 2;
                    const int kvd = c.nkv * HD, group = c.group;
                    const float qscale = rsqrtf((float)HD);
                    float r0 = 0.f, r1 = 0.f;
                    bool have_r = false;
                    uint32_t *stash = stash_of(sm);
                    __nv_bfloat16 *pool = reinterpret_cast<__nv_bfloat16 *>(c.kv_pool);
                    gemm_consume<1>(S, g, blockIdx.x, G, r, [&](int tile) {
                        // rotary factors and cache pages of this lane's two columns, fetched while the weights stream
                        const int n0 = tile * 16;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int cc = c0 + q;
                            if (!((mask >> cc) & 1u)) continue;
                            if (n0 < qd + kvd) {
                                const float *cs = c.rope_cs + ((size_t)cc * HALF + ((n0 & (HD - 1)) >> 1) + rq) * 2;
                                cp_async4(stash + (2 * q) * 32, cs);
                                cp_async4(stash + (2 * q + 1) * 32, cs + 1);
                            }
                            if (n0 >= qd) cp_async4(stash + (4 + q) * 32, c.page_table + (size_t)(A.seq0 + (A.nseq == 1 ? 0 : cc / c.slots)) * c.max_pages + (d.pos[cc] >> c.page_shift));
                        }
                    }, [&](int tile, float (&acc)[1][4]) {
                        if (!have_r) { vec_wait(S, vseq); r0 = sm->vec[c0]; r1 = sm->vec[c0 + 1]; have_r = true; }
                        cp_async_wait_all();
                        const int n0 = tile * 16;
                        if (n0 >= c.qkv_rows) return;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int cc = c0 + q;
                            if (!((mask >> cc) & 1u)) continue;
                            const float rs = q ? r1 : r0;
                            const float x0 = acc[0][q] * rs, x1 = acc[0][2 + q] * rs;   // rows rq and rq + 8 of the tile
                            if (n0 < qd + kvd) {
                                const float co = __uint_as_float(stash[(2 * q) * 32]), si = __uint_as_float(stash[(2 * q + 1) * 32]);
                                const int j = ((n0 & (HD - 1)) >> 1) + rq;   // feature j pairs with j + hd/2
                                float y0 = x0 * co - x1 * si, y1 = x1 * co + x0 * si;
                                if (n0 < qd) {
                                    const int h = n0 / HD, kvh = div_group(h, group), qcol = cc * group + (h - kvh * group);
                                    const int row = qcol & 15, m = qcol >> 4;
                                    __nv_bfloat16 *f0 = reinterpret_cast<__nv_bfloat16 *>(A.qfrag + (((size_t)kvh * 2 + m) * KSQ) * 256);
#pragma unroll
                                    for (int hh = 0; hh < 2; ++hh) {
                                        const int dim = j + hh * HALF;
                                        const float y = (hh ? y1 : y0) * qscale;
                                        const int ks = dim >> 4, kk = dim & 15;
                                        const int ln = (row & 7) * 4 + ((kk & 7) >> 1), reg = (row >> 3) + 2 * (kk >> 3);
                                        const __nv_bfloat16 hi = __float2bfloat16_rn(y);
                                        const __nv_bfloat16 lo = __float2bfloat16_rn(y - __bfloat162float(hi));
                                        __nv_bfloat16 *f = f0 + ((size_t)ks * 32 + ln) * 16;
                                        f[reg * 2 + (kk & 1)] = hi;
                                        f[8 + reg * 2 + (kk & 1)] = lo;
                                    }
                                } else {
                                    const int kvh = (n0 - qd) / HD, pos = d.pos[cc], t = pos & (ATT_PAGE - 1);
                                    const size_t blk = ((((size_t)stash[(4 + q) * 32] * c.L + l) * 2 + 0) * c.nkv + kvh) * ((size_t)ATT_PAGE * HD) + (size_t)t * HD;
                                    pool[blk + ((((j >> 3) ^ (pos & 7)) << 3) | (j & 7))] = __float2bfloat16_rn(y0);
                                    pool[blk + (((((j + HALF) >> 3) ^ (pos & 7)) << 3) | (j & 7))] = __float2bfloat16_rn(y1);
                                }
                            } else {
                                const int nv = n0 - qd - kvd, kvh = nv / HD, j = (nv & (HD - 1)) + rq, pos = d.pos[cc], t = pos & (ATT_PAGE - 1);
                                const size_t blk = ((((size_t)stash[(4 + q) * 32] * c.L + l) * 2 + 1) * c.nkv + kvh) * ((size_t)ATT_PAGE * HD) + (size_t)t * HD;
                                pool[blk + ((((j >> 3) ^ (pos & 7)) << 3) | (j & 7))] = __float2bfloat16_rn(x0);
                                pool[blk + (((((j + 8) >> 3) ^ (pos & 7)) << 3) | (j & 7))] = __float2bfloat16_rn(x1);
                            }
                        }
                    });
                } else if (ROLE == 1) gemm_produce_x(S, g, blockIdx.x, G, r, pol, [&]() { rstd_produce(sm, A.ssq_a, ntd, d_model, c.eps, vseq); });
                else gemm_phase<ROLE, 1>(S, g, r, pol, NoEpi());
                phase_barrier(2);
            }
            // ---- attention (work items that hold no row of this pass are fetched before the QKV phase has ended)
            if (ROLE == 1) {
                if (attn_items(A, d, mask) <= G) attn_produce_single(A, S, d, l, mask, bar_no * (unsigned)G, r, pol);
                else attn_produce(A, S, d, l, mask, bar_no * (unsigned)G, r, pol);
            }
            if (ROLE == 2) {
                if (attn_items(A, d, mask) <= G) attn_consume_single<HD>(A, S, d, l, mask, r);
                else attn_consume<HD>(A, S, d, l, mask, r);
            }
            phase_barrier(4);
            // ---- O projection + residual; prepares the FFN input
            {
                Gemm g; g.W = ly.wo; g.X = reinterpret_cast<const uint4 *>(A.XO); g.N = d_model; g.K = qd; g.pair = 1; g.half = 0; g.ctas = n_d; g.part = nullptr; g.phase_id = bar_no + 1; g.columns(mask);
                x_ready();
                if (ROLE == 2) {
                    const __nv_bfloat16 *gain = ly.ffn_norm;
                    uint32_t *stash = stash_of(sm);
                    gemm_consume<1>(S, g, blockIdx.x, G, r, [&](int tile) {   // residual and gain are fetched while the weights stream
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, cc = 2 * (lane & 3) + (i & 1);
                            if ((mask >> cc) & 1u) cp_async4(stash + i * 32, c.resid + (size_t)cc * d_model + n);
                        }
#pragma unroll
                        for (int h = 0; h < 2; ++h) cp_async4(stash + (4 + h) * 32, gain + ((tile * 16 + (lane >> 2) + h * 8) & ~1));
                    }, [&](int tile, float (&acc)[1][4]) {
                        const int c0 = 2 * (lane & 3);
                        float sq[2] = {0.f, 0.f};
                        cp_async_wait_all();
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, cc = c0 + (i & 1);
                            if ((mask >> cc) & 1u) {
                                float *rp = c.resid + (size_t)cc * d_model + n;
                                const float v = __uint_as_float(stash[i * 32]) + acc[0][i];
                                *rp = v;
                                xfrag_store(A.XB, n, cc, v * bf16_of_word(stash[(4 + (i >> 1)) * 32], n));
                                sq[i & 1] += v * v;
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            sq[q] += __shfl_xor_sync(0xffffffffu, sq[q], 4);
                            sq[q] += __shfl_xor_sync(0xffffffffu, sq[q], 8);
                            sq[q] += __shfl_xor_sync(0xffffffffu, sq[q], 16);
                            if (lane < 4 && ((mask >> (c0 + q)) & 1u)) A.ssq_b[(size_t)tile * MAX_COLS + c0 + q] = sq[q];
                        }
                    });
                } else gemm_phase<ROLE, 1>(S, g, r, pol, NoEpi());
                phase_barrier(5);
            }
            // ---- gate / up + SwiGLU
            {
                Gemm g; g.W = ly.wgu; g.W2 = ly.wup; g.X = reinterpret_cast<const uint4 *>(A.XB); g.N = 2 * c.dff; g.K = d_model; g.pair = 2; g.half = c.dff; g.ctas = n_gu;
                // the one GEMM of the layer where the unit-balanced split pays (measured: it shortens gate-up by 1.4 us,
                // but lengthens down, QKV and O, whose tile groups are k-split among the warps)
                g.part = A.part; g.phase_id = bar_no + 1; g.columns(mask);
                x_ready();
                const unsigned vseq = bar_no + 1;
                if (ROLE == 2) {
                    const int c0 = 2 * (lane & 3);
                    float r0 = 0.f, r1 = 0.f;
                    bool have_r = false;
                    gemm_consume<2>(S, g, blockIdx.x, G, r, [&](int tile, float (&acc)[2][4]) {
                        if (!have_r) { vec_wait(S, vseq); r0 = sm->vec[c0]; r1 = sm->vec[c0 + 1]; have_r = true; }
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, cc = c0 + (i & 1);
                            if ((mask >> cc) & 1u) {
                                const float rs = (i & 1) ? r1 : r0;
                                const float gv = acc[0][i] * rs, u = acc[1][i] * rs;
                                xfrag_store(A.XH, n, cc, gv / (1.0f + expf(-gv)) * u);
                            }
                        }
                    });
                } else if (ROLE == 1) gemm_produce_x(S, g, blockIdx.x, G, r, pol, [&]() { rstd_produce(sm, A.ssq_b, ntd, d_model, c.eps, vseq); });
                else gemm_phase<ROLE, 2>(S, g, r, pol, NoEpi());
                phase_barrier(6);
            }
            // ---- down projection + residual; prepares the next layer's (and the head's) input
            {
                Gemm g; g.W = ly.wdown; g.X = reinterpret_cast<const uint4 *>(A.XH); g.N = d_model; g.K = c.dff; g.pair = 1; g.half = 0; g.ctas = n_d; g.part = nullptr; g.phase_id = bar_no + 1; g.columns(mask);
                x_ready();
                if (ROLE == 2) {
                    const __nv_bfloat16 *gain_next = l + 1 < L ? M.layer[l + 1].attn_norm : nullptr;
                    const bool want_f = l + 1 == L || A.exit_at[l + 1] != 0;
                    const __nv_bfloat16 *gain_f = M.final_norm;
                    uint32_t *stash = stash_of(sm);
                    gemm_consume<1>(S, g, blockIdx.x, G, r, [&](int tile) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, cc = 2 * (lane & 3) + (i & 1);
                            if ((mask >> cc) & 1u) cp_async4(stash + i * 32, c.resid + (size_t)cc * d_model + n);
                        }
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int n2 = (tile * 16 + (lane >> 2) + h * 8) & ~1;
                            if (gain_next) cp_async4(stash + (4 + h) * 32, gain_next + n2);
                            if (want_f) cp_async4(stash + (6 + h) * 32, gain_f + n2);
                        }
                    }, [&](int tile, float (&acc)[1][4]) {
                        const int c0 = 2 * (lane & 3);
                        float sq[2] = {0.f, 0.f};
                        cp_async_wait_all();
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, cc = c0 + (i & 1);
                            if ((mask >> cc) & 1u) {
                                float *rp = c.resid + (size_t)cc * d_model + n;
                                const float v = __uint_as_float(stash[i * 32]) + acc[0][i];
                                *rp = v;
                                if (gain_next) xfrag_store(A.XA, n, cc, v * bf16_of_word(stash[(4 + (i >> 1)) * 32], n));
                                if (want_f) xfrag_store(A.XF, n, cc, v * bf16_of_word(stash[(6 + (i >> 1)) * 32], n));
                                sq[i & 1] += v * v;
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            sq[q] += __shfl_xor_sync(0xffffffffu, sq[q], 4);
                            sq[q] += __shfl_xor_sync(0xffffffffu, sq[q], 8);
                            sq[q] += __shfl_xor_sync(0xffffffffu, sq[q], 16);
                            if (lane < 4 && ((mask >> (c0 + q)) & 1u)) A.ssq_a[(size_t)tile * MAX_COLS + c0 + q] = sq[q];
                        }
                    });
                } else gemm_phase<ROLE, 1>(S, g, r, pol, NoEpi());
                phase_barrier(8);
            }
            // ---- intermediate head (Section 2.1) and the early-prediction rule (Eq. 1)
            const unsigned hcols = (unsigned)d.head_mask & mask;   // newest tokens that reached this layer and may exit early
            if (l + 1 < L && A.exit_at[l + 1] != 0 && hcols != 0) {
                const MegaLayer &hl = M.layer[l + 1];
                if (hl.wT) {
                    Gemm g; g.W = hl.wT; g.X = reinterpret_cast<const uint4 *>(A.XF); g.N = d_model; g.K = d_model; g.pair = 1; g.half = 0; g.ctas = n_d; g.part = nullptr; g.phase_id = bar_no + 1; g.columns(hcols);
                    x_ready();
                    const unsigned vseq = bar_no + 1;
                    if (ROLE == 2) {
                        const int c0 = 2 * (lane & 3);
                        float r0 = 0.f, r1 = 0.f;
                        bool have_r = false;
                        gemm_consume<1>(S, g, blockIdx.x, G, r, [&](int tile, float (&acc)[1][4]) {
                            if (!have_r) { vec_wait(S, vseq); r0 = sm->vec[c0]; r1 = sm->vec[c0 + 1]; have_r = true; }
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, cc = c0 + (i & 1);
                                xfrag_store(A.XT, n, cc, acc[0][i] * ((i & 1) ? r1 : r0));
                            }
                        });
                    } else if (ROLE == 1) gemm_produce_x(S, g, blockIdx.x, G, r, pol, [&]() { rstd_produce(sm, A.ssq_a, ntd, d_model, c.eps, vseq); });
                    else gemm_phase<ROLE, 1>(S, g, r, pol, NoEpi());
                    phase_barrier(10);
                    head_phase(A.XT, nullptr, hl.head_scale, hcols, true);
                } else {
                    head_phase(A.XF, A.ssq_a, hl.head_scale, hcols, true);
                }
                action = control_point<ROLE>(A, S, CTRL_HEAD, l + 1, pub_no, d, steps_started);
                book_control();
                if (action != ACT_CONTINUE) { restart = true; break; }
            }
        }
        if (!restart) {
            // ---- final head for every column, then verification (Eq. 2 at temperature zero) in the control point
            if (d.run_final) head_phase(A.XF, A.ssq_a, 1.0f, active_mask(d, L - 1), false);
            action = control_point<ROLE>(A, S, CTRL_TOP, 0, pub_no, d, steps_started);
            book_control();
        }
    }
}

// Repack on load.  Destination row `prow` of the fused q | k | v matrix: v rows are copied as they are; inside
// every q and k head the rows are reordered so that the 16-row tile t of the head holds the features
// [8 t, 8 t + 8) in its rows 0..7 and [hd/2 + 8 t, hd/2 + 8 t + 8) in its rows 8..15.  The two partners
// (i, i + hd/2) of a rotation then sit in rows r and r + 8 of one tensor-core tile, i.e. in one thread of the
// QKV epilogue.  d must be a multiple of 8 and every pointer 16-byte aligned.
__global__ void k_repack_qkv(const __nv_bfloat16 *__restrict__ wq, const __nv_bfloat16 *__restrict__ wk, const __nv_bfloat16 *__restrict__ wv,
                             __nv_bfloat16 *__restrict__ dst, int nq, int nkv, int hd, int d) {
    const int prow = blockIdx.x, qd = nq * hd, kvd = nkv * hd;
    const __nv_bfloat16 *src;
    if (prow < qd + kvd) {
        const __nv_bfloat16 *w = prow < qd ? wq : wk;
        const int rr = prow < qd ? prow : prow - qd;
        const int h = rr / hd, pr = rr - h * hd, t = pr >> 4, r = pr & 15;
        src = w + (size_t)(h * hd + t * 8 + (r & 7) + (r >> 3) * (hd / 2)) * d;
    } else {
        src = wv + (size_t)(prow - qd - kvd) * d;
    }
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
    uint4 *d4 = reinterpret_cast<uint4 *>(dst + (size_t)prow * d);
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x) d4[i] = s4[i];
}

// Arms the prompt passes of the persistent kernel for one sequence (KV cache <- LM(x), first line of Algorithm 1).
__global__ void k_prefill_arm(Ctx c, int seq, int n_prompt) {
    DevState *st = c.st;
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    st->pf_pos = 0;
    st->pf_end = n_prompt;
    st->done[seq] = 0;
    st->n_done = 0;
    st->len[seq] = 0;
    st->base[seq] = 0;
    st->tape_n = 0;
    st->tape_i = 0;
    for (int l = 0; l < c.L; ++l) c.fill[(size_t)seq * c.L + l] = 0;
}

template <int HD>
__global__ void __launch_bounds__(THREADS, 1) k_decode_persistent(const __grid_constant__ MegaArgs A) {
    extern __shared__ unsigned char smem_raw[];
    Smem *sm = smem_base(smem_raw);
    smem_init(sm);
    __syncthreads();
    Shared S{sm, A.err, A.trace, 0, A.wait_ns};
    const int warp = threadIdx.x >> 5;
    if (warp == CONS_WARPS) run<0, HD>(A, S);
    else if (warp == CONS_WARPS + 1) run<1, HD>(A, S);
    else run<2, HD>(A, S);
    settle_on_abort(S);
}

}  // namespace mg
}  // namespace ada
