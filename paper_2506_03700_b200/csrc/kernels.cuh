// CUDA-core kernels of the layer-parallel decode step (any dtype) and the control kernels.
//
// Invariance rule kept by every kernel here: the value computed for a row (a token) depends only
// on that row's own inputs and on the launch geometry, never on which other rows ride along in
// the same pass.  Each row's reductions run in a fixed order.  This is what makes the adaptive
// procedure (rows processed several at a time, Algorithm 1) reproduce plain greedy decoding (one
// row at a time) bit for bit.
#pragma once

#include <limits.h>
#include <math.h>

#include "common.cuh"

namespace ada {

constexpr int SEL_HEAD = -1;   // newest token of every climbing sequence that may consult a head
constexpr int SEL_FINAL = -2;  // every row that reached the last layer in this step
constexpr int SEL_LAST = -3;   // the single row rt->n_rows-1 (prefill: last prompt token)

struct Ctx {
    int d, nq, nkv, hd, dff, vocab, L, qkv_rows, group;
    float eps;
    int page_tokens, page_shift, max_pages, max_seq, slots, n_chunks, kv_swz;
    DevState *st;
    RowTable *rt;
    int32_t *fill;        // [batch][L]
    int32_t *tokens;      // [batch][max_seq]
    int32_t *page_table;  // [batch][max_pages]
    HeadResult *head_res; // [kMaxRows]
    float *resid;         // [R][d]
    float *xn;            // [R][d]  normalised GEMM input
    float *qkv;           // [R][qkv_rows]
    float *q;             // [R][nq*hd]
    float *attn_out;      // [R][nq*hd]
    float *gu;            // [R][2*dff]
    float *hact;          // [R][dff]
    float *rope_cs;       // [R][hd/2][2]
    float *attn_part;     // [R][nq][n_chunks][hd+2]
    float *head_part;     // [head_blocks][R][4]
    float *logit_stage;   // [R][vocab] or nullptr
    float *capture;       // [cap][vocab] or nullptr
    float *head_log;      // [kHeadLogCap][4]
    void *kv_pool;
};

// ------------------------------------------------------------------ small helpers

template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int E = 4;
    static __device__ __forceinline__ void load_stream(const float *p, float (&o)[4]) {
        float4 v = __ldcs(reinterpret_cast<const float4 *>(p));
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
    static __device__ __forceinline__ void load(const float *p, float (&o)[4]) {
        float4 v = *reinterpret_cast<const float4 *>(p);
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int E = 8;
    static __device__ __forceinline__ void unpack(const uint4 &v, float (&o)[8]) {
        o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
        o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
        o[4] = __uint_as_float(v.z << 16); o[5] = __uint_as_float(v.z & 0xffff0000u);
        o[6] = __uint_as_float(v.w << 16); o[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    static __device__ __forceinline__ void load_stream(const __nv_bfloat16 *p, float (&o)[8]) {
        unpack(__ldcs(reinterpret_cast<const uint4 *>(p)), o);
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&o)[8]) {
        unpack(*reinterpret_cast<const uint4 *>(p), o);
    }
};

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// E consecutive fp32 activations (E = 4 or 8) as 16-byte loads.
template <int E> __device__ __forceinline__ void load_x(const float *p, float (&o)[E]) {
#pragma unroll
    for (int q = 0; q < E / 4; ++q) {
        float4 v = *reinterpret_cast<const float4 *>(p + 4 * q);
        o[4 * q] = v.x; o[4 * q + 1] = v.y; o[4 * q + 2] = v.z; o[4 * q + 3] = v.w;
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ bool selected(const Ctx &c, int r, int sel) {
    const RowTable *rt = c.rt;
    if (r >= rt->n_rows) return false;
    int fl = rt->first_layer[r];
    if (sel >= 0) return fl <= sel;
    if (fl == INT_MAX) return false;
    if (sel == SEL_FINAL) return true;
    if (sel == SEL_LAST) return r == rt->n_rows - 1;
    const DevState *st = c.st;
    int s = rt->seq[r];
    int len = st->len[s], base = st->base[s];
    return rt->pos[r] == len - 1 && (len - 1 - base) < st->max_early && len < st->target_len[s];
}

// Compact list of selected rows into shared memory (same order for every block).
__device__ __forceinline__ int build_row_list(const Ctx &c, int sel, int *rows_sh, int *n_sh) {
    if (threadIdx.x == 0) {
        int n = 0, nr = c.rt->n_rows;
        for (int r = 0; r < nr; ++r)
            if (selected(c, r, sel)) rows_sh[n++] = r;
        *n_sh = n;
    }
    __syncthreads();
    return *n_sh;
}

// Element index of the first element of one cached row (K or V of one position, one kv head).
// Pool layout: [page][layer][K|V][kv head][position in page][head_dim].
__device__ __forceinline__ size_t kv_index(const Ctx &c, int seq, int layer, int which, int head, int pos) {
    int page = c.page_table[seq * c.max_pages + (pos >> c.page_shift)];
    int t = pos & (c.page_tokens - 1);
    return ((((size_t)page * c.L + layer) * 2 + which) * c.nkv + head) * ((size_t)c.page_tokens * c.hd) + (size_t)t * c.hd;
}
// Inside a bf16 row the 16-byte chunks (8 elements) are stored xor-swizzled by the position:
// element j sits at chunk (j/8) ^ (pos & swz), swz = 7 when head_dim is a multiple of 64 (else the
// largest of 3, 1, 0 whose block size divides head_dim/8).  A page of rows copied verbatim into
// shared memory can then be read with ldmatrix (8 rows x 16 bytes) without bank conflicts.  fp32
// rows are stored plainly (swz = 0).
__device__ __forceinline__ int kv_swz(const Ctx &c, int j, int pos) {
    return (((j >> 3) ^ (pos & c.kv_swz)) << 3) | (j & 7);
}

// ------------------------------------------------------------------ step set-up

// Embed `tok` into resid[r] and compute the rotary cos/sin of position pos for row r.
template <typename T>
__device__ void embed_row(const Ctx &c, const T *embed, float rope_base, int r, int tok, int pos) {
    for (int i = threadIdx.x; i < c.d; i += blockDim.x) c.resid[(size_t)r * c.d + i] = to_f<T>(embed[(size_t)tok * c.d + i]);
    int half = c.hd / 2;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        double freq = pow((double)rope_base, -2.0 * i / c.hd);
        double sn, cs;
        sincos((double)pos * freq, &sn, &cs);
        c.rope_cs[((size_t)r * half + i) * 2 + 0] = (float)cs;
        c.rope_cs[((size_t)r * half + i) * 2 + 1] = (float)sn;
    }
}

// Start of one iteration of Algorithm 1's while loop for every sequence: the newest token t_i
// (position len-1) gets its embedding; the row table lists, per sequence, the in-flight early
// tokens and t_i with the layer at which each resumes (P[l] (+) t_i for every l at once).
template <typename T>
__global__ void k_step_begin(Ctx c, const T *embed, float rope_base) {
    DevState *st = c.st;
    RowTable *rt = c.rt;
    if (threadIdx.x == 0) {
        int nclimb = 0;
        for (int s = 0; s < st->batch; ++s) {
            int climbing = !st->done[s];
            st->climbing[s] = climbing;
            nclimb += climbing;
            int len = st->len[s], base = st->base[s];
            for (int slot = 0; slot < c.slots; ++slot) {
                int r = s * c.slots + slot, pos = base + slot;
                rt->seq[r] = s;
                rt->pos[r] = pos;
                int fl = INT_MAX;
                if (climbing && pos < len) {
                    fl = 0;
                    for (int l = 0; l < c.L; ++l) fl += c.fill[s * c.L + l] > pos;
                }
                rt->first_layer[r] = fl;
            }
        }
        rt->n_rows = st->batch * c.slots;
        st->n_climbing = nclimb;
    }
    __syncthreads();
    for (int s = 0; s < st->batch; ++s) {
        if (!st->climbing[s]) continue;
        int pos = st->len[s] - 1;
        int r = s * c.slots + (pos - st->base[s]);
        embed_row<T>(c, embed, rope_base, r, c.tokens[(size_t)s * c.max_seq + pos], pos);
    }
}

// Prefill pass: rows 0..n-1 are prompt positions pos0.. of sequence seq, all starting at layer 0.
template <typename T>
__global__ void k_prefill_begin(Ctx c, const T *embed, float rope_base, int seq, int pos0, int n) {
    RowTable *rt = c.rt;
    if (threadIdx.x == 0) {
        for (int r = 0; r < n; ++r) { rt->seq[r] = seq; rt->pos[r] = pos0 + r; rt->first_layer[r] = 0; }
        rt->n_rows = n;
    }
    __syncthreads();
    for (int r = 0; r < n; ++r) embed_row<T>(c, embed, rope_base, r, c.tokens[(size_t)seq * c.max_seq + pos0 + r], pos0 + r);
}

// End of a prefill pass: positions < pos_end are complete at every layer.  After the last pass
// the full-depth argmax at the last prompt token becomes the first generated (pending) token.
__global__ void k_prefill_end(Ctx c, int seq, int pos_end, int last, int n_prompt) {
    DevState *st = c.st;
    if (threadIdx.x != 0) return;
    for (int l = 0; l < c.L; ++l) c.fill[seq * c.L + l] = pos_end;
    st->base[seq] = pos_end;
    st->len[seq] = pos_end;
    if (last) {
        int r = c.rt->n_rows - 1;
        c.tokens[(size_t)seq * c.max_seq + n_prompt] = c.head_res[r].token;
        st->len[seq] = n_prompt + 1;
        st->n_prompt[seq] = n_prompt;
        st->done[seq] = 1;
        if (seq == 0 && c.capture) {
            st->keep_rows = 1;
        }
    }
}

// ------------------------------------------------------------------ RMSNorm

// out[r] = resid[r] / sqrt(mean(resid[r]^2) + eps) * g, one block per row.
template <typename T>
__global__ void __launch_bounds__(256) k_rmsnorm(Ctx c, const T *gain, int sel, float *out, int ldo) {
    int r = blockIdx.x;
    if (!selected(c, r, sel)) return;
    const float *x = c.resid + (size_t)r * c.d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < c.d; i += blockDim.x) ss = fmaf(x[i], x[i], ss);
    __shared__ float red[8];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    float rstd = 1.0f / sqrtf(tot / c.d + c.eps);
    for (int i = threadIdx.x; i < c.d; i += blockDim.x) out[(size_t)r * ldo + i] = x[i] * rstd * to_f<T>(gain[i]);
}

// ------------------------------------------------------------------ skinny GEMM on CUDA cores

// Y[r][n] = sum_k W[n][k] * X[r][k] for every selected row r.  One warp per output feature n;
// lanes stride over K in 16-byte chunks; per row the sum order is fixed (chunk order per lane,
// then a shuffle tree), so a row's result does not depend on the other rows.
// EPI 0: store to Y.  EPI 1: Y[r][n] += result (residual add; each (r, n) has one writer).
template <typename T, int EPI>
__global__ void __launch_bounds__(256) k_gemv(Ctx c, const T *__restrict__ W, int N, int K, const float *__restrict__ X,
                                              int ldx, float *__restrict__ Y, int ldy, int sel) {
    __shared__ int rows[kMaxRows];
    __shared__ int nr_sh;
    const int nr = build_row_list(c, sel, rows, &nr_sh);
    if (nr == 0) return;
    constexpr int E = Vec16<T>::E;
    const int nch = K / E;
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int n = warp; n < N; n += nwarps) {
        const T *wrow = W + (size_t)n * K;
        for (int g0 = 0; g0 < nr; g0 += 8) {
            const int cnt = min(8, nr - g0);
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.f;
            for (int c0 = lane; c0 < nch; c0 += 128) {
                float w[4][E];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    int cc = c0 + 32 * u;
                    if (cc < nch) {
                        if (g0 == 0) Vec16<T>::load_stream(wrow + (size_t)cc * E, w[u]);
                        else Vec16<T>::load(wrow + (size_t)cc * E, w[u]);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    int cc = c0 + 32 * u;
                    if (cc < nch) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            if (j < cnt) {
                                float x[E];
                                load_x<E>(X + (size_t)rows[g0 + j] * ldx + (size_t)cc * E, x);
#pragma unroll
                                for (int e = 0; e < E; ++e) acc[j] = fmaf(w[u][e], x[e], acc[j]);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j < cnt) {
                    float v = warp_sum(acc[j]);
                    if (lane == 0) {
                        float *y = Y + (size_t)rows[g0 + j] * ldy + n;
                        if (EPI == 0) *y = v; else *y += v;
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------ RoPE + KV write

// q <- RoPE(q) into the q buffer; k <- RoPE(k) and v into the layer's cache pages at the row's
// position (Algorithm 1: "update KV cache at layer l").  One block per row.
template <typename T>
__global__ void k_rope_kv(Ctx c, int layer) {
    int r = blockIdx.x;
    if (!selected(c, r, layer)) return;
    const int half = c.hd / 2, seq = c.rt->seq[r], pos = c.rt->pos[r];
    const float *in = c.qkv + (size_t)r * c.qkv_rows;
    const float *cs = c.rope_cs + (size_t)r * half * 2;
    T *pool = reinterpret_cast<T *>(c.kv_pool);
    const int nqh = c.nq * half;
    for (int i = threadIdx.x; i < nqh; i += blockDim.x) {
        int h = i / half, j = i - h * half;
        float x0 = in[h * c.hd + j], x1 = in[h * c.hd + j + half];
        float co = cs[2 * j], si = cs[2 * j + 1];
        c.q[(size_t)r * c.nq * c.hd + h * c.hd + j] = x0 * co - x1 * si;
        c.q[(size_t)r * c.nq * c.hd + h * c.hd + j + half] = x1 * co + x0 * si;
    }
    const float *kin = in + c.nq * c.hd, *vin = kin + c.nkv * c.hd;
    const int nkh = c.nkv * half;
    for (int i = threadIdx.x; i < nkh; i += blockDim.x) {
        int h = i / half, j = i - h * half;
        float x0 = kin[h * c.hd + j], x1 = kin[h * c.hd + j + half];
        float co = cs[2 * j], si = cs[2 * j + 1];
        size_t o = kv_index(c, seq, layer, 0, h, pos);
        pool[o + kv_swz(c, j, pos)] = from_f<T>(x0 * co - x1 * si);
        pool[o + kv_swz(c, j + half, pos)] = from_f<T>(x1 * co + x0 * si);
    }
    for (int i = threadIdx.x; i < c.nkv * c.hd; i += blockDim.x) {
        int h = i / c.hd, j = i - h * c.hd;
        pool[kv_index(c, seq, layer, 1, h, pos) + kv_swz(c, j, pos)] = from_f<T>(vin[i]);
    }
}

// ------------------------------------------------------------------ attention (CUDA cores)

// Partial attention of one (row, q head, chunk): online softmax over cache positions
// [256*chunk, min(pos, 256*chunk+255)] in ascending order.  Chunks are anchored at position 0 and
// do not depend on the context length or on other rows.  One warp per block; lane holds hd/32 dims.
template <typename T, int EPL>
__global__ void __launch_bounds__(32) k_attn_partial(Ctx c, int layer) {
    const int r = blockIdx.z;
    if (!selected(c, r, layer)) return;
    const int pos = c.rt->pos[r], seq = c.rt->seq[r];
    const int chunk = blockIdx.x, t0 = chunk * kAttnChunk;
    if (t0 > pos) return;
    const int t1 = min(pos, t0 + kAttnChunk - 1);
    const int h = blockIdx.y, kvh = h / c.group, lane = threadIdx.x;
    const T *pool = reinterpret_cast<const T *>(c.kv_pool);
    float qv[EPL], acc[EPL];
    const float scale = rsqrtf((float)c.hd);
#pragma unroll
    for (int e = 0; e < EPL; ++e) { qv[e] = c.q[((size_t)r * c.nq + h) * c.hd + lane * EPL + e]; acc[e] = 0.f; }
    float m = -INFINITY, l = 0.f;
    for (int t = t0; t <= t1; ++t) {
        const T *kp = pool + kv_index(c, seq, layer, 0, kvh, t);
        const T *vp = pool + kv_index(c, seq, layer, 1, kvh, t);
        float dot = 0.f, vv[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const int j = kv_swz(c, lane * EPL + e, t);
            dot = fmaf(qv[e], to_f<T>(kp[j]), dot);
            vv[e] = to_f<T>(vp[j]);
        }
        float sc = warp_sum(dot) * scale;
        float mn = fmaxf(m, sc);
        float corr = expf(m - mn), p = expf(sc - mn);
        l = l * corr + p;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * corr + p * vv[e];
        m = mn;
    }
    float *out = c.attn_part + (((size_t)r * c.nq + h) * c.n_chunks + chunk) * (c.hd + 2);
#pragma unroll
    for (int e = 0; e < EPL; ++e) out[lane * EPL + e] = acc[e];
    if (lane == 0) { out[c.hd] = m; out[c.hd + 1] = l; }
}

// Merge the chunk partials of one (row, head) in ascending chunk order; write attn_out.
__global__ void k_attn_combine(Ctx c, int layer) {
    const int r = blockIdx.y, h = blockIdx.x;
    if (!selected(c, r, layer)) return;
    const int nch = c.rt->pos[r] / kAttnChunk + 1;
    const float *part = c.attn_part + (((size_t)r * c.nq + h) * c.n_chunks) * (c.hd + 2);
    float M = -INFINITY;
    for (int k = 0; k < nch; ++k) M = fmaxf(M, part[(size_t)k * (c.hd + 2) + c.hd]);
    float den = 0.f;
    for (int k = 0; k < nch; ++k) den += part[(size_t)k * (c.hd + 2) + c.hd + 1] * expf(part[(size_t)k * (c.hd + 2) + c.hd] - M);
    float *out = c.attn_out + (size_t)r * c.nq * c.hd + h * c.hd;
    for (int i = threadIdx.x; i < c.hd; i += blockDim.x) {
        float a = 0.f;
        for (int k = 0; k < nch; ++k) a += part[(size_t)k * (c.hd + 2) + i] * expf(part[(size_t)k * (c.hd + 2) + c.hd] - M);
        out[i] = a / den;
    }
}

// Causal attention of a block of prompt rows (a dense prompt pass), bf16 cache.  One block = one kv head x
// PF_Q consecutive rows (one warp per row, serving all `group` q heads of the kv head); the K and V rows of 32
// cache positions at a time are staged in shared memory once for the whole block, so a cached row is fetched
// from L2 once per PF_Q x group (query, head) pairs instead of once per pair.  Online softmax in position
// order per (row, head); the context is not split, so the result goes straight to attn_out.
// EPL = head_dim / 32 elements per lane, GROUP = q heads per kv head (1, 2 or 4).
constexpr int PF_Q = 4, PF_T = 32;
template <int EPL, int GROUP>
__global__ void __launch_bounds__(PF_Q * 32) k_pf_attn(Ctx c, int layer, int rows) {
    constexpr int HD = EPL * 32;
    __shared__ __align__(16) __nv_bfloat16 sK[PF_T][HD], sV[PF_T][HD];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, kvh = blockIdx.y;
    const int r = blockIdx.x * PF_Q + warp;
    const bool live = r < rows;
    const int seq = c.rt->seq[min(r, rows - 1)], pos = live ? c.rt->pos[r] : -1;
    const int r_last = min(blockIdx.x * PF_Q + PF_Q, rows) - 1, pos_max = c.rt->pos[r_last];   // rows of a block are consecutive positions
    const __nv_bfloat16 *pool = reinterpret_cast<const __nv_bfloat16 *>(c.kv_pool);
    const float scale = rsqrtf((float)HD);
    float q[GROUP][EPL], acc[GROUP][EPL], m[GROUP], l[GROUP];
#pragma unroll
    for (int g = 0; g < GROUP; ++g) {
        m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            q[g][e] = live ? c.q[((size_t)r * c.nq + kvh * GROUP + g) * HD + lane * EPL + e] * scale : 0.f;
            acc[g][e] = 0.f;
        }
    }
    for (int t0 = 0; t0 <= pos_max; t0 += PF_T) {
        __syncthreads();   // the previous tile has been used
        for (int i = threadIdx.x; i < PF_T * (HD / 8); i += PF_Q * 32) {
            const int t = i / (HD / 8), ch = i - t * (HD / 8), p = t0 + t;
            uint4 kq = make_uint4(0, 0, 0, 0), vq = kq;
            if (p <= pos_max) {
                const int sc = ch ^ (p & c.kv_swz);   // stored chunk of logical chunk ch
                kq = *reinterpret_cast<const uint4 *>(pool + kv_index(c, seq, layer, 0, kvh, p) + sc * 8);
                vq = *reinterpret_cast<const uint4 *>(pool + kv_index(c, seq, layer, 1, kvh, p) + sc * 8);
            }
            *reinterpret_cast<uint4 *>(&sK[t][ch * 8]) = kq;
            *reinterpret_cast<uint4 *>(&sV[t][ch * 8]) = vq;
        }
        __syncthreads();
        const int tn = min(PF_T, pos - t0 + 1);   // keys of this tile the row may see (causal)
        for (int t = 0; t < tn; ++t) {
            float kf[EPL], vf[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) { kf[e] = __bfloat162float(sK[t][lane * EPL + e]); vf[e] = __bfloat162float(sV[t][lane * EPL + e]); }
#pragma unroll
            for (int g = 0; g < GROUP; ++g) {
                float dot = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) dot = fmaf(q[g][e], kf[e], dot);
                const float sc = warp_sum(dot);
                const float mn = fmaxf(m[g], sc);
                const float corr = expf(m[g] - mn), pr = expf(sc - mn);
                l[g] = l[g] * corr + pr;
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[g][e] = acc[g][e] * corr + pr * vf[e];
                m[g] = mn;
            }
        }
    }
    if (live) {
#pragma unroll
        for (int g = 0; g < GROUP; ++g)
#pragma unroll
            for (int e = 0; e < EPL; ++e) c.attn_out[((size_t)r * c.nq + kvh * GROUP + g) * HD + lane * EPL + e] = acc[g][e] / l[g];
    }
}

// ------------------------------------------------------------------ SwiGLU

__global__ void k_swiglu(Ctx c, int layer) {
    const int r = blockIdx.y;
    if (!selected(c, r, layer)) return;
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= c.dff) return;
    float g = c.gu[(size_t)r * 2 * c.dff + i], u = c.gu[(size_t)r * 2 * c.dff + c.dff + i];
    float s = g / (1.0f + expf(-g));
    c.hact[(size_t)r * c.dff + i] = s * u;
}

// ------------------------------------------------------------------ LM head with fused reduction

// (max, sum exp, argmax) merge; ties keep the lower index.
struct Msa { float m, s; int i; };
__device__ __forceinline__ Msa msa_merge(Msa a, Msa b) {
    Msa o;
    if (b.m > a.m || (b.m == a.m && b.i < a.i)) { Msa t = a; a = b; b = t; }
    o.m = a.m; o.i = a.i;
    o.s = a.s + (b.m == -INFINITY ? 0.f : b.s * expf(b.m - a.m));
    return o;
}

// Logits z[r][v] = scale * E[v] . x[r] for the selected rows, reduced on the fly to per-block
// (max, sum exp(z - max), argmax); logits go to memory only when logit_stage is set (tests).
template <typename T>
__global__ void __launch_bounds__(256) k_head_partial(Ctx c, const T *__restrict__ E, const float *__restrict__ X, int ldx,
                                                      float scale, int sel, int store_logits) {
    __shared__ int rows[kMaxRows];
    __shared__ int nr_sh;
    __shared__ Msa red[8][8];
    const int nr = build_row_list(c, sel, rows, &nr_sh);
    if (nr == 0) return;
    constexpr int EV = Vec16<T>::E;
    const int K = c.d, nch = K / EV, N = c.vocab;
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    for (int g0 = 0; g0 < nr; g0 += 8) {
        const int cnt = min(8, nr - g0);
        Msa run[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { run[j].m = -INFINITY; run[j].s = 0.f; run[j].i = INT_MAX; }
        for (int n = warp; n < N; n += nwarps) {
            const T *wrow = E + (size_t)n * K;
            float acc[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = 0.f;
            for (int c0 = lane; c0 < nch; c0 += 128) {
                float w[4][EV];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    int cc = c0 + 32 * u;
                    if (cc < nch) Vec16<T>::load_stream(wrow + (size_t)cc * EV, w[u]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    int cc = c0 + 32 * u;
                    if (cc < nch) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            if (j < cnt) {
                                float x[EV];
                                load_x<EV>(X + (size_t)rows[g0 + j] * ldx + (size_t)cc * EV, x);
#pragma unroll
                                for (int e = 0; e < EV; ++e) acc[j] = fmaf(w[u][e], x[e], acc[j]);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j < cnt) {
                    float z = warp_sum(acc[j]) * scale;
                    if (store_logits && lane == 0) c.logit_stage[(size_t)rows[g0 + j] * N + n] = z;
                    Msa one; one.m = z; one.s = 1.f; one.i = n;
                    run[j] = msa_merge(run[j], one);
                }
            }
        }
        // block combine in warp order
#pragma unroll
        for (int j = 0; j < 8; ++j) if (lane == 0) red[wib][j] = run[j];
        __syncthreads();
        if (threadIdx.x < cnt) {
            Msa a = red[0][threadIdx.x];
            for (int w = 1; w < 8; ++w) a = msa_merge(a, red[w][threadIdx.x]);
            float *o = c.head_part + ((size_t)blockIdx.x * kMaxRows + rows[g0 + threadIdx.x]) * 4;
            o[0] = a.m; o[1] = a.s; o[2] = __int_as_float(a.i);
        }
        __syncthreads();
    }
}

// Merge the per-block partials of a row in block order -> token, p = 1 / sum exp(z - zmax).
__global__ void k_head_final(Ctx c, int n_blocks, int sel) {
    const int r = blockIdx.x;
    if (threadIdx.x != 0 || !selected(c, r, sel)) return;
    Msa a; a.m = -INFINITY; a.s = 0.f; a.i = INT_MAX;
    for (int b = 0; b < n_blocks; ++b) {
        const float *o = c.head_part + ((size_t)b * kMaxRows + r) * 4;
        Msa x; x.m = o[0]; x.s = o[1]; x.i = __float_as_int(o[2]);
        a = msa_merge(a, x);
    }
    HeadResult hr; hr.token = a.i; hr.zmax = a.m; hr.sumexp = a.s; hr.p = 1.0f / a.s;
    c.head_res[r] = hr;
}

// ------------------------------------------------------------------ control

__device__ __forceinline__ void mark_idle(const Ctx &c, int s) {
    for (int slot = 0; slot < c.slots; ++slot) c.rt->first_layer[s * c.slots + slot] = INT_MAX;
}

// After the head at 1-based layer e: Eq. 1.  If p > gamma the predicted token is appended to the
// sequence (tentatively), the newest token stays in flight at depth e, and the sequence stops
// climbing for this step.
__global__ void k_exit_control(Ctx c, int e) {
    DevState *st = c.st;
    if (threadIdx.x == 0) {
        int nclimb = 0;
        for (int s = 0; s < st->batch; ++s) {
            if (!st->climbing[s]) continue;
            int len = st->len[s], base = st->base[s], slot = len - 1 - base;
            bool eligible = slot < st->max_early && len < st->target_len[s];
            if (eligible) {
                HeadResult hr = c.head_res[s * c.slots + slot];
                bool decide = hr.p > st->gamma;
                if (s == 0 && st->tape_i < st->tape_n) {
                    uint8_t t = st->tape[st->tape_i++];
                    if (t == 0) decide = false;
                    if (t == 1) decide = true;
                }
                st->st.head_evals++;
                if (c.head_log && st->head_log_n < kHeadLogCap) {
                    float *hl = c.head_log + 4 * (size_t)st->head_log_n;
                    hl[0] = (float)st->st.steps; hl[1] = (float)e; hl[2] = (float)hr.token; hl[3] = hr.p;
                    st->head_log_n++;
                }
                if (decide) {
                    for (int l = 0; l < e; ++l) {
                        st->st.row_layers += len - c.fill[s * c.L + l];
                        c.fill[s * c.L + l] = len;
                    }
                    c.tokens[(size_t)s * c.max_seq + len] = hr.token;
                    st->len[s] = len + 1;
                    st->st.early_exits++;
                    st->st.exits_at_layer[e]++;
                    st->st.steps++;
                    st->climbing[s] = 0;
                    mark_idle(c, s);
                }
            }
            nclimb += st->climbing[s];
        }
        st->n_climbing = nclimb;
    }
}

// At the last layer: verification (Eq. 2 at temperature zero).  Row j of a sequence holds the
// token at position base+j; its full-depth argmax a_j must equal the tentative token at
// base+j+1.  First mismatch: the token is replaced by a_j, the sequence is cut after it and every
// layer's fill level drops to its position.  No mismatch: a_last is appended.
__global__ void k_verify(Ctx c) {
    DevState *st = c.st;
    if (threadIdx.x != 0) return;
    int ndone = 0;
    for (int s = 0; s < st->batch; ++s) {
        if (st->climbing[s]) {
            int len = st->len[s], base = st->base[s], nrow = len - base;
            int32_t *tok = c.tokens + (size_t)s * c.max_seq;
            for (int l = 0; l < c.L; ++l) st->st.row_layers += len - c.fill[s * c.L + l];
            int bad = -1;
            for (int j = 0; j + 1 < nrow; ++j)
                if (c.head_res[s * c.slots + j].token != tok[base + j + 1]) { bad = j; break; }
            int new_base, keep;
            if (bad < 0) {
                st->st.accepted += nrow - 1;
                tok[len] = c.head_res[s * c.slots + nrow - 1].token;
                new_base = len;
                keep = nrow;
            } else {
                st->st.accepted += bad;
                st->st.rejected += 1;
                st->st.discarded += nrow - 2 - bad;
                new_base = base + bad + 1;
                tok[new_base] = c.head_res[s * c.slots + bad].token;
                keep = bad + 1;
            }
            // "while t_i != [EOS]" (Algorithm 1): the first verified end-of-sequence token ends the sequence
            int target = st->target_len[s];
            if (st->eos_id >= 0) {
                for (int j = 0; j < keep; ++j)
                    if (c.head_res[s * c.slots + j].token == st->eos_id) {
                        if (base + j + 2 <= target) { target = base + j + 2; st->eos_hit[s] = 1; }
                        break;
                    }
            }
            int new_len = new_base + 1;
            if (new_len > target) {
                st->st.truncated += new_len - target;
                new_len = target;
                new_base = new_len - 1;
            }
            keep = new_len - 1 - base;   // verified tokens that stay
            for (int l = 0; l < c.L; ++l) c.fill[s * c.L + l] = new_base;
            st->len[s] = new_len;
            st->base[s] = new_base;
            st->st.verify_steps++;
            st->st.steps++;
            st->climbing[s] = 0;
            if (new_len >= target) st->done[s] = 1;
            if (s == 0) st->keep_rows = keep;
        } else if (s == 0) {
            st->keep_rows = 0;
        }
        ndone += st->done[s];
    }
    st->n_climbing = 0;
    st->n_done = ndone;
}

// Copy the kept rows' staged final logits of sequence 0 into the capture buffer.
__global__ void k_capture(Ctx c, int row0) {
    DevState *st = c.st;
    const int keep = st->keep_rows, at = st->capture_n;
    for (int j = 0; j < keep; ++j) {
        if (at + j >= st->capture_cap) break;
        const float *src = c.logit_stage + (size_t)(row0 + j) * c.vocab;
        float *dst = c.capture + (size_t)(at + j) * c.vocab;
        for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < c.vocab; i += gridDim.x * blockDim.x) dst[i] = src[i];
    }
}
__global__ void k_capture_advance(Ctx c) {
    if (threadIdx.x == 0 && blockIdx.x == 0) c.st->capture_n += c.st->keep_rows;
}

// Start of a decode call: set targets and parameters.
struct CallTargets { int32_t target_len[ADA_MAX_BATCH]; };
__global__ void k_call_begin(Ctx c, CallTargets tg, float gamma, int max_early, int tape_n, int eos_id) {
    DevState *st = c.st;
    if (threadIdx.x != 0) return;
    int ndone = 0;
    st->eos_id = eos_id;
    for (int s = 0; s < st->batch; ++s) {
        st->target_len[s] = tg.target_len[s];
        st->eos_hit[s] = 0;
        // the pending token (verified, not yet returned) may itself be the end-of-sequence token
        if (eos_id >= 0 && st->len[s] >= 1 && st->len[s] <= tg.target_len[s] &&
            c.tokens[(size_t)s * c.max_seq + st->len[s] - 1] == eos_id) {
            st->target_len[s] = st->len[s];
            st->eos_hit[s] = 1;
        }
        st->done[s] = st->len[s] >= st->target_len[s];
        st->climbing[s] = 0;
        ndone += st->done[s];
    }
    st->gamma = gamma;
    st->max_early = max_early;
    st->tape_n = tape_n;
    st->tape_i = 0;
    st->head_log_n = 0;
    st->n_done = ndone;
    st->n_climbing = 0;
}

}  // namespace ada
