// Host side of the decode library: C ABI, model/session bookkeeping, paged KV allocator, and the
// loops that issue the kernels of Algorithm 1.  All decoding state lives on the device; the host
// only decides how far to launch and reads back a few counters.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <memory>
#include <string>
#include <vector>

#include "kernels.cuh"
#include "gemm_probe.cuh"
#include "mega.cuh"
#include "dense.cuh"

using namespace ada;

namespace {

thread_local std::string g_cuda_err;

#define CK(expr)                                                                                    \
    do {                                                                                            \
        cudaError_t e__ = (expr);                                                                   \
        if (e__ != cudaSuccess) {                                                                   \
            g_cuda_err = std::string(#expr) + ": " + cudaGetErrorString(e__);                       \
            return ADA_ECUDA;                                                                       \
        }                                                                                           \
    } while (0)

struct LayerW {
    // q, k, v and gate, up are held as separate matrices: lent fused (wqkv, w_gate_up) they point into
    // the one tensor.  wqkv_perm is the library's own copy of q | k | v in the caller's arena, with the
    // rows of every q and k head reordered for the persistent kernel's QKV epilogue.
    const void *attn_norm = nullptr, *wq = nullptr, *wk = nullptr, *wv = nullptr, *wo = nullptr, *ffn_norm = nullptr,
               *w_gate = nullptr, *w_up = nullptr, *w_down = nullptr, *wqkv_perm = nullptr;
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Tensor map of a row-major bf16 weight matrix [N][K] for the streaming GEMM: dimensions (64
// elements, N rows, K/64 groups), box (64, 16, 8), 128-byte swizzle, zero fill outside.  The
// driver entry point is looked up at run time, so the library loads without libcuda.
int make_weight_map(CUtensorMap *out, const void *W, int N, int K) {
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qr);
        if (e != cudaSuccess || qr != cudaDriverEntryPointSuccess || !fn) {
            g_cuda_err = std::string("cuTensorMapEncodeTiled is not available: ") + cudaGetErrorString(e);
            return ADA_ECUDA;
        }
        encode = (EncodeFn)fn;
    }
    if (K % 64 || N < 1 || (uintptr_t)W % 16) return ADA_EUNSUPPORTED;
    const cuuint64_t dims[3] = {64, (cuuint64_t)N, (cuuint64_t)(K / 64)};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)st::TILE_N, (cuuint32_t)st::KG};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(W), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_cuda_err = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
        return ADA_ECUDA;
    }
    return ADA_OK;
}

// Tensor map of a row-major bf16 matrix [rows][K] for the dense GEMM of the prompt pass: dimensions (K, rows),
// box (64, box_rows), 128-byte swizzle, zero fill outside.
int make_map_2d(CUtensorMap *out, const void *base, int rows, int K, int box_rows) {
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qr);
        if (e != cudaSuccess || qr != cudaDriverEntryPointSuccess || !fn) {
            g_cuda_err = std::string("cuTensorMapEncodeTiled is not available: ") + cudaGetErrorString(e);
            return ADA_ECUDA;
        }
        encode = (EncodeFn)fn;
    }
    if (K % 64 || rows < 1 || (uintptr_t)base % 16) return ADA_EUNSUPPORTED;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_cuda_err = "cuTensorMapEncodeTiled (2-D) failed with CUresult " + std::to_string((int)r);
        return ADA_ECUDA;
    }
    return ADA_OK;
}

}  // namespace

struct ada_model {
    ada_config cfg;
    size_t esz;
    const void *tok_embed = nullptr, *lm_head = nullptr, *final_norm = nullptr;
    std::vector<LayerW> layers;
    std::vector<int> has_head;
    std::vector<const void *> head_T;
    std::vector<float> head_scale;
    void *arena = nullptr;
    size_t arena_bytes = 0;
    bool finalized = false;
};

struct ada_session {
    const ada_model *m;
    int batch, max_seq, page_tokens, max_early, slots, rows_alloc, n_pages, max_pages, n_chunks, head_blocks;
    cudaStream_t stream;
    Ctx c;
    void *scratch;
    size_t scratch_bytes;
    float *t_out; // [R][d] output of the head transformation
    std::vector<int> free_pages;
    std::vector<std::vector<int>> seq_pages;
    std::vector<int> h_len, h_prompt, h_reported;
    std::vector<char> prefilled, finished;   // finished: the sequence ended on an end-of-sequence token (eos_tok)
    std::vector<int> eos_tok;
    int32_t *pinned = nullptr; // small read-back area
    cudaEvent_t ev0 = nullptr, ev1 = nullptr;
    int path = 0;
    // persistent-kernel path (bf16, one sequence, up to eight token columns)
    bool mega = false;
    int grid = 0;
    mg::MegaArgs margs;
    CUtensorMap *maps_dev = nullptr;      // [6 L + 2]: wqkv, wo, wgu, wup, wdown per layer, lm_head, then T per 1-based layer
    mg::MegaModel *mm_dev = nullptr;
    int *exit_at_dev = nullptr;
    bool sampling = false;   // the call in progress draws its tokens (ada_sampling_decode)
    float inv_temp = 1.0f;
    int steps_per_launch = 256;
    unsigned long long wait_ns = st::WAIT_NS_DEFAULT;
    // dense prompt pass (tcgen05 GEMMs over blocks of up to 128 positions)
    bool dense_ok = false, dense_on = false;   // available for this session / in use by the prefill that is running
    int cur_rows = 0;                          // rows of the pass being issued
    __nv_bfloat16 *pf_hi = nullptr, *pf_lo = nullptr;   // [128][max K]: high and low parts of a GEMM's input
    int *pf_err = nullptr;
    float *pf_part = nullptr;                  // shares of depth-split products: [splits][128][N]
    size_t pf_part_bytes = 0;
    bool prefill_dense = true;                 // ada_debug_set_prefill
    int64_t launches = 0, syncs = 0, layer_passes = 0;
    // per-class profiling
    bool prof = false;
    std::vector<cudaEvent_t> prof_ev;
    std::vector<std::pair<int, double>> prof_rec;  // (class, bytes) per recorded launch
    double prof_ms[ADA_PROF_CLASSES] = {0}, prof_bytes[ADA_PROF_CLASSES] = {0};
    int64_t prof_launches[ADA_PROF_CLASSES] = {0};
    // debug
    float *capture_dev = nullptr;
    int capture_cap = 0;
    float *head_log_host = nullptr;
    int head_log_cap = 0;
    int32_t *head_log_n_out = nullptr;
    std::vector<uint8_t> tape;
    std::vector<CUtensorMap> maps_host;
    std::unique_ptr<mg::MegaModel> mm_host;
};

namespace {

// Scratch layout (all offsets 256-byte aligned).
struct Layout {
    size_t st, rt, fill, tokens, page_table, head_res, resid, xn, qkv, q, attn_out, gu, hact, rope_cs, attn_part,
        head_part, logit_stage, head_log, t_out, pf_hi, pf_lo, pf_err, pf_part, maps, mm, exit_at, xa, xb, xo, xh, xf, xt, ssq_a, ssq_b, qfrag, attn_cnt, rope_freq, part,
        grid_ctr, pub, err, q_stage, qinfo, uniforms, total;
};

bool model_fits_persistent(const ada_config &g);
constexpr size_t kDenseSplitMax = 4;   // shares of a depth-split dense product (O and down projections)
// rows a layer pass may carry: the decode rows of all sequences, or a 128-position block of a dense prompt pass
int rows_alloc_for(const ada_config &g, int batch, int max_early) {
    return std::max(batch * (max_early + 1), model_fits_persistent(g) ? dg::BM : 32);
}

// exchange area of weight tiles split between two CTAs: 8 k-splits x 256 tagged words per CTA
constexpr size_t kPartBytesPerCta = (size_t)st::CONS_WARPS * 256 * sizeof(unsigned long long);
constexpr int kPartMaxGrid = 256;

Layout make_layout(const ada_config &g, int batch, int max_seq, int max_early, int head_blocks) {
    Layout L{};
    const int R = rows_alloc_for(g, batch, max_early);
    const int qd = g.n_q_heads * g.head_dim, qkv_rows = (g.n_q_heads + 2 * g.n_kv_heads) * g.head_dim;
    const int n_chunks = (max_seq + kAttnChunk - 1) / kAttnChunk;
    const int max_pages = (max_seq + 15) / 16;  // upper bound for any page size >= 16
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    L.st = take(sizeof(DevState));
    L.rt = take(sizeof(RowTable));
    L.fill = take(sizeof(int32_t) * batch * g.n_layers);
    L.tokens = take(sizeof(int32_t) * (size_t)batch * max_seq);
    L.page_table = take(sizeof(int32_t) * (size_t)batch * max_pages);
    L.head_res = take(sizeof(HeadResult) * kMaxRows);
    L.resid = take(sizeof(float) * (size_t)R * g.d_model);
    L.xn = take(sizeof(float) * (size_t)R * g.d_model);
    L.qkv = take(sizeof(float) * (size_t)R * qkv_rows);
    L.q = take(sizeof(float) * (size_t)R * qd);
    L.attn_out = take(sizeof(float) * (size_t)R * qd);
    L.gu = take(sizeof(float) * (size_t)R * 2 * g.d_ff);
    L.hact = take(sizeof(float) * (size_t)R * g.d_ff);
    L.rope_cs = take(sizeof(float) * (size_t)R * g.head_dim);
    L.attn_part = take(sizeof(float) * (size_t)R * g.n_q_heads * n_chunks * (g.head_dim + 2));
    L.head_part = take(sizeof(float) * (size_t)head_blocks * kMaxRows * 4);
    L.logit_stage = take(sizeof(float) * (size_t)R * g.vocab);
    L.head_log = take(sizeof(float) * 4 * kHeadLogCap);
    L.t_out = take(sizeof(float) * (size_t)R * g.d_model);
    if (model_fits_persistent(g)) {   // dense prompt pass: a GEMM's input as two bf16 matrices [128][K]
        const size_t kmax = (size_t)std::max(std::max(g.d_model, g.n_q_heads * g.head_dim), g.d_ff);
        L.pf_hi = take(sizeof(__nv_bfloat16) * dg::BM * kmax);
        L.pf_lo = take(sizeof(__nv_bfloat16) * dg::BM * kmax);
        L.pf_err = take(256);
        L.pf_part = take(kDenseSplitMax * sizeof(float) * dg::BM * (size_t)g.d_model);
    }
    // persistent-kernel buffers (bf16 models)
    if (g.dtype == ADA_DTYPE_BF16) {
        L.maps = take(sizeof(CUtensorMap) * (6 * (size_t)g.n_layers + 2));
        L.mm = take(sizeof(mg::MegaModel));
        L.exit_at = take(sizeof(int) * (g.n_layers + 1));
        L.xa = take(st::xfrag_bytes(g.d_model));
        L.xb = take(st::xfrag_bytes(g.d_model));
        L.xf = take(st::xfrag_bytes(g.d_model));
        L.xt = take(st::xfrag_bytes(g.d_model));
        L.xo = take(st::xfrag_bytes(qd));
        L.xh = take(st::xfrag_bytes(g.d_ff));
        L.ssq_a = take(sizeof(float) * (size_t)((g.d_model + 15) / 16) * st::MAX_COLS);
        L.ssq_b = take(sizeof(float) * (size_t)((g.d_model + 15) / 16) * st::MAX_COLS);
        L.qfrag = take((size_t)g.n_kv_heads * 2 * (g.head_dim / 16) * 1024);
        L.attn_cnt = take(sizeof(unsigned) * g.n_kv_heads * st::MAX_COLS);   // per (sequence of a launch, kv head)
        L.rope_freq = take(sizeof(double) * (g.head_dim / 2));
        L.part = take(kPartBytesPerCta * kPartMaxGrid);
        L.grid_ctr = take(256);
        L.pub = take(sizeof(mg::Pub) * 2);
        L.err = take(256);
        // sampled decoding: the logits and normalisers of the intermediate head that drew each token in flight, and the
        // random numbers of every sequence position
        L.q_stage = take(sizeof(float) * (size_t)batch * st::MAX_COLS * g.vocab);
        L.qinfo = take(sizeof(float4) * (size_t)batch * st::MAX_COLS);
        L.uniforms = take(sizeof(float) * (size_t)batch * max_seq * mg::SAMPLE_NU);
    }
    L.total = o;
    return L;
}

constexpr int kHeadBlocks = 148 * 4;

int check_cfg(const ada_config &g) {
    if (g.n_layers < 1 || g.n_layers > ADA_MAX_LAYERS - 1 || g.d_model < 8 || g.vocab < 2) return ADA_EINVAL;
    if (g.dtype != ADA_DTYPE_FP32 && g.dtype != ADA_DTYPE_BF16) return ADA_EINVAL;
    if (g.n_q_heads < 1 || g.n_kv_heads < 1 || g.n_q_heads % g.n_kv_heads) return ADA_EINVAL;
    if (g.d_model % 8 || g.d_ff % 8 || (g.n_q_heads * g.head_dim) % 8) return ADA_EUNSUPPORTED;
    if (g.head_dim % 32 || g.head_dim > 256 || g.head_dim < 32) return ADA_EUNSUPPORTED;
    return ADA_OK;
}

// ---- profiling: events around every launch when switched on ------------------------------------

constexpr size_t kProfMaxRec = 1 << 17;

struct Prof {
    ada_session *S;
    bool on;
    Prof(ada_session *S_, int cls, double bytes) : S(S_), on(S_->prof && S_->prof_rec.size() < kProfMaxRec) {
        if (!on) return;
        size_t i = S->prof_rec.size();
        while (S->prof_ev.size() < 2 * (i + 1)) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
            S->prof_ev.push_back(e);
        }
        S->prof_rec.push_back({cls, bytes});
        cudaEventRecord(S->prof_ev[2 * i], S->stream);
    }
    ~Prof() {
        if (on) cudaEventRecord(S->prof_ev[2 * (S->prof_rec.size() - 1) + 1], S->stream);
    }
};

// Fold the recorded events into the per-class sums (stream must be idle).
void prof_collect(ada_session *S) {
    for (size_t i = 0; i < S->prof_rec.size(); ++i) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, S->prof_ev[2 * i], S->prof_ev[2 * i + 1]) != cudaSuccess) continue;
        int cls = S->prof_rec[i].first;
        S->prof_ms[cls] += ms;
        S->prof_bytes[cls] += S->prof_rec[i].second;
        S->prof_launches[cls] += 1;
    }
    S->prof_rec.clear();
}

// ---- typed launch helpers --------------------------------------------------------------------

// ---- dense prompt pass: one decoder layer over a block of up to 128 prompt rows (rows 0 .. cur_rows - 1) -------

// One tcgen05 GEMM over the input last split into S->pf_hi / pf_lo (depth K): Y = or += X W^T.  Products with few
// tiles are split in depth over several CTAs per tile (shares added in a fixed order by k_dense_reduce).
int dense_gemm(ada_session *S, int cls, bool add, const void *W, int N, int K, float *Y, int ldy) {
    Prof pf(S, cls, (double)N * K * 2);
    CUtensorMap mhi, mlo, mw;
    int rc;
    if ((rc = make_map_2d(&mhi, S->pf_hi, dg::BM, K, dg::BM)) || (rc = make_map_2d(&mlo, S->pf_lo, dg::BM, K, dg::BM)) ||
        (rc = make_map_2d(&mw, W, N, K, dg::BN)))
        return rc;
    const int tiles = (N + dg::BN - 1) / dg::BN, nkb = K / dg::BK;
    int splits = 1;
    while (tiles * splits < 96 && splits * 2 <= nkb / 8 && (size_t)(splits * 2) * dg::BM * N * sizeof(float) <= S->pf_part_bytes && N % 4 == 0) splits *= 2;
    if (splits == 1) {
        if (add) dg::k_dense_gemm<1><<<tiles, dg::DTHREADS, dg::DSMEM_BYTES, S->stream>>>(mhi, mlo, mw, Y, ldy, S->cur_rows, N, K, 0, S->pf_err);
        else dg::k_dense_gemm<0><<<tiles, dg::DTHREADS, dg::DSMEM_BYTES, S->stream>>>(mhi, mlo, mw, Y, ldy, S->cur_rows, N, K, 0, S->pf_err);
        CK(cudaGetLastError());
        S->launches++;
    } else {
        const size_t stride = (size_t)dg::BM * N;
        dg::k_dense_gemm<0><<<dim3(tiles, splits), dg::DTHREADS, dg::DSMEM_BYTES, S->stream>>>(mhi, mlo, mw, S->pf_part, N, S->cur_rows, N, K, stride, S->pf_err);
        CK(cudaGetLastError());
        dg::k_dense_reduce<<<dim3((N / 4 + 255) / 256, S->cur_rows), 256, 0, S->stream>>>(S->pf_part, stride, splits, Y, ldy, S->cur_rows, N, add ? 1 : 0);
        CK(cudaGetLastError());
        S->launches += 2;
    }
    return ADA_OK;
}

int run_layer_dense(ada_session *S, int layer, int rows) {
    const ada_model *m = S->m;
    const ada_config &g = m->cfg;
    const LayerW &w = m->layers[layer];
    const int d = g.d_model, hd = g.head_dim, qd = g.n_q_heads * hd, kvd = g.n_kv_heads * hd, qkv_rows = S->c.qkv_rows;
    typedef __nv_bfloat16 T;
    int rc;
    S->layer_passes++;
    {
        Prof pf(S, 1, 0.0);
        dg::k_norm_split_rows<<<dg::BM, 256, 0, S->stream>>>(S->c.resid, rows, d, (const T *)w.attn_norm, g.rms_eps, S->pf_hi, S->pf_lo);
    }
    CK(cudaGetLastError());
    S->launches++;
    if ((const T *)w.wk == (const T *)w.wq + (size_t)qd * d && (const T *)w.wv == (const T *)w.wk + (size_t)kvd * d) {
        if ((rc = dense_gemm(S, 2, false, w.wq, qkv_rows, d, S->c.qkv, qkv_rows))) return rc;
    } else {
        if ((rc = dense_gemm(S, 2, false, w.wq, qd, d, S->c.qkv, qkv_rows))) return rc;
        if ((rc = dense_gemm(S, 2, false, w.wk, kvd, d, S->c.qkv + qd, qkv_rows))) return rc;
        if ((rc = dense_gemm(S, 2, false, w.wv, kvd, d, S->c.qkv + qd + kvd, qkv_rows))) return rc;
    }
    {
        Prof pf(S, 3, 0.0);
        k_rope_kv<T><<<rows, 128, 0, S->stream>>>(S->c, layer);
    }
    CK(cudaGetLastError());
    S->launches++;
    {
        Prof pf(S, 4, 0.0);
        const int group = g.n_q_heads / g.n_kv_heads;
        if (group != 1 && group != 2 && group != 4) return ADA_EUNSUPPORTED;
        const dim3 grid((rows + 64 / group - 1) / (64 / group), g.n_kv_heads);   // four warps of 16 / group positions each
#define PF_ATTN(H, G) dg::k_pf_attn_mma<H, G><<<grid, 128, 0, S->stream>>>(S->c, layer, rows)
        if (hd == 128) { if (group == 4) PF_ATTN(128, 4); else if (group == 2) PF_ATTN(128, 2); else PF_ATTN(128, 1); }
        else if (hd == 64) { if (group == 4) PF_ATTN(64, 4); else if (group == 2) PF_ATTN(64, 2); else PF_ATTN(64, 1); }
        else return ADA_EUNSUPPORTED;
#undef PF_ATTN
    }
    CK(cudaGetLastError());
    S->launches++;
    {
        Prof pf(S, 11, 0.0);
        dg::k_split_rows<<<dg::BM, 256, 0, S->stream>>>(S->c.attn_out, qd, rows, qd, S->pf_hi, S->pf_lo);
    }
    CK(cudaGetLastError());
    if ((rc = dense_gemm(S, 5, true, w.wo, d, qd, S->c.resid, d))) return rc;
    {
        Prof pf(S, 1, 0.0);
        dg::k_norm_split_rows<<<dg::BM, 256, 0, S->stream>>>(S->c.resid, rows, d, (const T *)w.ffn_norm, g.rms_eps, S->pf_hi, S->pf_lo);
    }
    CK(cudaGetLastError());
    if ((const T *)w.w_up == (const T *)w.w_gate + (size_t)g.d_ff * d) {
        if ((rc = dense_gemm(S, 6, false, w.w_gate, 2 * g.d_ff, d, S->c.gu, 2 * g.d_ff))) return rc;
    } else {
        if ((rc = dense_gemm(S, 6, false, w.w_gate, g.d_ff, d, S->c.gu, 2 * g.d_ff))) return rc;
        if ((rc = dense_gemm(S, 6, false, w.w_up, g.d_ff, d, S->c.gu + g.d_ff, 2 * g.d_ff))) return rc;
    }
    {
        Prof pf(S, 7, 0.0);
        k_swiglu<<<dim3((g.d_ff + 255) / 256, rows), 256, 0, S->stream>>>(S->c, layer);
    }
    CK(cudaGetLastError());
    {
        Prof pf(S, 11, 0.0);
        dg::k_split_rows<<<dg::BM, 256, 0, S->stream>>>(S->c.hact, g.d_ff, rows, g.d_ff, S->pf_hi, S->pf_lo);
    }
    CK(cudaGetLastError());
    S->launches += 4;
    if ((rc = dense_gemm(S, 8, true, w.w_down, d, g.d_ff, S->c.resid, d))) return rc;
    return ADA_OK;
}

template <typename T>
int launch_gemv(ada_session *S, int cls, int epi, const void *W, int N, int K, const float *X, int ldx, float *Y, int ldy, int sel) {
    Prof pf(S, cls, (double)N * K * sizeof(T));
    int blocks = std::min((N + 7) / 8, 148 * 4);
    if (epi == 0)
        k_gemv<T, 0><<<blocks, 256, 0, S->stream>>>(S->c, (const T *)W, N, K, X, ldx, Y, ldy, sel);
    else
        k_gemv<T, 1><<<blocks, 256, 0, S->stream>>>(S->c, (const T *)W, N, K, X, ldx, Y, ldy, sel);
    S->launches++;
    CK(cudaGetLastError());
    return ADA_OK;
}

template <typename T>
int launch_attn(ada_session *S, int layer, int rows) {
    const ada_config &g = S->m->cfg;
    Prof pf(S, 4, 0.0);
    dim3 grid(S->n_chunks, g.n_q_heads, rows);
    switch (g.head_dim / 32) {
        case 1: k_attn_partial<T, 1><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        case 2: k_attn_partial<T, 2><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        case 3: k_attn_partial<T, 3><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        case 4: k_attn_partial<T, 4><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        case 5: k_attn_partial<T, 5><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        case 6: k_attn_partial<T, 6><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        case 7: k_attn_partial<T, 7><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
        default: k_attn_partial<T, 8><<<grid, 32, 0, S->stream>>>(S->c, layer); break;
    }
    CK(cudaGetLastError());
    k_attn_combine<<<dim3(g.n_q_heads, rows), 64, 0, S->stream>>>(S->c, layer);
    CK(cudaGetLastError());
    S->launches += 2;
    return ADA_OK;
}

// One decoder layer over the rows active at `layer` (0-based); `rows` bounds the row indices.
template <typename T>
int run_layer_t(ada_session *S, int layer, int rows) {
    const ada_model *m = S->m;
    const ada_config &g = m->cfg;
    const LayerW &w = m->layers[layer];
    const int d = g.d_model, qd = g.n_q_heads * g.head_dim, qkv_rows = S->c.qkv_rows;
    const int ldx = d;
    int rc;
    S->layer_passes++;
    {
        Prof pf(S, 1, 0.0);
        k_rmsnorm<T><<<rows, 256, 0, S->stream>>>(S->c, (const T *)w.attn_norm, layer, S->c.xn, ldx);
    }
    CK(cudaGetLastError());
    S->launches++;
    {
        const int kvd = g.n_kv_heads * g.head_dim;
        const bool fused = (const T *)w.wk == (const T *)w.wq + (size_t)qd * d && (const T *)w.wv == (const T *)w.wk + (size_t)kvd * d;
        if (fused) {
            if ((rc = launch_gemv<T>(S, 2, 0, w.wq, qkv_rows, d, S->c.xn, ldx, S->c.qkv, qkv_rows, layer))) return rc;
        } else {
            if ((rc = launch_gemv<T>(S, 2, 0, w.wq, qd, d, S->c.xn, ldx, S->c.qkv, qkv_rows, layer))) return rc;
            if ((rc = launch_gemv<T>(S, 2, 0, w.wk, kvd, d, S->c.xn, ldx, S->c.qkv + qd, qkv_rows, layer))) return rc;
            if ((rc = launch_gemv<T>(S, 2, 0, w.wv, kvd, d, S->c.xn, ldx, S->c.qkv + qd + kvd, qkv_rows, layer))) return rc;
        }
    }
    {
        Prof pf(S, 3, 0.0);
        k_rope_kv<T><<<rows, 128, 0, S->stream>>>(S->c, layer);
    }
    CK(cudaGetLastError());
    S->launches++;
    if ((rc = launch_attn<T>(S, layer, rows))) return rc;
    if ((rc = launch_gemv<T>(S, 5, 1, w.wo, d, qd, S->c.attn_out, qd, S->c.resid, d, layer))) return rc;
    {
        Prof pf(S, 1, 0.0);
        k_rmsnorm<T><<<rows, 256, 0, S->stream>>>(S->c, (const T *)w.ffn_norm, layer, S->c.xn, ldx);
    }
    CK(cudaGetLastError());
    S->launches++;
    if ((const T *)w.w_up == (const T *)w.w_gate + (size_t)g.d_ff * d) {
        if ((rc = launch_gemv<T>(S, 6, 0, w.w_gate, 2 * g.d_ff, d, S->c.xn, ldx, S->c.gu, 2 * g.d_ff, layer))) return rc;
    } else {
        if ((rc = launch_gemv<T>(S, 6, 0, w.w_gate, g.d_ff, d, S->c.xn, ldx, S->c.gu, 2 * g.d_ff, layer))) return rc;
        if ((rc = launch_gemv<T>(S, 6, 0, w.w_up, g.d_ff, d, S->c.xn, ldx, S->c.gu + g.d_ff, 2 * g.d_ff, layer))) return rc;
    }
    {
        Prof pf(S, 7, 0.0);
        k_swiglu<<<dim3((g.d_ff + 255) / 256, rows), 256, 0, S->stream>>>(S->c, layer);
    }
    CK(cudaGetLastError());
    S->launches++;
    if ((rc = launch_gemv<T>(S, 8, 1, w.w_down, d, g.d_ff, S->c.hact, g.d_ff, S->c.resid, d, layer))) return rc;
    return ADA_OK;
}

// Head over the rows picked by `sel`: layer1 >= 1 is the intermediate head registered there,
// layer1 == 0 the final LM head (unscaled, T = I).
template <typename T>
int run_head_t(ada_session *S, int layer1, int sel, int rows) {
    const ada_model *m = S->m;
    const ada_config &g = m->cfg;
    const int d = g.d_model;
    int rc;
    {
        Prof pf(S, 1, 0.0);
        k_rmsnorm<T><<<rows, 256, 0, S->stream>>>(S->c, (const T *)m->final_norm, sel, S->c.xn, d);
    }
    CK(cudaGetLastError());
    S->launches++;
    const float *x = S->c.xn;
    float scale = 1.0f;
    if (layer1 > 0) {
        scale = m->head_scale[layer1];
        if (m->head_T[layer1]) {
            if ((rc = launch_gemv<T>(S, 10, 0, m->head_T[layer1], d, d, S->c.xn, d, S->t_out, d, sel))) return rc;
            x = S->t_out;
        }
    }
    const int store = (layer1 == 0 && S->capture_dev) ? 1 : 0;
    {
        Prof pf(S, 9, (double)g.vocab * d * sizeof(T));
        k_head_partial<T><<<S->head_blocks, 256, 0, S->stream>>>(S->c, (const T *)m->lm_head, x, d, scale, sel, store);
        CK(cudaGetLastError());
        k_head_final<<<rows, 32, 0, S->stream>>>(S->c, S->head_blocks, sel);
    }
    CK(cudaGetLastError());
    S->launches += 2;
    return ADA_OK;
}

int run_layer(ada_session *S, int layer, int rows) {
    if (S->dense_on) return run_layer_dense(S, layer, rows);
    return S->m->cfg.dtype == ADA_DTYPE_BF16 ? run_layer_t<__nv_bfloat16>(S, layer, rows) : run_layer_t<float>(S, layer, rows);
}
int run_head(ada_session *S, int layer1, int sel, int rows) {
    return S->m->cfg.dtype == ADA_DTYPE_BF16 ? run_head_t<__nv_bfloat16>(S, layer1, sel, rows) : run_head_t<float>(S, layer1, sel, rows);
}

int step_begin(ada_session *S) {
    const ada_model *m = S->m;
    Prof pf(S, 0, 0.0);
    if (m->cfg.dtype == ADA_DTYPE_BF16)
        k_step_begin<__nv_bfloat16><<<1, 256, 0, S->stream>>>(S->c, (const __nv_bfloat16 *)m->tok_embed, m->cfg.rope_base);
    else
        k_step_begin<float><<<1, 256, 0, S->stream>>>(S->c, (const float *)m->tok_embed, m->cfg.rope_base);
    CK(cudaGetLastError());
    S->launches++;
    return ADA_OK;
}

int capture_rows(ada_session *S, int row0) {
    if (!S->capture_dev) return ADA_OK;
    Prof pf(S, 11, 0.0);
    k_capture<<<64, 256, 0, S->stream>>>(S->c, row0);
    CK(cudaGetLastError());
    k_capture_advance<<<1, 32, 0, S->stream>>>(S->c);
    CK(cudaGetLastError());
    S->launches += 2;
    return ADA_OK;
}

// Read n_climbing / n_done (one stream synchronisation).
int read_progress(ada_session *S, int *n_climbing, int *n_done) {
    CK(cudaMemcpyAsync(S->pinned, &S->c.st->n_climbing, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, S->stream));
    CK(cudaStreamSynchronize(S->stream));
    S->syncs++;
    *n_climbing = S->pinned[0];
    *n_done = S->pinned[1];
    return ADA_OK;
}

int ensure_pages(ada_session *S, int seq, int positions) {
    int need = (positions + S->page_tokens - 1) / S->page_tokens;
    if (need > S->max_pages) return ADA_ECAPACITY;
    std::vector<int> &pg = S->seq_pages[seq];
    if ((int)pg.size() >= need) return ADA_OK;
    if ((int)S->free_pages.size() < need - (int)pg.size()) return ADA_ECAPACITY;
    size_t first = pg.size();
    while ((int)pg.size() < need) { pg.push_back(S->free_pages.back()); S->free_pages.pop_back(); }
    CK(cudaMemcpyAsync(S->c.page_table + (size_t)seq * S->c.max_pages + first, pg.data() + first,
                       sizeof(int32_t) * (pg.size() - first), cudaMemcpyHostToDevice, S->stream));
    CK(cudaStreamSynchronize(S->stream));  // pg may reallocate before the copy is consumed
    return ADA_OK;
}

void add_stats(ada_session *S, const DevStats &d, ada_stats *out, float ms, int64_t l0, int64_t s0, int64_t p0) {
    if (!out) return;
    out->steps += d.steps; out->head_evals += d.head_evals; out->early_exits += d.early_exits;
    out->verify_steps += d.verify_steps; out->accepted += d.accepted; out->rejected += d.rejected;
    out->discarded += d.discarded; out->row_layers += d.row_layers; out->truncated += d.truncated;
    for (int i = 0; i < ADA_MAX_LAYERS; ++i) out->exits_at_layer[i] += d.exits_at_layer[i];
    out->layer_passes += S->layer_passes - p0 + d.layer_passes;
    out->host_syncs += S->syncs - s0;
    out->kernel_launches += S->launches - l0;
    out->decode_ms += ms;
    out->path = (S->mega && S->path == 1) ? 1 : 0;
}

// ---- persistent-kernel path --------------------------------------------------------------------

template <int HD> const void *persistent_kernel() { return (const void *)mg::k_decode_persistent<HD>; }
const void *persistent_kernel_for(int hd) { return hd == 64 ? persistent_kernel<64>() : persistent_kernel<128>(); }

// Whether a model's shape and dtype are ones the persistent kernel is built for (the session adds its
// own conditions: at most eight token columns per sequence, 64-token pages).
bool model_fits_persistent(const ada_config &g) {
    const int qd = g.n_q_heads * g.head_dim, group = g.n_q_heads / g.n_kv_heads;
    if (g.dtype != ADA_DTYPE_BF16) return false;
    if ((g.head_dim != 64 && g.head_dim != 128) || group > 4) return false;
    if (g.d_model % 64 || qd % 64 || g.d_ff % 64) return false;
    return true;
}

// Decide whether this session can run the persistent kernel and build what it needs: tensor maps
// of every weight matrix, the device-side model description, the argument block.  A session that
// does not qualify runs one kernel per operation (path 0) and says so through ada_debug_get_path and
// ada_stats.path; a session that qualifies but cannot be set up (no cooperative launch, a tensor map
// the driver refuses) fails with that error instead of quietly taking the slow path.
int setup_persistent(ada_session *S, const Layout &lay) {
    const ada_model *m = S->m;
    const ada_config &g = m->cfg;
    S->mega = false;
    S->path = 0;
    const int qd = g.n_q_heads * g.head_dim;
    if (!model_fits_persistent(g) || S->slots > st::MAX_COLS || S->page_tokens != mg::ATT_PAGE) return ADA_OK;
    int dev = 0, sms = 0, coop = 0, nb = 0;
    CK(cudaGetDevice(&dev));
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CK(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    const void *kern = persistent_kernel_for(g.head_dim);
    if (!coop || sms < 1) {
        g_cuda_err = "the device does not support cooperative launches, which the persistent decode kernel needs";
        return ADA_EUNSUPPORTED;
    }
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st::SMEM_BYTES));
    CK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, kern, st::THREADS, st::SMEM_BYTES));
    if (nb < 1) {
        g_cuda_err = "the persistent decode kernel does not fit on one multiprocessor of this device";
        return ADA_EUNSUPPORTED;
    }
    S->grid = std::min(sms, S->head_blocks);
    const int L = g.n_layers;
    char *b = (char *)S->scratch;
    S->maps_dev = (CUtensorMap *)(b + lay.maps);
    S->mm_dev = (mg::MegaModel *)(b + lay.mm);
    S->exit_at_dev = (int *)(b + lay.exit_at);
    S->maps_host.assign(6 * (size_t)L + 2, CUtensorMap());
    S->mm_host.reset(new mg::MegaModel());
    mg::MegaModel &M = *S->mm_host;
    memset(&M, 0, sizeof(M));
    int rc;
    for (int l = 0; l < L; ++l) {
        const LayerW &w = m->layers[l];
        const bool gu_fused = (const __nv_bfloat16 *)w.w_up == (const __nv_bfloat16 *)w.w_gate + (size_t)g.d_ff * g.d_model;
        if (!w.wqkv_perm) return ADA_ESTATE;
        if ((rc = make_weight_map(&S->maps_host[5 * l + 0], w.wqkv_perm, S->c.qkv_rows, g.d_model))) return rc;
        if ((rc = make_weight_map(&S->maps_host[5 * l + 1], w.wo, g.d_model, qd))) return rc;
        if ((rc = make_weight_map(&S->maps_host[5 * l + 2], w.w_gate, gu_fused ? 2 * g.d_ff : g.d_ff, g.d_model))) return rc;
        if (!gu_fused && (rc = make_weight_map(&S->maps_host[5 * l + 3], w.w_up, g.d_ff, g.d_model))) return rc;
        if ((rc = make_weight_map(&S->maps_host[5 * l + 4], w.w_down, g.d_model, g.d_ff))) return rc;
        M.layer[l].wqkv = S->maps_dev + 5 * l + 0;
        M.layer[l].wo = S->maps_dev + 5 * l + 1;
        M.layer[l].wgu = S->maps_dev + 5 * l + 2;
        M.layer[l].wup = gu_fused ? nullptr : S->maps_dev + 5 * l + 3;
        M.layer[l].wdown = S->maps_dev + 5 * l + 4;
        M.layer[l].attn_norm = (const __nv_bfloat16 *)w.attn_norm;
        M.layer[l].ffn_norm = (const __nv_bfloat16 *)w.ffn_norm;
    }
    if ((rc = make_weight_map(&S->maps_host[5 * L], m->lm_head, g.vocab, g.d_model))) return rc;
    M.lm_head = S->maps_dev + 5 * L;
    M.tok_embed = (const __nv_bfloat16 *)m->tok_embed;
    M.final_norm = (const __nv_bfloat16 *)m->final_norm;
    M.rope_base = g.rope_base;
    CK(cudaMemcpyAsync(S->maps_dev, S->maps_host.data(), sizeof(CUtensorMap) * S->maps_host.size(), cudaMemcpyHostToDevice, S->stream));
    CK(cudaMemcpyAsync(S->mm_dev, &M, sizeof(M), cudaMemcpyHostToDevice, S->stream));
    std::vector<double> freq(g.head_dim / 2);
    for (int i = 0; i < g.head_dim / 2; ++i) freq[i] = pow((double)g.rope_base, -2.0 * i / g.head_dim);
    CK(cudaMemcpyAsync(b + lay.rope_freq, freq.data(), sizeof(double) * freq.size(), cudaMemcpyHostToDevice, S->stream));
    CK(cudaStreamSynchronize(S->stream));
    mg::MegaArgs &a = S->margs;
    a.c = S->c;
    a.mm = S->mm_dev;
    a.exit_at = S->exit_at_dev;
    a.XA = (__nv_bfloat16 *)(b + lay.xa); a.XB = (__nv_bfloat16 *)(b + lay.xb); a.XO = (__nv_bfloat16 *)(b + lay.xo);
    a.XH = (__nv_bfloat16 *)(b + lay.xh); a.XF = (__nv_bfloat16 *)(b + lay.xf); a.XT = (__nv_bfloat16 *)(b + lay.xt);
    a.ssq_a = (float *)(b + lay.ssq_a); a.ssq_b = (float *)(b + lay.ssq_b);
    a.qfrag = (uint32_t *)(b + lay.qfrag);
    a.attn_part = S->c.attn_part;
    a.head_part = S->c.head_part;
    a.attn_cnt = (unsigned *)(b + lay.attn_cnt);
    a.rope_freq = (const double *)(b + lay.rope_freq);
    a.part = S->grid <= kPartMaxGrid ? (unsigned long long *)(b + lay.part) : nullptr;
    a.grid_ctr = (unsigned *)(b + lay.grid_ctr);
    a.pub = (mg::Pub *)(b + lay.pub);
    a.err = (int *)(b + lay.err);
    a.step_budget = S->steps_per_launch;
    a.seq0 = 0;
    a.nseq = 1;
    a.wait_ns = S->wait_ns;
    a.store_logits = 0;
    a.sampling = 0;
    a.inv_temp = 1.0f;
    a.uniforms = (const float *)(b + lay.uniforms);
    a.q_stage = (float *)(b + lay.q_stage);
    a.qinfo = (float4 *)(b + lay.qinfo);
    a.trace = st::Trace{nullptr, nullptr, 0};
    a.trace_step0 = a.trace_step1 = 0;
    S->mega = true;
    S->path = 1;
    return ADA_OK;
}

// Run the persistent kernel until the call's token targets are met.
// The kernel holds eight token columns.  A sequence needs max_early + 1 of them, so a launch decodes
// min(8 / (max_early + 1), batch) sequences together (one weight stream for all of them, lock-step: every step runs
// up to the highest layer any of them reaches); the sequences seq_begin .. seq_end - 1 go in such groups, one group
// after another.  `together` false: one sequence per launch (prompt passes, which use all eight columns).
int run_persistent(ada_session *S, const int32_t *exit_layers, int n_exit, bool plain, int seq_begin, int seq_end, bool together) {
    const ada_model *m = S->m;
    const ada_config &g = m->cfg;
    const int L = g.n_layers;
    std::vector<int> ex(L + 1, 0);
    mg::MegaModel &M = *S->mm_host;
    if (!plain) {
        for (int i = 0; i < n_exit; ++i) {
            const int e = exit_layers[i];
            ex[e] = 1 + i;
            M.layer[e].has_head = 1;
            M.layer[e].head_scale = m->head_scale[e];
            M.layer[e].wT = nullptr;
            if (m->head_T[e]) {
                CUtensorMap &tm = S->maps_host[5 * (size_t)L + 1 + e];
                int rc = make_weight_map(&tm, m->head_T[e], g.d_model, g.d_model);
                if (rc) return rc;
                CK(cudaMemcpyAsync(S->maps_dev + 5 * L + 1 + e, &tm, sizeof(tm), cudaMemcpyHostToDevice, S->stream));
                M.layer[e].wT = S->maps_dev + 5 * L + 1 + e;
            }
            CK(cudaMemcpyAsync(&S->mm_dev->layer[e], &M.layer[e], sizeof(mg::MegaLayer), cudaMemcpyHostToDevice, S->stream));
        }
    }
    CK(cudaMemcpyAsync(S->exit_at_dev, ex.data(), sizeof(int) * (L + 1), cudaMemcpyHostToDevice, S->stream));
    // a call that ended on a device-side error may have left the error word and the attention counters set
    CK(cudaMemsetAsync(S->margs.err, 0, sizeof(int), S->stream));
    CK(cudaMemsetAsync(S->margs.attn_cnt, 0, sizeof(unsigned) * g.n_kv_heads * st::MAX_COLS, S->stream));
    CK(cudaStreamSynchronize(S->stream));   // ex and the maps live on the host until copied
    S->syncs++;
    const void *kern = persistent_kernel_for(g.head_dim);
    const int per_launch = together ? std::max(1, st::MAX_COLS / S->slots) : 1;
    for (int sq = seq_begin; sq < seq_end; sq += per_launch) {
        mg::MegaArgs a = S->margs;
        a.c = S->c;   // capture pointers may have changed
        a.seq0 = sq;
        a.nseq = std::min(per_launch, seq_end - sq);
        a.step_budget = S->steps_per_launch;
        a.wait_ns = S->wait_ns;
        a.store_logits = (S->capture_dev && sq == 0) ? 1 : 0;
        a.sampling = S->sampling ? 1 : 0;
        a.inv_temp = S->sampling ? S->inv_temp : 1.0f;
        CK(cudaMemsetAsync(&S->c.st->n_done, 0, sizeof(int32_t), S->stream));
        for (long long guard = 0;; ++guard) {
            if (guard > (1ll << 24)) return ADA_ETIMEOUT;
            CK(cudaMemsetAsync(a.grid_ctr, 0, sizeof(unsigned), S->stream));
            CK(cudaMemsetAsync(a.pub, 0, sizeof(mg::Pub) * 2, S->stream));
            if (a.part) CK(cudaMemsetAsync(a.part, 0, kPartBytesPerCta * (size_t)S->grid, S->stream));
            void *params[] = {(void *)&a};
            CK(cudaLaunchCooperativeKernel(kern, dim3(S->grid), dim3(st::THREADS), params, st::SMEM_BYTES, S->stream));
            S->launches++;
            CK(cudaMemcpyAsync(S->pinned, &S->c.st->n_climbing, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, S->stream));
            CK(cudaMemcpyAsync(S->pinned + 2, a.err, sizeof(int32_t), cudaMemcpyDeviceToHost, S->stream));
            CK(cudaStreamSynchronize(S->stream));
            S->syncs++;
            if (S->pinned[2] != 0) {
                g_cuda_err = "persistent decode kernel: device-side error " + std::to_string(S->pinned[2]);
                return S->pinned[2] == mg::ERR_BAD_STATE ? ADA_ESTATE : ADA_ETIMEOUT;
            }
            if (S->pinned[1] >= 1) break;   // the sequences of this launch have reached their targets
        }
    }
    return ADA_OK;
}

// Shared body of both decode calls.
int decode(ada_session *S, int n_tokens, float gamma, const int32_t *exit_layers, int n_exit, int max_early, int eos_id,
           int32_t *out_host, ada_stats *stats) {
    const ada_model *m = S->m;
    const int L = m->cfg.n_layers;
    if (!out_host || n_tokens < 1 || eos_id >= m->cfg.vocab) return ADA_EINVAL;
    if (eos_id < 0) eos_id = -1;
    int n_live = 0;
    for (int s = 0; s < S->batch; ++s) {
        if (!S->prefilled[s]) return ADA_ESTATE;
        n_live += !S->finished[s];
    }
    if (n_live == 0) return ADA_ESTATE;   // every sequence has already ended on its end-of-sequence token
    if (max_early < 0 || max_early > S->max_early) return ADA_ECAPACITY;
    for (int e = 0; e < n_exit; ++e) {
        if (exit_layers[e] < 1 || exit_layers[e] >= L || !m->has_head[exit_layers[e]]) return ADA_EINVAL;
        if (e && exit_layers[e] <= exit_layers[e - 1]) return ADA_EINVAL;
    }
    CallTargets tg;
    memset(&tg, 0, sizeof(tg));
    int max_steps_plain = 0;
    for (int s = 0; s < S->batch; ++s) {
        int target = S->h_prompt[s] + S->h_reported[s] + (S->finished[s] ? 0 : n_tokens);
        if (target + 1 > S->max_seq) return ADA_ECAPACITY;
        int rc = ensure_pages(S, s, target + 1);
        if (rc) return rc;
        tg.target_len[s] = target;
        max_steps_plain = std::max(max_steps_plain, target - S->h_len[s]);
    }
    const int64_t l0 = S->launches, s0 = S->syncs, p0 = S->layer_passes;
    const int rows = S->batch * S->slots;
    int rc;
    // zero the device counters, set targets
    CK(cudaMemsetAsync(&S->c.st->st, 0, sizeof(DevStats), S->stream));
    int tape_n = (int)std::min<size_t>(S->tape.size(), kMaxTape);
    if (tape_n) CK(cudaMemcpyAsync(S->c.st->tape, S->tape.data(), tape_n, cudaMemcpyHostToDevice, S->stream));
    CK(cudaEventRecord(S->ev0, S->stream));
    k_call_begin<<<1, 32, 0, S->stream>>>(S->c, tg, gamma, max_early, tape_n, eos_id);
    CK(cudaGetLastError());
    S->launches++;

    const bool plain = (n_exit == 0 || max_early == 0);
    if (S->mega && S->path == 1) {
        if ((rc = run_persistent(S, exit_layers, n_exit, plain, 0, S->batch, true))) return rc;
    } else if (plain) {
        // every step is one token through all layers; the step count is known, no read-back needed
        for (int it = 0; it < max_steps_plain; ++it) {
            if ((rc = step_begin(S))) return rc;
            for (int l = 0; l < L; ++l) if ((rc = run_layer(S, l, rows))) return rc;
            if ((rc = run_head(S, 0, SEL_FINAL, rows))) return rc;
            {
                Prof pf(S, 0, 0.0);
                k_verify<<<1, 32, 0, S->stream>>>(S->c);
            }
            CK(cudaGetLastError());
            S->launches++;
            if ((rc = capture_rows(S, 0))) return rc;
        }
    } else {
        int n_done = 0, n_climbing = 0;
        if ((rc = read_progress(S, &n_climbing, &n_done))) return rc;
        // generous bound on the loop: every step emits or verifies at least one token
        long long guard = (long long)(n_tokens + 2) * (max_early + 2) * 4 + 16;
        while (n_done < S->batch) {
            if (--guard < 0) return ADA_ETIMEOUT;
            if ((rc = step_begin(S))) return rc;
            int e_i = 0;
            bool reached_top = true;
            for (int l = 0; l < L; ++l) {
                if ((rc = run_layer(S, l, rows))) return rc;
                if (e_i < n_exit && exit_layers[e_i] == l + 1) {
                    if ((rc = run_head(S, l + 1, SEL_HEAD, rows))) return rc;
                    {
                        Prof pf(S, 0, 0.0);
                        k_exit_control<<<1, 32, 0, S->stream>>>(S->c, l + 1);
                    }
                    CK(cudaGetLastError());
                    S->launches++;
                    ++e_i;
                    if ((rc = read_progress(S, &n_climbing, &n_done))) return rc;
                    if (n_climbing == 0) { reached_top = false; break; }
                }
            }
            if (reached_top) {
                if ((rc = run_head(S, 0, SEL_FINAL, rows))) return rc;
                {
                    Prof pf(S, 0, 0.0);
                    k_verify<<<1, 32, 0, S->stream>>>(S->c);
                }
                CK(cudaGetLastError());
                S->launches++;
                if ((rc = capture_rows(S, 0))) return rc;
                if ((rc = read_progress(S, &n_climbing, &n_done))) return rc;
            }
        }
    }
    CK(cudaEventRecord(S->ev1, S->stream));
    // results: how far every sequence got (a verified end-of-sequence token ends it before the requested
    // count), then its tokens
    int32_t len_host[ADA_MAX_BATCH], eos_host[ADA_MAX_BATCH];
    CK(cudaMemcpyAsync(len_host, S->c.st->len, sizeof(int32_t) * S->batch, cudaMemcpyDeviceToHost, S->stream));
    CK(cudaMemcpyAsync(eos_host, S->c.st->eos_hit, sizeof(int32_t) * S->batch, cudaMemcpyDeviceToHost, S->stream));
    DevStats ds;
    CK(cudaMemcpyAsync(&ds, &S->c.st->st, sizeof(DevStats), cudaMemcpyDeviceToHost, S->stream));
    int32_t hl_n = 0;
    if (S->head_log_host) {
        CK(cudaMemcpyAsync(&hl_n, &S->c.st->head_log_n, sizeof(int32_t), cudaMemcpyDeviceToHost, S->stream));
    }
    if (eos_id < 0) {   // no end-of-sequence token: every sequence still running delivers the requested count
        for (int s = 0; s < S->batch; ++s) {
            if (S->finished[s]) {
                for (int i = 0; i < n_tokens; ++i) out_host[(size_t)s * n_tokens + i] = S->eos_tok[s];
                continue;
            }
            CK(cudaMemcpyAsync(out_host + (size_t)s * n_tokens, S->c.tokens + (size_t)s * S->max_seq + S->h_prompt[s] + S->h_reported[s],
                               sizeof(int32_t) * n_tokens, cudaMemcpyDeviceToHost, S->stream));
        }
    }
    CK(cudaStreamSynchronize(S->stream));
    S->syncs++;
    int emitted[ADA_MAX_BATCH];
    for (int s = 0; s < S->batch; ++s) {
        emitted[s] = eos_id < 0 ? n_tokens : std::min(n_tokens, std::max(0, len_host[s] - (S->h_prompt[s] + S->h_reported[s])));
        if (S->finished[s]) emitted[s] = 0;
    }
    if (eos_id >= 0) {
        for (int s = 0; s < S->batch; ++s) {
            int32_t *row = out_host + (size_t)s * n_tokens;
            if (emitted[s] > 0)
                CK(cudaMemcpyAsync(row, S->c.tokens + (size_t)s * S->max_seq + S->h_prompt[s] + S->h_reported[s],
                                   sizeof(int32_t) * emitted[s], cudaMemcpyDeviceToHost, S->stream));
            for (int i = emitted[s]; i < n_tokens; ++i) row[i] = S->finished[s] ? S->eos_tok[s] : eos_id;
        }
        CK(cudaStreamSynchronize(S->stream));
        S->syncs++;
    }
    if (S->head_log_host) {
        int n = std::min(hl_n, S->head_log_cap);
        if (n > 0) CK(cudaMemcpy(S->head_log_host, S->c.head_log, sizeof(float) * 4 * n, cudaMemcpyDeviceToHost));
        if (S->head_log_n_out) *S->head_log_n_out = hl_n;
    }
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, S->ev0, S->ev1));
    for (int s = 0; s < S->batch; ++s) {
        S->h_reported[s] += emitted[s];
        S->h_len[s] = S->h_prompt[s] + S->h_reported[s];
        if (eos_id >= 0 && eos_host[s] && !S->finished[s]) {
            S->finished[s] = 1;
            S->eos_tok[s] = eos_id;
            if (stats) stats->finished += 1;
        }
        if (stats) stats->emitted[s] += emitted[s];
    }
    S->tape.clear();
    if (S->prof) {
        prof_collect(S);
        const ada_config &g = m->cfg;
        const double esz = (double)m->esz, d = g.d_model, qdm = (double)g.n_q_heads * g.head_dim;
        const double wbytes[ADA_PROF_CLASSES] = {0, 0, (double)S->c.qkv_rows * d * esz, 0, 0, d * qdm * esz, 2.0 * g.d_ff * d * esz, 0,
                                                 d * g.d_ff * esz, (double)g.vocab * d * esz, d * d * esz, 0};
        for (int i = 0; i < ADA_PROF_CLASSES; ++i) {   // phases of the persistent kernel, timed on the device
            S->prof_ms[i] += (double)ds.phase_ns[i] * 1e-6;
            S->prof_launches[i] += ds.phase_count[i];
            S->prof_bytes[i] += wbytes[i] * (double)ds.phase_count[i];
        }
    }
    add_stats(S, ds, stats, ms, l0, s0, p0);
    return ADA_OK;
}

}  // namespace

// =============================================================================== C ABI

extern "C" {

const char *ada_strerror(int code) {
    switch (code) {
        case ADA_OK: return "ok";
        case ADA_EINVAL: return "invalid argument";
        case ADA_ESTATE: return "wrong call order or missing tensor";
        case ADA_ECAPACITY: return "capacity exceeded (KV pages, max_seq_len, max_early or scratch)";
        case ADA_ECUDA: return "CUDA error";
        case ADA_ETIMEOUT: return "bounded wait expired";
        case ADA_EUNSUPPORTED: return "unsupported shape or dtype";
        default: return "unknown error";
    }
}

const char *ada_last_cuda_error(void) { return g_cuda_err.c_str(); }

int ada_model_create(const ada_config *cfg, ada_model **out) {
    if (!cfg || !out) return ADA_EINVAL;
    int rc = check_cfg(*cfg);
    if (rc) return rc;
    ada_model *m = new ada_model();
    m->cfg = *cfg;
    m->esz = cfg->dtype == ADA_DTYPE_BF16 ? 2 : 4;
    m->layers.resize(cfg->n_layers);
    m->has_head.assign(cfg->n_layers + 1, 0);
    m->head_T.assign(cfg->n_layers + 1, nullptr);
    m->head_scale.assign(cfg->n_layers + 1, 1.0f);
    *out = m;
    return ADA_OK;
}

int ada_model_set_tensor(ada_model *m, const char *name, const void *dev_ptr, size_t bytes) {
    if (!m || !name || !dev_ptr) return ADA_EINVAL;
    if (m->finalized) return ADA_ESTATE;
    if ((uintptr_t)dev_ptr % 16) return ADA_EINVAL;
    const ada_config &g = m->cfg;
    const size_t d = g.d_model, qd = (size_t)g.n_q_heads * g.head_dim;
    const size_t qkv_rows = (size_t)(g.n_q_heads + 2 * g.n_kv_heads) * g.head_dim;
    size_t want = 0;
    const void **slot = nullptr;
    std::string n(name);
    if (n == "tok_embed") { want = (size_t)g.vocab * d; slot = &m->tok_embed; }
    else if (n == "lm_head") { if (g.tied_lm_head) return ADA_EINVAL; want = (size_t)g.vocab * d; slot = &m->lm_head; }
    else if (n == "final_norm") { want = d; slot = &m->final_norm; }
    else if (n.rfind("layers.", 0) == 0) {
        size_t dot = n.find('.', 7);
        if (dot == std::string::npos) return ADA_EINVAL;
        int l = -1;
        try { l = std::stoi(n.substr(7, dot - 7)); } catch (...) { return ADA_EINVAL; }
        if (l < 0 || l >= g.n_layers) return ADA_EINVAL;
        std::string f = n.substr(dot + 1);
        LayerW &w = m->layers[l];
        const size_t kvd = (size_t)g.n_kv_heads * g.head_dim;
        const char *base = (const char *)dev_ptr;
        if (f == "attn_norm") { want = d; slot = &w.attn_norm; }
        else if (f == "ffn_norm") { want = d; slot = &w.ffn_norm; }
        else if (f == "wq") { want = qd * d; slot = &w.wq; }
        else if (f == "wk") { want = kvd * d; slot = &w.wk; }
        else if (f == "wv") { want = kvd * d; slot = &w.wv; }
        else if (f == "wqkv") {   // the three matrices stacked in one tensor: q rows, k rows, v rows
            if (bytes != qkv_rows * d * m->esz) return ADA_EINVAL;
            w.wq = base; w.wk = base + qd * d * m->esz; w.wv = base + (qd + kvd) * d * m->esz;
            return ADA_OK;
        }
        else if (f == "wo") { want = d * qd; slot = &w.wo; }
        else if (f == "w_gate") { want = (size_t)g.d_ff * d; slot = &w.w_gate; }
        else if (f == "w_up") { want = (size_t)g.d_ff * d; slot = &w.w_up; }
        else if (f == "w_gate_up") {   // gate rows stacked over up rows
            if (bytes != 2 * (size_t)g.d_ff * d * m->esz) return ADA_EINVAL;
            w.w_gate = base; w.w_up = base + (size_t)g.d_ff * d * m->esz;
            return ADA_OK;
        }
        else if (f == "w_down") { want = d * (size_t)g.d_ff; slot = &w.w_down; }
        else return ADA_EINVAL;
    } else return ADA_EINVAL;
    if (bytes != want * m->esz) return ADA_EINVAL;
    *slot = dev_ptr;
    return ADA_OK;
}

size_t ada_model_arena_bytes(const ada_model *m) {
    if (!m || !model_fits_persistent(m->cfg)) return 0;
    const ada_config &g = m->cfg;
    const size_t per_layer = align_up((size_t)(g.n_q_heads + 2 * g.n_kv_heads) * g.head_dim * g.d_model * 2, 256);
    return per_layer * g.n_layers;
}

int ada_model_set_arena(ada_model *m, void *arena_dev, size_t bytes) {
    if (!m || !arena_dev) return ADA_EINVAL;
    if (m->finalized) return ADA_ESTATE;
    if ((uintptr_t)arena_dev % 256) return ADA_EINVAL;
    if (bytes < ada_model_arena_bytes(m)) return ADA_ECAPACITY;
    m->arena = arena_dev;
    m->arena_bytes = bytes;
    return ADA_OK;
}

int ada_model_set_exit_head(ada_model *m, int32_t layer, const void *T_dev, float logit_scale) {
    if (!m) return ADA_EINVAL;
    if (layer < 1 || layer >= m->cfg.n_layers) return ADA_EINVAL;
    if (!(logit_scale > 0.0f)) return ADA_EINVAL;
    if (T_dev && (uintptr_t)T_dev % 16) return ADA_EINVAL;
    m->has_head[layer] = 1;
    m->head_T[layer] = T_dev;
    m->head_scale[layer] = logit_scale;
    return ADA_OK;
}

int ada_model_finalize(ada_model *m) {
    if (!m) return ADA_EINVAL;
    if (m->finalized) return ADA_OK;
    if (!m->tok_embed || !m->final_norm) return ADA_ESTATE;
    if (m->cfg.tied_lm_head) m->lm_head = m->tok_embed;
    if (!m->lm_head) return ADA_ESTATE;
    for (const LayerW &w : m->layers)
        if (!w.attn_norm || !w.wq || !w.wk || !w.wv || !w.wo || !w.ffn_norm || !w.w_gate || !w.w_up || !w.w_down) return ADA_ESTATE;
    const size_t need = ada_model_arena_bytes(m);
    if (need) {
        // Repack on load: q | k | v of every layer, copied into the caller's arena with the rows of each q and
        // k head reordered (see k_repack_qkv).  The tensors the caller lent stay as they are.
        if (!m->arena || m->arena_bytes < need) {
            g_cuda_err = "ada_model_finalize: this model needs an arena of ada_model_arena_bytes() bytes (ada_model_set_arena)";
            return ADA_ESTATE;
        }
        const ada_config &g = m->cfg;
        const size_t per_layer = need / g.n_layers;
        const int rows = (g.n_q_heads + 2 * g.n_kv_heads) * g.head_dim;
        for (int l = 0; l < g.n_layers; ++l) {
            LayerW &w = m->layers[l];
            __nv_bfloat16 *dst = (__nv_bfloat16 *)((char *)m->arena + per_layer * l);
            mg::k_repack_qkv<<<rows, 128>>>((const __nv_bfloat16 *)w.wq, (const __nv_bfloat16 *)w.wk, (const __nv_bfloat16 *)w.wv, dst,
                                            g.n_q_heads, g.n_kv_heads, g.head_dim, g.d_model);
            CK(cudaGetLastError());
            w.wqkv_perm = dst;
        }
        CK(cudaDeviceSynchronize());
    }
    m->finalized = true;
    return ADA_OK;
}

void ada_model_destroy(ada_model *m) { delete m; }

size_t ada_session_scratch_bytes(const ada_model *m, int32_t batch, int32_t max_seq_len, int32_t max_early) {
    if (!m || batch < 1 || max_seq_len < 2 || max_early < 0) return 0;
    return make_layout(m->cfg, batch, max_seq_len, max_early, kHeadBlocks).total;
}

size_t ada_kv_page_bytes(const ada_model *m, int32_t page_tokens) {
    if (!m || page_tokens < 1) return 0;
    const ada_config &g = m->cfg;
    return (size_t)g.n_layers * 2 * g.n_kv_heads * page_tokens * g.head_dim * m->esz;
}

int ada_session_create(const ada_model *m, int32_t batch, int32_t max_seq_len, int32_t page_tokens, int32_t max_early,
                       void *kv_pool_dev, size_t kv_pool_bytes, void *scratch_dev, size_t scratch_bytes,
                       void *cuda_stream, ada_session **out) {
    if (!m || !out || !kv_pool_dev || !scratch_dev) return ADA_EINVAL;
    if (!m->finalized) return ADA_ESTATE;
    if (batch < 1 || batch > ADA_MAX_BATCH || max_seq_len < 2 || max_early < 0) return ADA_EINVAL;
    if (page_tokens < 16 || page_tokens > 256 || (page_tokens & (page_tokens - 1))) return ADA_EINVAL;
    if (batch * (max_early + 1) > kMaxRows) return ADA_ECAPACITY;
    if ((uintptr_t)scratch_dev % 256 || (uintptr_t)kv_pool_dev % 256) return ADA_EINVAL;
    const ada_config &g = m->cfg;
    Layout lay = make_layout(g, batch, max_seq_len, max_early, kHeadBlocks);
    if (scratch_bytes < lay.total) return ADA_ECAPACITY;
    size_t page_bytes = ada_kv_page_bytes(m, page_tokens);
    int n_pages = (int)std::min<size_t>(kv_pool_bytes / page_bytes, 1u << 30);
    if (n_pages < 1) return ADA_ECAPACITY;

    ada_session *S = new ada_session();
    S->m = m;
    S->batch = batch; S->max_seq = max_seq_len; S->page_tokens = page_tokens; S->max_early = max_early;
    S->slots = max_early + 1;
    S->rows_alloc = rows_alloc_for(g, batch, max_early);
    S->n_pages = n_pages;
    S->max_pages = (max_seq_len + 15) / 16;
    S->n_chunks = (max_seq_len + kAttnChunk - 1) / kAttnChunk;
    S->head_blocks = kHeadBlocks;
    S->stream = (cudaStream_t)cuda_stream;
    S->scratch = scratch_dev;
    S->scratch_bytes = scratch_bytes;
    char *b = (char *)scratch_dev;
    Ctx &c = S->c;
    c.d = g.d_model; c.nq = g.n_q_heads; c.nkv = g.n_kv_heads; c.hd = g.head_dim; c.dff = g.d_ff; c.vocab = g.vocab;
    c.L = g.n_layers; c.qkv_rows = (g.n_q_heads + 2 * g.n_kv_heads) * g.head_dim; c.group = g.n_q_heads / g.n_kv_heads;
    c.eps = g.rms_eps;
    c.page_tokens = page_tokens;
    c.page_shift = 0;
    while ((1 << c.page_shift) < page_tokens) c.page_shift++;
    c.kv_swz = 0;
    if (g.dtype == ADA_DTYPE_BF16) c.kv_swz = (g.head_dim / 8) % 8 == 0 ? 7 : (g.head_dim / 8) % 4 == 0 ? 3 : (g.head_dim / 8) % 2 == 0 ? 1 : 0;
    c.max_pages = S->max_pages; c.max_seq = max_seq_len; c.slots = S->slots; c.n_chunks = S->n_chunks;
    c.st = (DevState *)(b + lay.st); c.rt = (RowTable *)(b + lay.rt); c.fill = (int32_t *)(b + lay.fill);
    c.tokens = (int32_t *)(b + lay.tokens); c.page_table = (int32_t *)(b + lay.page_table);
    c.head_res = (HeadResult *)(b + lay.head_res); c.resid = (float *)(b + lay.resid); c.xn = (float *)(b + lay.xn);
    c.qkv = (float *)(b + lay.qkv); c.q = (float *)(b + lay.q); c.attn_out = (float *)(b + lay.attn_out);
    c.gu = (float *)(b + lay.gu); c.hact = (float *)(b + lay.hact); c.rope_cs = (float *)(b + lay.rope_cs);
    c.attn_part = (float *)(b + lay.attn_part); c.head_part = (float *)(b + lay.head_part);
    c.logit_stage = (float *)(b + lay.logit_stage); c.capture = nullptr; c.head_log = (float *)(b + lay.head_log);
    c.kv_pool = kv_pool_dev;
    S->t_out = (float *)(b + lay.t_out);

    auto fail = [&](int code) { ada_session_destroy(S); return code; };
#define CKS(expr)                                                                   \
    do {                                                                            \
        cudaError_t e__ = (expr);                                                   \
        if (e__ != cudaSuccess) {                                                   \
            g_cuda_err = std::string(#expr) + ": " + cudaGetErrorString(e__);       \
            return fail(ADA_ECUDA);                                                 \
        }                                                                           \
    } while (0)
    CKS(cudaMallocHost((void **)&S->pinned, 256));
    CKS(cudaEventCreate(&S->ev0));
    CKS(cudaEventCreate(&S->ev1));
    CKS(cudaMemsetAsync(scratch_dev, 0, lay.total, S->stream));
    DevState hs;
    memset(&hs, 0, sizeof(hs));
    hs.batch = batch; hs.slots = S->slots; hs.n_layers = g.n_layers; hs.max_seq = max_seq_len;
    CKS(cudaMemcpyAsync(c.st, &hs, offsetof(DevState, len), cudaMemcpyHostToDevice, S->stream));
    CKS(cudaMemsetAsync(kv_pool_dev, 0, (size_t)n_pages * page_bytes, S->stream));   // masked cache rows must hold finite numbers
    CKS(cudaStreamSynchronize(S->stream));
#undef CKS
    {
        int rc = setup_persistent(S, lay);
        if (rc) return fail(rc);
    }
    // dense prompt pass: bf16 models of the shapes above on a device with fifth-generation tensor cores
    S->dense_ok = false;
    if (model_fits_persistent(g)) {
        int dev = 0, major = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (major == 10 &&
            cudaFuncSetAttribute(dg::k_dense_gemm<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dg::DSMEM_BYTES) == cudaSuccess &&
            cudaFuncSetAttribute(dg::k_dense_gemm<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dg::DSMEM_BYTES) == cudaSuccess) {
            S->dense_ok = true;
            S->pf_hi = (__nv_bfloat16 *)(b + lay.pf_hi);
            S->pf_lo = (__nv_bfloat16 *)(b + lay.pf_lo);
            S->pf_err = (int *)(b + lay.pf_err);
            S->pf_part = (float *)(b + lay.pf_part);
            S->pf_part_bytes = kDenseSplitMax * sizeof(float) * dg::BM * (size_t)g.d_model;
        } else cudaGetLastError();
    }
    // free list: pages are handed out from the back, in a scrambled order so that the page-table
    // indirection is always exercised
    S->free_pages.resize(n_pages);
    for (int i = 0; i < n_pages; ++i) S->free_pages[i] = (int)(((long long)i * 7919 + 13) % n_pages);
    {
        std::vector<char> seen(n_pages, 0);
        bool perm = true;
        for (int p : S->free_pages) { if (seen[p]) perm = false; seen[p] = 1; }
        if (!perm) for (int i = 0; i < n_pages; ++i) S->free_pages[i] = n_pages - 1 - i;
    }
    S->seq_pages.resize(batch);
    S->h_len.assign(batch, 0); S->h_prompt.assign(batch, 0); S->h_reported.assign(batch, 0);
    S->prefilled.assign(batch, 0);
    S->finished.assign(batch, 0);
    S->eos_tok.assign(batch, -1);
    *out = S;
    return ADA_OK;
}

void ada_session_destroy(ada_session *S) {
    if (!S) return;
    if (S->pinned) cudaFreeHost(S->pinned);
    if (S->ev0) cudaEventDestroy(S->ev0);
    if (S->ev1) cudaEventDestroy(S->ev1);
    for (cudaEvent_t e : S->prof_ev) cudaEventDestroy(e);
    delete S;
}

int ada_session_reset(ada_session *S, int32_t seq) {
    if (!S || seq >= S->batch) return ADA_EINVAL;
    for (int s = 0; s < S->batch; ++s) {
        if (seq >= 0 && s != seq) continue;
        for (int p : S->seq_pages[s]) S->free_pages.push_back(p);
        S->seq_pages[s].clear();
        S->prefilled[s] = 0;
        S->finished[s] = 0;
        S->h_len[s] = S->h_prompt[s] = S->h_reported[s] = 0;
    }
    return ADA_OK;
}

int ada_prefill(ada_session *S, int32_t seq, const int32_t *prompt_host, int32_t n_prompt) {
    if (!S || !prompt_host || seq < 0 || seq >= S->batch || n_prompt < 1) return ADA_EINVAL;
    const ada_model *m = S->m;
    const ada_config &g = m->cfg;
    if (n_prompt + 2 > S->max_seq) return ADA_ECAPACITY;
    for (int i = 0; i < n_prompt; ++i) if (prompt_host[i] < 0 || prompt_host[i] >= g.vocab) return ADA_EINVAL;
    int rc = ada_session_reset(S, seq);
    if (rc) return rc;
    if ((rc = ensure_pages(S, seq, n_prompt + 1))) return rc;
    CK(cudaMemcpyAsync(S->c.tokens + (size_t)seq * S->max_seq, prompt_host, sizeof(int32_t) * n_prompt,
                       cudaMemcpyHostToDevice, S->stream));
    if (seq == 0 && S->capture_dev) {
        int32_t zero = 0;
        CK(cudaMemcpyAsync(&S->c.st->capture_n, &zero, sizeof(int32_t), cudaMemcpyHostToDevice, S->stream));
    }
    // Prompts of some length take the dense pass: blocks of 128 positions, every weight matrix streamed once per block
    // through the tcgen05 GEMM, the other operations by the per-operation kernels.
    const bool dense = S->dense_ok && S->prefill_dense && n_prompt >= 32;
    if (!dense && S->mega && S->path == 1) {
        // prompt passes of eight positions through the persistent kernel
        mg::k_prefill_arm<<<1, 32, 0, S->stream>>>(S->c, seq, n_prompt);
        CK(cudaGetLastError());
        if ((rc = run_persistent(S, nullptr, 0, true, seq, seq + 1, false))) return rc;
        S->prefilled[seq] = 1;
        S->h_prompt[seq] = n_prompt;
        S->h_len[seq] = n_prompt + 1;
        S->h_reported[seq] = 0;
        return ADA_OK;
    }
    const int chunk = dense ? dg::BM : std::min(std::min(S->rows_alloc, kMaxRows), 64);
    if (dense) CK(cudaMemsetAsync(S->pf_err, 0, sizeof(int), S->stream));
    struct DenseScope {   // dense_on only while this prefill issues its passes
        ada_session *S;
        ~DenseScope() { S->dense_on = false; }
    } scope{S};
    S->dense_on = dense;
    for (int p0 = 0; p0 < n_prompt; p0 += chunk) {
        const int n = std::min(chunk, n_prompt - p0);
        const int last = p0 + n == n_prompt;
        S->cur_rows = n;
        if (g.dtype == ADA_DTYPE_BF16)
            k_prefill_begin<__nv_bfloat16><<<1, 256, 0, S->stream>>>(S->c, (const __nv_bfloat16 *)m->tok_embed, g.rope_base, seq, p0, n);
        else
            k_prefill_begin<float><<<1, 256, 0, S->stream>>>(S->c, (const float *)m->tok_embed, g.rope_base, seq, p0, n);
        CK(cudaGetLastError());
        for (int l = 0; l < g.n_layers; ++l) if ((rc = run_layer(S, l, n))) return rc;
        if (last && (rc = run_head(S, 0, SEL_LAST, n))) return rc;
        k_prefill_end<<<1, 32, 0, S->stream>>>(S->c, seq, p0 + n, last, n_prompt);
        CK(cudaGetLastError());
        if (last && seq == 0 && (rc = capture_rows(S, n - 1))) return rc;
    }
    if (dense) {
        CK(cudaMemcpyAsync(S->pinned, S->pf_err, sizeof(int), cudaMemcpyDeviceToHost, S->stream));
        CK(cudaStreamSynchronize(S->stream));
        if (S->pinned[0] != 0) {
            g_cuda_err = "dense prompt pass: a bounded device-side wait expired";
            return ADA_ETIMEOUT;
        }
    }
    CK(cudaStreamSynchronize(S->stream));
    S->prefilled[seq] = 1;
    S->h_prompt[seq] = n_prompt;
    S->h_len[seq] = n_prompt + 1;
    S->h_reported[seq] = 0;
    return ADA_OK;
}

int ada_plain_decode(ada_session *S, int32_t n_tokens, int32_t eos_id, int32_t *out_host, ada_stats *stats) {
    if (!S) return ADA_EINVAL;
    return decode(S, n_tokens, 2.0f, nullptr, 0, 0, eos_id, out_host, stats);
}

int ada_adaptive_decode(ada_session *S, int32_t n_tokens, float threshold, const int32_t *exit_layers,
                        int32_t n_exit_layers, int32_t max_early, int32_t eos_id, int32_t *out_host, ada_stats *stats) {
    if (!S || n_exit_layers < 0 || (n_exit_layers > 0 && !exit_layers)) return ADA_EINVAL;
    return decode(S, n_tokens, threshold, exit_layers, n_exit_layers, max_early, eos_id, out_host, stats);
}

int ada_sampling_decode(ada_session *S, int32_t n_tokens, float temperature, float threshold, const int32_t *exit_layers,
                        int32_t n_exit_layers, int32_t max_early, int32_t eos_id, const float *uniforms_host, int32_t first_pos,
                        int32_t n_pos, int32_t *out_host, ada_stats *stats) {
    if (!S || n_exit_layers < 0 || (n_exit_layers > 0 && !exit_layers) || !uniforms_host) return ADA_EINVAL;
    if (!(temperature > 0.0f) || first_pos < 0 || n_pos < 1 || first_pos + (int64_t)n_pos > S->max_seq) return ADA_EINVAL;
    if (n_exit_layers > mg::SAMPLE_NU - 3) return ADA_ECAPACITY;
    if (!(S->mega && S->path == 1) || S->m->cfg.vocab > mg::DRAW_MAX_VOCAB) return ADA_EUNSUPPORTED;
    // every position the call may draw, test or resample must have its random numbers
    for (int s = 0; s < S->batch; ++s) {
        if (!S->prefilled[s]) return ADA_ESTATE;
        if (S->finished[s]) continue;
        if (S->h_len[s] < first_pos || S->h_prompt[s] + S->h_reported[s] + n_tokens + 1 > first_pos + n_pos) return ADA_EINVAL;
    }
    float *dev = const_cast<float *>(S->margs.uniforms);
    for (int s = 0; s < S->batch; ++s)
        CK(cudaMemcpyAsync(dev + ((size_t)s * S->max_seq + first_pos) * mg::SAMPLE_NU, uniforms_host + (size_t)s * n_pos * mg::SAMPLE_NU,
                           sizeof(float) * (size_t)n_pos * mg::SAMPLE_NU, cudaMemcpyHostToDevice, S->stream));
    S->sampling = true;
    S->inv_temp = 1.0f / temperature;
    const int rc = decode(S, n_tokens, threshold, exit_layers, n_exit_layers, max_early, eos_id, out_host, stats);
    S->sampling = false;
    return rc;
}

int ada_debug_set_wait_limit(ada_session *S, uint64_t ns) {
    if (!S || ns < 1) return ADA_EINVAL;
    S->wait_ns = ns;
    return ADA_OK;
}

int ada_debug_capture_logits(ada_session *S, float *dev_buf, int32_t max_tokens) {
    if (!S || (dev_buf && max_tokens < 1)) return ADA_EINVAL;
    S->capture_dev = dev_buf;
    S->capture_cap = dev_buf ? max_tokens : 0;
    S->c.capture = dev_buf;
    int32_t v[2] = {S->capture_cap, 0};
    CK(cudaMemcpyAsync(&S->c.st->capture_cap, v, sizeof(v), cudaMemcpyHostToDevice, S->stream));
    CK(cudaStreamSynchronize(S->stream));
    return ADA_OK;
}

int ada_debug_logits_captured(ada_session *S, int32_t *n_out) {
    if (!S || !n_out) return ADA_EINVAL;
    CK(cudaMemcpyAsync(n_out, &S->c.st->capture_n, sizeof(int32_t), cudaMemcpyDeviceToHost, S->stream));
    CK(cudaStreamSynchronize(S->stream));
    return ADA_OK;
}

int ada_debug_capture_heads(ada_session *S, float *host_buf, int32_t max_evals, int32_t *n_out) {
    if (!S || (host_buf && max_evals < 1)) return ADA_EINVAL;
    S->head_log_host = host_buf;
    S->head_log_cap = host_buf ? std::min(max_evals, kHeadLogCap) : 0;
    S->head_log_n_out = n_out;
    return ADA_OK;
}

int ada_debug_set_exit_tape(ada_session *S, const uint8_t *tape_host, int32_t n) {
    if (!S || n < 0 || n > kMaxTape || (n > 0 && !tape_host)) return ADA_EINVAL;
    S->tape.assign(tape_host, tape_host + n);
    return ADA_OK;
}

int ada_debug_get_state(ada_session *S, int32_t seq, int32_t *len_out, int32_t *fill_out) {
    if (!S || seq < 0 || seq >= S->batch) return ADA_EINVAL;
    if (len_out) CK(cudaMemcpyAsync(len_out, &S->c.st->len[seq], sizeof(int32_t), cudaMemcpyDeviceToHost, S->stream));
    if (fill_out)
        CK(cudaMemcpyAsync(fill_out, S->c.fill + (size_t)seq * S->m->cfg.n_layers, sizeof(int32_t) * S->m->cfg.n_layers,
                           cudaMemcpyDeviceToHost, S->stream));
    CK(cudaStreamSynchronize(S->stream));
    return ADA_OK;
}

int ada_debug_read_kv(ada_session *S, int32_t seq, int32_t which, int32_t layer0, int32_t pos, float *host_out) {
    if (!S || !host_out || seq < 0 || seq >= S->batch || which < 0 || which > 1) return ADA_EINVAL;
    const ada_config &g = S->m->cfg;
    if (layer0 < 0 || layer0 >= g.n_layers || pos < 0) return ADA_EINVAL;
    int pi = pos / S->page_tokens;
    if (pi >= (int)S->seq_pages[seq].size()) return ADA_EINVAL;
    const int page = S->seq_pages[seq][pi], t = pos % S->page_tokens;
    const size_t esz = S->m->esz;
    std::vector<unsigned char> tmp((size_t)g.head_dim * esz);
    for (int h = 0; h < g.n_kv_heads; ++h) {
        size_t idx = ((((size_t)page * g.n_layers + layer0) * 2 + which) * g.n_kv_heads + h) *
                         ((size_t)S->page_tokens * g.head_dim) + (size_t)t * g.head_dim;
        CK(cudaMemcpy(tmp.data(), (const char *)S->c.kv_pool + idx * esz, tmp.size(), cudaMemcpyDeviceToHost));
        for (int i = 0; i < g.head_dim; ++i) {
            float f;
            if (esz == 4) memcpy(&f, tmp.data() + 4 * i, 4);
            else {   // bf16 rows are stored with their 16-byte chunks xor-swizzled by the position
                const int j = (((i >> 3) ^ (pos & S->c.kv_swz)) << 3) | (i & 7);
                uint32_t b = ((uint32_t)tmp[2 * j] | ((uint32_t)tmp[2 * j + 1] << 8)) << 16;
                memcpy(&f, &b, 4);
            }
            host_out[h * g.head_dim + i] = f;
        }
    }
    return ADA_OK;
}

int ada_debug_profile(ada_session *S, int32_t on) {
    if (!S) return ADA_EINVAL;
    CK(cudaStreamSynchronize(S->stream));
    if (on && !S->prof) {
        for (int i = 0; i < ADA_PROF_CLASSES; ++i) { S->prof_ms[i] = 0; S->prof_bytes[i] = 0; S->prof_launches[i] = 0; }
        S->prof_rec.clear();
    }
    if (!on && S->prof) prof_collect(S);
    S->prof = on != 0;
    return ADA_OK;
}

int ada_debug_profile_read(ada_session *S, double *ms_out, int64_t *launches_out, double *bytes_out) {
    if (!S || !ms_out || !launches_out || !bytes_out) return ADA_EINVAL;
    CK(cudaStreamSynchronize(S->stream));
    prof_collect(S);
    for (int i = 0; i < ADA_PROF_CLASSES; ++i) {
        ms_out[i] = S->prof_ms[i]; launches_out[i] = S->prof_launches[i]; bytes_out[i] = S->prof_bytes[i];
    }
    return ADA_OK;
}

int ada_debug_set_path(ada_session *S, int32_t path) {
    if (!S || path < 0 || path > 1) return ADA_EINVAL;
    if (path == 1 && !S->mega) return ADA_EUNSUPPORTED;
    S->path = path;
    return ADA_OK;
}

int ada_debug_get_path(ada_session *S, int32_t *path_out) {
    if (!S || !path_out) return ADA_EINVAL;
    *path_out = S->path;
    return ADA_OK;
}

int ada_debug_set_prefill(ada_session *S, int32_t dense) {
    if (!S || dense < 0 || dense > 1) return ADA_EINVAL;
    if (dense && !S->dense_ok) return ADA_EUNSUPPORTED;
    S->prefill_dense = dense != 0;
    return ADA_OK;
}

int ada_debug_set_launch_steps(ada_session *S, int32_t steps) {
    if (!S || steps < 1) return ADA_EINVAL;
    S->steps_per_launch = steps;
    return ADA_OK;
}

int ada_debug_trace(ada_session *S, uint64_t *dev_buf, uint32_t *count_dev, uint32_t cap_events, int32_t step0, int32_t step1) {
    if (!S || !S->mega) return ADA_EUNSUPPORTED;
    if (dev_buf && (!count_dev || cap_events < 1 || step0 < 0 || step1 < step0)) return ADA_EINVAL;
    S->margs.trace = st::Trace{(unsigned long long *)dev_buf, count_dev, dev_buf ? cap_events : 0};
    S->margs.trace_step0 = dev_buf ? step0 : 0;
    S->margs.trace_step1 = dev_buf ? step1 : 0;
    return ADA_OK;
}

int ada_debug_gemm_plan(int32_t N, int32_t K, int32_t mode, int32_t grid, int32_t cta, int32_t split, int32_t *out9) {
    if (!out9 || N < 1 || K < 64 || K % 64 || mode < 0 || mode > 1 || grid < 1 || cta < 0 || cta >= grid) return ADA_EINVAL;
    if (mode == 1 && (N % 2 || (N / 2) % 16)) return ADA_EINVAL;
    st::Gemm g;
    memset(&g, 0, sizeof(g));
    g.N = N; g.K = K; g.pair = mode == 1 ? 2 : 1; g.half = mode == 1 ? N / 2 : 0; g.ctas = grid;
    static unsigned long long dummy;
    g.part = split ? &dummy : nullptr;   // only tested for null by the plan
    const st::Plan p = st::make_plan(g, cta, grid);
    const int32_t v[9] = {p.split, p.t0, p.t1, p.n, p.ta, p.tb, p.s0_own_k0, p.s0_pub_k1, p.sl_k1};
    memcpy(out9, v, sizeof(v));
    return ADA_OK;
}

size_t ada_debug_gemm_work_bytes(int32_t K) {
    if (K < 64) return 0;
    return st::xfrag_bytes(K) + 512 + kPartBytesPerCta * kPartMaxGrid + 256;
}

int ada_debug_gemm(const void *W_dev, int32_t N, int32_t K, int32_t mode, const float *X_dev, int32_t cols, void *work_dev,
                   size_t work_bytes, float *Y_dev, int32_t ldy, int32_t repeat, void *cuda_stream, float *ms_out) {
    if (!W_dev || !X_dev || !work_dev || !Y_dev || N < 1 || K < 64 || K % 64 || cols < 1 || cols > st::MAX_COLS) return ADA_EINVAL;
    if (mode < 0 || mode > 1 || repeat < 1) return ADA_EINVAL;
    if (mode == 1 && (N % 2 || (N / 2) % 16)) return ADA_EINVAL;
    if ((uintptr_t)W_dev % 16 || (uintptr_t)work_dev % 256 || ldy < (mode == 1 ? N / 2 : N)) return ADA_EINVAL;
    if (work_bytes < ada_debug_gemm_work_bytes(K)) return ADA_ECAPACITY;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int dev = 0, sms = 0;
    CK(cudaGetDevice(&dev));
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CK(cudaFuncSetAttribute(k_gemm_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st::SMEM_BYTES));
    int *err = (int *)((char *)work_dev + st::xfrag_bytes(K));
    CUtensorMap *dmap = (CUtensorMap *)((char *)work_dev + st::xfrag_bytes(K) + 256);
    CUtensorMap hmap;
    int rc = make_weight_map(&hmap, W_dev, N, K);
    if (rc) return rc;
    CK(cudaMemsetAsync(err, 0, sizeof(int), stream));
    CK(cudaMemcpyAsync(dmap, &hmap, sizeof(hmap), cudaMemcpyHostToDevice, stream));
    CK(cudaStreamSynchronize(stream));   // hmap lives on this stack frame
    k_xfrag_pack<<<(K + 255) / 256, 256, 0, stream>>>(X_dev, K, cols, (__nv_bfloat16 *)work_dev);
    CK(cudaGetLastError());
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0));
    CK(cudaEventCreate(&e1));
    cudaEventRecord(e0, stream);
    unsigned long long *part = (unsigned long long *)((char *)work_dev + st::xfrag_bytes(K) + 512);
    if (sms > kPartMaxGrid || repeat != 1) part = nullptr;
    else CK(cudaMemsetAsync(part, 0, kPartBytesPerCta * (size_t)sms, stream));
    k_gemm_probe<<<sms, st::THREADS, st::SMEM_BYTES, stream>>>(dmap, N, K, mode, (const uint4 *)work_dev, Y_dev, ldy, cols, repeat, err, part);
    cudaError_t le = cudaGetLastError();
    cudaEventRecord(e1, stream);
    int herr = 0;
    cudaError_t ce = le == cudaSuccess ? cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, stream) : le;
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
    float ms = 0.f;
    if (ce == cudaSuccess) ce = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    CK(ce);
    if (ms_out) *ms_out = ms;
    return herr ? ADA_ETIMEOUT : ADA_OK;
}

size_t ada_debug_dense_gemm_work_bytes(int32_t K) {
    if (K < 64) return 0;
    return 2 * (size_t)dg::BM * K * sizeof(__nv_bfloat16) + 256;
}

int ada_debug_dense_gemm(const void *W_dev, int32_t N, int32_t K, const float *X_dev, int32_t rows, float *Y_dev, int32_t ldy,
                         int32_t accumulate, void *work_dev, size_t work_bytes, void *cuda_stream) {
    if (!W_dev || !X_dev || !Y_dev || !work_dev || N < 1 || K < 64 || K % 64 || rows < 1 || rows > dg::BM || ldy < N) return ADA_EINVAL;
    if ((uintptr_t)W_dev % 16 || (uintptr_t)work_dev % 256 || (uintptr_t)Y_dev % 16 || ldy % 4) return ADA_EINVAL;
    if (work_bytes < ada_debug_dense_gemm_work_bytes(K)) return ADA_ECAPACITY;
    int dev = 0, major = 0;
    CK(cudaGetDevice(&dev));
    CK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return ADA_EUNSUPPORTED;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    __nv_bfloat16 *hi = (__nv_bfloat16 *)work_dev, *lo = hi + (size_t)dg::BM * K;
    int *err = (int *)(lo + (size_t)dg::BM * K);
    CUtensorMap mhi, mlo, mw;
    int rc;
    if ((rc = make_map_2d(&mhi, hi, dg::BM, K, dg::BM)) || (rc = make_map_2d(&mlo, lo, dg::BM, K, dg::BM)) || (rc = make_map_2d(&mw, W_dev, N, K, dg::BN)))
        return rc;
    CK(cudaFuncSetAttribute(dg::k_dense_gemm<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dg::DSMEM_BYTES));
    CK(cudaFuncSetAttribute(dg::k_dense_gemm<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dg::DSMEM_BYTES));
    CK(cudaMemsetAsync(err, 0, sizeof(int), stream));
    dg::k_split_rows<<<dg::BM, 256, 0, stream>>>(X_dev, K, rows, K, hi, lo);
    CK(cudaGetLastError());
    const int grid = (N + dg::BN - 1) / dg::BN;
    if (accumulate) dg::k_dense_gemm<1><<<grid, dg::DTHREADS, dg::DSMEM_BYTES, stream>>>(mhi, mlo, mw, Y_dev, ldy, rows, N, K, 0, err);
    else dg::k_dense_gemm<0><<<grid, dg::DTHREADS, dg::DSMEM_BYTES, stream>>>(mhi, mlo, mw, Y_dev, ldy, rows, N, K, 0, err);
    CK(cudaGetLastError());
    int herr = 0;
    CK(cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, stream));
    CK(cudaStreamSynchronize(stream));
    return herr ? ADA_ETIMEOUT : ADA_OK;
}

// ---- streaming GEMM without caller scratch ---------------------------------------------------------

#define ADA_NOALLOC_MAX_K 16384
// Fragment-layout activations for K <= ADA_NOALLOC_MAX_K, then the error word (at +0) and the tensor
// map (at +256) in a 512-byte tail.  Lives in every GPU context that loads this library.
static __device__ __align__(256) unsigned char g_noalloc_scratch[(ADA_NOALLOC_MAX_K / st::KC) * st::X_STAGE + 512];

int ada_gemm_noalloc(const void *W_dev, int32_t N, int32_t K, int32_t mode, const float *X_dev, int32_t cols, float *Y_dev,
                     int32_t ldy, void *cuda_stream) {
    if (!W_dev || !X_dev || !Y_dev || N < 1 || K < 64 || K % 64 || cols < 1 || cols > st::MAX_COLS) return ADA_EINVAL;
    if (mode < 0 || mode > 1) return ADA_EINVAL;
    if (mode == 1 && (N % 2 || (N / 2) % 16)) return ADA_EINVAL;
    if ((uintptr_t)W_dev % 16 || ldy < (mode == 1 ? N / 2 : N)) return ADA_EINVAL;
    if (K > ADA_NOALLOC_MAX_K) {
        g_cuda_err = "ada_gemm_noalloc: K exceeds the built-in scratch (ADA_NOALLOC_MAX_K = 16384)";
        return ADA_ECAPACITY;
    }
    // Once per device: the address of the scratch array in that device's memory.  The array's name
    // in host code is only a handle; kernels must be given the address looked up here.
    static unsigned char *scratch_of_device[64] = {nullptr};
    static int sms_of_device[64] = {0};
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ADA_EUNSUPPORTED;
    if (!scratch_of_device[dev]) {
        unsigned char *ptr = nullptr;
        CK(cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch));
        CK(cudaDeviceGetAttribute(&sms_of_device[dev], cudaDevAttrMultiProcessorCount, dev));
        CK(cudaFuncSetAttribute(k_gemm_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st::SMEM_BYTES));
        scratch_of_device[dev] = ptr;
    }
    unsigned char *base = scratch_of_device[dev];
    const size_t xb = st::xfrag_bytes(K);
    int *err = (int *)(base + xb);
    CUtensorMap *dmap = (CUtensorMap *)(base + xb + 256);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    CUtensorMap hmap;
    int rc = make_weight_map(&hmap, W_dev, N, K);
    if (rc) return rc;
    CK(cudaMemsetAsync(err, 0, sizeof(int), stream));   // the one word that must start at zero
    CK(cudaMemcpyAsync(dmap, &hmap, sizeof(hmap), cudaMemcpyHostToDevice, stream));
    CK(cudaStreamSynchronize(stream));   // hmap lives on this stack frame
    k_xfrag_pack<<<(K + 255) / 256, 256, 0, stream>>>(X_dev, K, cols, (__nv_bfloat16 *)base);
    CK(cudaGetLastError());
    k_gemm_probe<<<sms_of_device[dev], st::THREADS, st::SMEM_BYTES, stream>>>(dmap, N, K, mode, (const uint4 *)base, Y_dev, ldy, cols, 1, err, nullptr);
    CK(cudaGetLastError());
    int herr = 0;
    CK(cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, stream));
    CK(cudaStreamSynchronize(stream));
    return herr ? ADA_ETIMEOUT : ADA_OK;
}

}  // extern "C"
