// Dense GEMM for the prompt pass ("KV cache <- LM(x)", first line of Algorithm 1) on the fifth-generation
// tensor cores of sm_100a: tcgen05.mma with the accumulator in tensor memory, operands staged in shared
// memory by TMA.
//
// A prompt block of up to 128 positions goes through a weight matrix in one product
//     Y[m][n] (+)= sum_k X[m][k] W[n][k],   m < 128 positions, n < N weight rows,
// so a weight byte fetched from HBM is used for 128 tokens instead of the eight of a decode pass: here the
// contraction really is dense, and the tensor cores are what it belongs on.  X arrives as two bf16
// matrices, a high part and a low part (x = hi + lo, as everywhere in this library: fp32 activations
// lose nothing), both multiplied into the same fp32 accumulator.
//
// One CTA computes a tile of 128 positions x 128 weight rows.  Warp 0 is the TMA producer (one k block of
// 64 elements per stage: the 128-byte-swizzled tiles of X.hi, X.lo and W), warp 1 allocates the tensor
// memory and issues the MMAs (one elected thread; UMMA shape M = 128, N = 128, K = 16, both operands
// K-major), warps 2..5 read the accumulator back (tcgen05.ld, 32 lanes per warp) and write it out.
// Every wait is bounded; on expiry an error word is set, the roles leave their loops, the tensor
// memory is released and the kernel ends.
#pragma once

#include "kernels.cuh"
#include "stream.cuh"

namespace ada {
namespace dg {

using namespace st;

constexpr int BM = 128;     // positions per tile (UMMA M)
constexpr int BN = 128;     // weight rows per tile (UMMA N)
constexpr int BK = 64;      // k elements per stage: one 128-byte swizzle row
constexpr int STAGES = 4;
constexpr int DTHREADS = 192;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = 2 * A_BYTES + B_BYTES;
// The tensor core adds into its fp32 accumulator with truncation, so the error of one accumulator grows in
// proportion to the products added (1e-3 absolute at K = 14336 with sums of size 10).  The k blocks therefore
// take NACC accumulators in turn, which the epilogue adds up in registers (round to nearest).
constexpr int NACC = 4;
constexpr int TMEM_COLS = NACC * BN;   // fp32 accumulator columns (a power of two >= 32)
constexpr unsigned long long DENSE_WAIT_NS = 2000000000ull;

struct DSmem {   // must start on a 1024-byte boundary (swizzle pattern)
    alignas(1024) unsigned char stage[STAGES][STAGE_BYTES];   // [X.hi 128 x 64 | X.lo 128 x 64 | W 128 x 64], rows of 128 B
    alignas(8) unsigned long long full[STAGES], empty[STAGES], acc_full;
    uint32_t tmem_base;
    int abort;
};
constexpr size_t DSMEM_BYTES = sizeof(DSmem) + 1024;
static_assert(STAGE_BYTES % 1024 == 0 && A_BYTES % 1024 == 0, "operand tiles must start on 1024-byte boundaries");
static_assert(DSMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a block may use");

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1, unsigned long long *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(s32(dst)),
                 "l"(map), "r"(c0), "r"(c1), "r"(s32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled (the layout
// a TMA box of 64 bf16 x rows leaves): start address / 16 in bits 0-13, leading byte offset / 16 in bits
// 16-29 (1: not used by swizzled K-major tiles), stride byte offset / 16 in bits 32-45 (1024 bytes from one
// group of eight rows to the next), descriptor version 1 in bits 46-47, swizzle mode 2 (128 bytes) in bits 61-63.
__device__ __forceinline__ unsigned long long smem_desc(uint32_t saddr) {
    return (unsigned long long)((saddr >> 4) & 0x3fffu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulator (bits 4-5 = 1), bf16 A and B (bits 7-9 and 10-12 = 1),
// both K-major (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void umma(uint32_t d_tmem, unsigned long long adesc, unsigned long long bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate)
        : "memory");
}
// the mbarrier is arrived on once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(unsigned long long *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(bar)) : "memory");
}

struct DWait {
    DSmem *sm;
    int *err;
};
__device__ __forceinline__ bool dwait(const DWait &w, unsigned long long *bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 0) {
            if (*(volatile int *)&w.sm->abort) return false;
            const unsigned long long t = gtime();
            if (t0 == 0) t0 = t;
            else if (t - t0 > DENSE_WAIT_NS) {
                atomicCAS(w.err, 0, ERR_TIMEOUT_MBAR);
                *(volatile int *)&w.sm->abort = 1;
                return false;
            }
        }
    }
}

// EPI 0: Y[m][n] = acc.  EPI 1: Y[m][n] += acc (every element has one writer).  Rows m >= rows are not written.
// gridDim.y > 1 splits the depth: block row y multiplies its share of the k blocks and writes (EPI 0) to
// Y + y * split_stride; k_dense_reduce then adds the shares in a fixed order.
// mapXhi / mapXlo: 2-D maps over the bf16 matrices [128][K] (box 64 x 128); mapW: over W [N][K] (box 64 x 128);
// all 128-byte swizzled, zero fill outside.  K a multiple of 64.
template <int EPI>
__global__ void __launch_bounds__(DTHREADS, 1)
k_dense_gemm(const __grid_constant__ CUtensorMap mapXhi, const __grid_constant__ CUtensorMap mapXlo,
             const __grid_constant__ CUtensorMap mapW, float *__restrict__ Y, int ldy, int rows, int N, int K, size_t split_stride, int *err) {
    extern __shared__ unsigned char dsm_raw[];
    DSmem *sm = reinterpret_cast<DSmem *>(dsm_raw + ((1024u - (s32(dsm_raw) & 1023u)) & 1023u));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, nkb_all = K / BK;
    const int kb_begin = (int)((long long)nkb_all * blockIdx.y / gridDim.y), kb_end = (int)((long long)nkb_all * (blockIdx.y + 1) / gridDim.y);
    const int nkb = kb_end - kb_begin;
    Y += (size_t)blockIdx.y * split_stride;
    const DWait W{sm, err};
    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(&sm->full[i], 1); mbar_init(&sm->empty[i], 1); }
        mbar_init(&sm->acc_full, 1);
        sm->abort = 0;
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncthreads();
    if (warp == 1) {   // tensor memory for the accumulator: allocated, and later released, by this one warp
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(&sm->tmem_base)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *(volatile uint32_t *)&sm->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % STAGES;
                if (!dwait(W, &sm->empty[s], ((kb / STAGES) & 1) ^ 1)) break;
                mbar_expect_tx(&sm->full[s], (uint32_t)STAGE_BYTES);
                tma_load_2d(sm->stage[s], &mapXhi, (kb_begin + kb) * BK, 0, &sm->full[s]);
                tma_load_2d(sm->stage[s] + A_BYTES, &mapXlo, (kb_begin + kb) * BK, 0, &sm->full[s]);
                tma_load_2d(sm->stage[s] + 2 * A_BYTES, &mapW, (kb_begin + kb) * BK, n0, &sm->full[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % STAGES;
                ok = dwait(W, &sm->full[s], (kb / STAGES) & 1);
                if (!ok) break;
                tc_fence_after();
                const unsigned long long ahi = smem_desc(s32(sm->stage[s])), alo = smem_desc(s32(sm->stage[s] + A_BYTES)),
                                         b = smem_desc(s32(sm->stage[s] + 2 * A_BYTES));
                const uint32_t acc = tmem + (uint32_t)((kb % NACC) * BN);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {   // 32 bytes further along the swizzled row per K = 16 step
                    umma(acc, ahi + 2 * k, b + 2 * k, (kb >= NACC || k != 0) ? 1u : 0u);
                    umma(acc, alo + 2 * k, b + 2 * k, 1u);
                }
                umma_commit(&sm->empty[s]);   // the stage is free once these MMAs have read it
            }
            umma_commit(&sm->acc_full);
        }
    } else {
        // epilogue: warp w may read the 32 lanes 32 (w % 4) .. of the tensor memory; lane = position within the block
        const int q = warp & 3, m = q * 32 + lane;
        const bool ok = dwait(W, &sm->acc_full, 0);
        tc_fence_after();
        if (ok) {
            const int nacc = min(NACC, nkb);
#pragma unroll
            for (int c0 = 0; c0 < BN; c0 += 16) {
                uint32_t v[16];
#pragma unroll
                for (int a = 0; a < NACC; ++a) {
                    if (a >= nacc) continue;
                    uint32_t t[16];
                    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                                 : "=r"(t[0]), "=r"(t[1]), "=r"(t[2]), "=r"(t[3]), "=r"(t[4]), "=r"(t[5]), "=r"(t[6]), "=r"(t[7]), "=r"(t[8]),
                                   "=r"(t[9]), "=r"(t[10]), "=r"(t[11]), "=r"(t[12]), "=r"(t[13]), "=r"(t[14]), "=r"(t[15])
                                 : "r"(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * BN + c0)));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = a == 0 ? t[j] : __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(t[j]));
                }
                if (m < rows) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        const int n = n0 + c0 + j;
                        if (n + 3 < N) {
                            float4 *p = reinterpret_cast<float4 *>(Y + (size_t)m * ldy + n);
                            float4 o = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                            if (EPI == 1) { const float4 r = *p; o.x += r.x; o.y += r.y; o.z += r.z; o.w += r.w; }
                            *p = o;
                        } else {
                            for (int e = 0; e < 4; ++e)
                                if (n + e < N) {
                                    float *p = Y + (size_t)m * ldy + n + e;
                                    *p = (EPI == 1 ? *p : 0.f) + __uint_as_float(v[j + e]);
                                }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*(volatile int *)&sm->abort) {   // copies already issued may still be landing: give them time before the block's memory goes
        const unsigned long long t0 = gtime();
        while (gtime() - t0 < 200000ull) __nanosleep(1000);
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// Y[m][n] = (or +=) sum over the `splits` shares of a depth-split product, added in index order.
__global__ void k_dense_reduce(const float *__restrict__ part, size_t split_stride, int splits, float *__restrict__ Y, int ldy, int rows, int N, int add) {
    const int m = blockIdx.y;
    if (m >= rows) return;
    for (int n = (blockIdx.x * blockDim.x + threadIdx.x) * 4; n < N; n += gridDim.x * blockDim.x * 4) {
        float4 a = *reinterpret_cast<const float4 *>(part + (size_t)m * N + n);
        for (int s = 1; s < splits; ++s) {
            const float4 b = *reinterpret_cast<const float4 *>(part + s * split_stride + (size_t)m * N + n);
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        float4 *y = reinterpret_cast<float4 *>(Y + (size_t)m * ldy + n);
        if (add) { const float4 r = *y; a.x += r.x; a.y += r.y; a.z += r.z; a.w += r.w; }
        *y = a;
    }
}

// RMSNorm and split in one pass: x = resid[r] / sqrt(mean(resid[r]^2) + eps) * g -> high and low parts.  One block
// (256 threads) per row; rows >= `rows` are zero.
__global__ void __launch_bounds__(256) k_norm_split_rows(const float *__restrict__ X, int rows, int K, const __nv_bfloat16 *__restrict__ gain,
                                                         float eps, __nv_bfloat16 *__restrict__ hi, __nv_bfloat16 *__restrict__ lo) {
    const int r = blockIdx.x;
    __shared__ float red[8];
    float rstd = 0.f;
    if (r < rows) {
        const float *x = X + (size_t)r * K;
        float ss = 0.f;
        for (int i = threadIdx.x; i < K; i += 256) ss = fmaf(x[i], x[i], ss);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += red[w];
        rstd = 1.0f / sqrtf(tot / K + eps);
    }
    for (int k = threadIdx.x; k < K; k += 256) {
        const float v = r < rows ? X[(size_t)r * K + k] * rstd * __bfloat162float(gain[k]) : 0.f;
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[(size_t)r * K + k] = h;
        lo[(size_t)r * K + k] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

// fp32 rows X[r][ldx] (r < rows) -> the two bf16 matrices [128][K] the dense GEMM reads: high part and low part
// (x = hi + lo); rows >= `rows` are zero.  One block per row.
__global__ void k_split_rows(const float *__restrict__ X, int ldx, int rows, int K, __nv_bfloat16 *__restrict__ hi, __nv_bfloat16 *__restrict__ lo) {
    const int r = blockIdx.x;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const float v = r < rows ? X[(size_t)r * ldx + k] : 0.f;
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[(size_t)r * K + k] = h;
        lo[(size_t)r * K + k] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
}

// Causal attention of a block of prompt rows on the tensor cores (mma.sync m16n8k16, bf16 cache).  One warp owns
// one 16-row query tile: 16 / GROUP consecutive prompt positions x the GROUP q heads of one kv head; a block of
// four warps shares the K and V rows of 64 cache positions at a time, copied into shared memory exactly as the
// cache stores them (16-byte chunks xor-swizzled by position: conflict-free for ldmatrix).  Queries are rotated
// already (k_rope_kv); they are scaled and split into bf16 high / low parts in registers, the probabilities
// likewise, so nothing but the cache itself is rounded to bf16.  Online softmax in position order; the context
// is not split, the result goes straight to attn_out.
template <int HD, int GROUP>
__global__ void __launch_bounds__(128) k_pf_attn_mma(Ctx c, int layer, int rows) {
    constexpr int KSQ = HD / 16, NT = HD / 8, PPW = 16 / GROUP, TILE = 64;
    __shared__ __align__(128) unsigned char sK[TILE * HD * 2], sV[TILE * HD * 2];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, kvh = blockIdx.y;
    const int r_blk = blockIdx.x * 4 * PPW, r_w = r_blk + warp * PPW;   // first row of the block / of this warp
    const int seq = c.rt->seq[0], pos0 = c.rt->pos[0];                   // rows of a prompt block: consecutive positions of one sequence
    const int pos_blk_max = pos0 + min(r_blk + 4 * PPW, rows) - 1;
    const __nv_bfloat16 *pool = reinterpret_cast<const __nv_bfloat16 *>(c.kv_pool);
    const float scale = rsqrtf((float)HD);
    // ---- this lane's parts of the query fragments: rows lane/4 and lane/4 + 8 of the tile
    int lim[2];
    uint32_t ah[KSQ][4], al[KSQ][4];
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
        const int row = (lane >> 2) + 8 * rh, r = r_w + row / GROUP, g = row % GROUP;
        const bool live = r < rows;
        lim[rh] = live ? pos0 + r : -1;
        const float *q = c.q + ((size_t)min(r, rows - 1) * c.nq + kvh * GROUP + g) * HD;
#pragma unroll
        for (int ks = 0; ks < KSQ; ++ks)
#pragma unroll
            for (int kh = 0; kh < 2; ++kh) {
                const float2 v = *reinterpret_cast<const float2 *>(q + ks * 16 + kh * 8 + 2 * (lane & 3));
                const float y0 = live ? v.x * scale : 0.f, y1 = live ? v.y * scale : 0.f;
                const __nv_bfloat162 h = __floats2bfloat162_rn(y0, y1);
                const __nv_bfloat162 l = __floats2bfloat162_rn(y0 - __low2float(h), y1 - __high2float(h));
                ah[ks][rh + 2 * kh] = *reinterpret_cast<const uint32_t *>(&h);
                al[ks][rh + 2 * kh] = *reinterpret_cast<const uint32_t *>(&l);
            }
    }
    const int lim_w = r_w < rows ? pos0 + min(r_w + PPW, rows) - 1 : -1;   // last position any row of this warp sees (the same in every lane)
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[nt][i] = 0.f;
    for (int t0 = 0; t0 <= pos_blk_max; t0 += TILE) {
        __syncthreads();   // the previous tile has been used
        for (int i = threadIdx.x; i < TILE * (HD / 8); i += 128) {
            const int t = i / (HD / 8), ch = i - t * (HD / 8), p = t0 + t;
            uint4 kq = make_uint4(0, 0, 0, 0), vq = kq;
            if (p <= pos_blk_max) {
                kq = *reinterpret_cast<const uint4 *>(pool + kv_index(c, seq, layer, 0, kvh, p) + ch * 8);
                vq = *reinterpret_cast<const uint4 *>(pool + kv_index(c, seq, layer, 1, kvh, p) + ch * 8);
            }
            *reinterpret_cast<uint4 *>(sK + (size_t)t * HD * 2 + ch * 16) = kq;
            *reinterpret_cast<uint4 *>(sV + (size_t)t * HD * 2 + ch * 16) = vq;
        }
        __syncthreads();
        for (int sl = 0; sl < TILE / 16; ++sl) {
            const int p0 = t0 + 16 * sl;
            if (p0 > lim_w) break;   // nothing further in this tile is visible to this warp (uniform per warp)
            // ---- scores of the 16 positions p0 .. p0 + 15
            float sh[2][4], sl_[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) { sh[nt][i] = 0.f; sl_[nt][i] = 0.f; }
            const int id = lane >> 3;
            {
                const int pl = 16 * sl + (lane & 7) + 8 * (id >> 1);
                const unsigned char *krow = sK + pl * (HD * 2);
#pragma unroll
                for (int ks = 0; ks < KSQ; ++ks) {
                    uint32_t kf[4];
                    ldmatrix_x4(kf, krow + ((((2 * ks) | (id & 1)) ^ (pl & 7)) << 4));
                    mma16816(sh[0], ah[ks], kf[0], kf[1]);
                    mma16816(sh[1], ah[ks], kf[2], kf[3]);
                    mma16816(sl_[0], al[ks], kf[0], kf[1]);
                    mma16816(sl_[1], al[ks], kf[2], kf[3]);
                }
            }
            float s[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int pos = p0 + 8 * nt + 2 * (lane & 3) + (i & 1);
                    s[nt][i] = pos <= lim[i >> 1] ? sh[nt][i] + sl_[nt][i] : -INFINITY;
                }
            // ---- online softmax
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
                const __nv_bfloat162 h0 = __floats2bfloat162_rn(p[0], p[1]), h1 = __floats2bfloat162_rn(p[2], p[3]);
                const __nv_bfloat162 l0 = __floats2bfloat162_rn(p[0] - __low2float(h0), p[1] - __high2float(h0));
                const __nv_bfloat162 l1 = __floats2bfloat162_rn(p[2] - __low2float(h1), p[3] - __high2float(h1));
                ph[rh] = *reinterpret_cast<const uint32_t *>(&h0);
                ph[2 + rh] = *reinterpret_cast<const uint32_t *>(&h1);
                plo[rh] = *reinterpret_cast<const uint32_t *>(&l0);
                plo[2 + rh] = *reinterpret_cast<const uint32_t *>(&l1);
            }
            // ---- o += P V
            {
                const int pl = 16 * sl + (lane & 7) + 8 * (id & 1);
                const unsigned char *vrow = sV + pl * (HD * 2);
#pragma unroll
                for (int np = 0; np < NT / 2; ++np) {
                    uint32_t vf[4];
                    ldmatrix_x4_trans(vf, vrow + ((((2 * np) | (id >> 1)) ^ (pl & 7)) << 4));
                    mma16816(o[2 * np], ph, vf[0], vf[1]);
                    mma16816(o[2 * np + 1], ph, vf[2], vf[3]);
                    mma16816(o[2 * np], plo, vf[0], vf[1]);
                    mma16816(o[2 * np + 1], plo, vf[2], vf[3]);
                }
            }
        }
    }
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
        l_run[rh] += __shfl_xor_sync(0xffffffffu, l_run[rh], 1);
        l_run[rh] += __shfl_xor_sync(0xffffffffu, l_run[rh], 2);
        const int row = (lane >> 2) + 8 * rh, r = r_w + row / GROUP, g = row % GROUP;
        if (r < rows) {
            float *out = c.attn_out + ((size_t)r * c.nq + kvh * GROUP + g) * HD;
            const float inv = 1.0f / l_run[rh];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                *reinterpret_cast<float2 *>(out + nt * 8 + 2 * (lane & 3)) = make_float2(o[nt][2 * rh] * inv, o[nt][2 * rh + 1] * inv);
        }
    }
}

}  // namespace dg
}  // namespace ada
