// Weight-streaming primitives of the persistent decode kernel (sm_100a).
//
// The decode step is bound by HBM bandwidth: every weight byte is read once per pass and used
// for at most eight tokens.  The pieces here keep the memory pipe full:
//   * weights reach shared memory through TMA tensor copies (cp.async.bulk.tensor, one 16 KB box
//     of 16 rows x 512 k per instruction, 128-byte swizzled) issued by a dedicated producer warp
//     into a ring of stages guarded by mbarriers; the producer runs ahead of the consumers across
//     phase boundaries, because the weight sequence of a CTA does not depend on activations.
//     (Sixteen 1 KB untiled bulk copies per stage reached only 3.6 TB/s on B200: the copy engine
//     spends about 40 ns per request whatever its size, so requests have to be large.)
//   * activations arrive through a second, small ring in the register layout the tensor-core
//     instruction wants, already split into a bf16 high part and a bf16 low part, so that
//     fp32 activations lose nothing: W.x = W.hi(x) + W.lo(x) with fp32 accumulation;
//   * eight consumer warps multiply with mma.sync m16n8k16 (weights are the 16-row operand, the
//     up-to-eight tokens are the 8 columns).  The tensor cores are used as a cheap way to issue
//     the multiply-adds; the bound stays the memory system.
//   * all CTAs of the persistent grid meet at a counter-based grid barrier between phases.
// Every wait is bounded: on expiry an error word is set and all later waits fall through.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ada {
namespace st {

constexpr int KC = 512;                          // k elements per stage
constexpr int KSTEPS = KC / 16;                  // mma k-steps per stage
constexpr int TILE_N = 16;                       // weight rows per stage (mma M)
constexpr int KG = KC / 64;                      // 64-element (128-byte) k groups per stage
constexpr int W_STAGE = TILE_N * KC * 2;         // 16384: [k group][row][128 B, 16-byte chunks xor-swizzled by row%8]
constexpr int X_STAGE = KSTEPS * 32 * 16;        // 16384: [column pair][k-step][8 slots][b0.hi b1.hi b0.lo b1.lo]
#ifndef ADA_NW
#define ADA_NW 9
#endif
#ifndef ADA_NX
#define ADA_NX 3
#endif
constexpr int NW = ADA_NW;                       // weight stages in flight per CTA
constexpr int NX = ADA_NX;                       // activation / KV stages
constexpr int CONS_WARPS = 8;
constexpr int CONS_THREADS = CONS_WARPS * 32;
constexpr int THREADS = CONS_THREADS + 64;       // + weight producer warp + activation producer warp
constexpr int MAX_COLS = 8;                      // tokens per pass (mma N)
constexpr int RED_BYTES = CONS_WARPS * 2 * 128 * 4;  // cross-warp reduction scratch (two tiles per warp)
constexpr int SCRATCH_BYTES = 33 * 1024;         // consumers' scratch: GEMM reduction, or the attention phase's buffers

constexpr int ERR_TIMEOUT_MBAR = 1, ERR_TIMEOUT_GRID = 2;
constexpr unsigned long long WAIT_NS_DEFAULT = 2000000000ull;   // a single wait gives up after two seconds unless told otherwise
constexpr unsigned long long SHORT_LIMIT_NS = 1000000ull;       // a limit below this is checked at every poll, not every 64th or 128th

struct Smem {                                    // must start on a 1024-byte boundary (swizzle pattern)
    alignas(1024) unsigned char w[NW][W_STAGE];
    alignas(128) unsigned char x[NX][X_STAGE];
    alignas(16) unsigned char scratch[SCRATCH_BYTES];
    alignas(16) float vec[64];                    // per-column scalars (rstd, ...)
    alignas(8) unsigned long long w_full[NW], w_empty[NW], x_full[NX], x_empty[NX];
    alignas(16) int desc[3][32];                  // per-role copy of the step descriptor (persistent decode kernel)
    int abort;
    int bcast[8];
    unsigned trace_n;
    unsigned vec_seq;                             // phase for which vec[] holds the normalisation factors (see vec_wait)
};

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t s32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(s32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long gtime() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// Bulk copy global -> shared of `bytes` (multiple of 16; both addresses 16-byte aligned), completing
// on `bar` with the byte count.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, unsigned long long *bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(s32(dst)),
        "l"(src), "r"(bytes), "r"(s32(bar)), "l"(pol)
        : "memory");
}
// TMA tensor copy of one box of a rank-3 map (coordinates innermost first) into shared memory.
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2, unsigned long long *bar,
                                            uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(
            s32(dst)),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(s32(bar)), "l"(pol)
        : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(s32(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&a)[4], const void *p) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(s32(p)));
}
// d += a (16x16, row) * b (16x8, col), bf16 inputs, fp32 accumulation.
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, %0;" ::"n"(CONS_THREADS) : "memory"); }

__device__ __forceinline__ uint32_t ld_acquire(const unsigned *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned *p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---------------------------------------------------------------- bounded waits

// Optional event trace (test hook): records (globaltimer ns, code) pairs while `tr_on` is set.
// Every CTA writes its own region of the buffer, so that recording costs a shared-memory counter
// and one store.
struct Trace {
    unsigned long long *buf;   // [grid][cap][2], or nullptr
    unsigned *count;           // [grid]
    unsigned cap;              // events per CTA
};

struct Shared {            // what every role needs to wait safely
    Smem *sm;
    int *err;              // global error word (0 = fine)
    Trace tr;
    int tr_on;             // this block is currently tracing
    unsigned long long wait_ns;   // a single wait gives up after this many nanoseconds
};

constexpr int EV_PHASE_BEGIN = 1, EV_X0 = 2, EV_W0 = 3, EV_MAIN_END = 4, EV_EPI_END = 5, EV_WP_BEGIN = 6, EV_WP_END = 7,
              EV_ITEM = 8, EV_COMBINE = 9, EV_ARRIVE = 10, EV_ATT = 14;

__device__ __forceinline__ void trace(const Shared &S, int ev, int arg) {
    if (S.tr_on && S.tr.buf) {
        const unsigned i = atomicAdd(&S.sm->trace_n, 1u);
        if (i < S.tr.cap) {
            unsigned long long *e = S.tr.buf + 2 * ((size_t)blockIdx.x * S.tr.cap + i);
            e[0] = gtime();
            e[1] = ((unsigned long long)blockIdx.x << 32) | ((unsigned long long)(arg & 0xffff) << 8) | (unsigned)ev;
            S.tr.count[blockIdx.x] = i + 1;
        }
    }
}

__device__ __forceinline__ bool aborted(const Shared &S) { return *(volatile int *)&S.sm->abort != 0; }

__device__ __noinline__ void raise_error(const Shared &S, int code) {
    atomicCAS(S.err, 0, code);
    *(volatile int *)&S.sm->abort = 1;
}

// Wait for an mbarrier phase.  Once an error is raised (here or anywhere in the grid) every wait
// falls through at once: the roles then run to the end of their loops on whatever data is there,
// so that no warp is left behind at a block-level barrier, and the kernel ends.
__device__ __forceinline__ void mbar_wait(const Shared &S, unsigned long long *bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return;
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try(bar, parity)) return;
        if ((it & 127u) == 0 || S.wait_ns < SHORT_LIMIT_NS) {
            if (aborted(S)) return;
            if (*(volatile int *)S.err != 0) { *(volatile int *)&S.sm->abort = 1; return; }
            unsigned long long t = gtime();
            if (t0 == 0) t0 = t;
            else if (t - t0 > S.wait_ns) { raise_error(S, ERR_TIMEOUT_MBAR); return; }
        }
    }
}

// Epilogue operands are fetched while the weights stream, by 4-byte asynchronous copies into a
// per-warp corner of the scratch area (word k of lane l at [k][l]) rather than into registers: a
// value held in a register across the main loop ties up the register file, and wherever the
// compiler has to move it the warp first waits for the load.  Each lane reads back only its own
// words, after cp_async_wait_all().  The k-split reduction uses the first 8 KB of the scratch area.
constexpr int STASH_OFFSET = 8192, STASH_WORDS = 8;
static_assert(STASH_OFFSET + CONS_WARPS * STASH_WORDS * 32 * 4 <= SCRATCH_BYTES, "stash exceeds the scratch area");
__device__ __forceinline__ uint32_t *stash_of(Smem *sm) {
    return reinterpret_cast<uint32_t *>(sm->scratch + STASH_OFFSET) + (threadIdx.x >> 5) * (STASH_WORDS * 32) + (threadIdx.x & 31);
}
__device__ __forceinline__ void cp_async4(uint32_t *dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// element n of a bf16 vector from the aligned 32-bit word that holds it
__device__ __forceinline__ float bf16_of_word(uint32_t w, int n) { return __uint_as_float((n & 1) ? (w & 0xffff0000u) : (w << 16)); }

// The consumers wait until the activation producer warp has left the per-column factors of phase
// `seq` in vec[] (it computes them while the first weight stages are being multiplied).
__device__ __forceinline__ void vec_wait(const Shared &S, unsigned seq) {
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (*(volatile unsigned *)&S.sm->vec_seq == seq) return;
        if ((it & 127u) == 127u || S.wait_ns < SHORT_LIMIT_NS) {
            if (aborted(S)) return;
            if (*(volatile int *)S.err != 0) { *(volatile int *)&S.sm->abort = 1; return; }
            unsigned long long t = gtime();
            if (t0 == 0) t0 = t;
            else if (t - t0 > S.wait_ns) { raise_error(S, ERR_TIMEOUT_MBAR); return; }
        }
    }
}

// Grid barrier on a monotonically increasing counter: arrive once per CTA, wait for `target`.
__device__ __forceinline__ void grid_arrive(unsigned *ctr) {
    // the release of the reduction orders this thread's earlier writes, and through the block-level
    // barrier before it those of the whole CTA; a separate fence before it only adds its latency
    fence_proxy_async();
    red_release_add(ctr, 1u);
}
__device__ __forceinline__ void grid_wait(const Shared &S, const unsigned *ctr, unsigned target) {
    unsigned long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (ld_acquire(ctr) >= target) return;
        if ((it & 63u) == 0 || S.wait_ns < SHORT_LIMIT_NS) {
            if (aborted(S)) return;
            if (*(volatile int *)S.err != 0) { *(volatile int *)&S.sm->abort = 1; return; }
            unsigned long long t = gtime();
            if (t0 == 0) t0 = t;
            else if (t - t0 > S.wait_ns) { raise_error(S, ERR_TIMEOUT_GRID); return; }
        }
        __nanosleep(32);
    }
}

// ---------------------------------------------------------------- activation layout

// Activations for a GEMM of depth K live in global memory as ceil(K/KC) blocks of X_STAGE bytes.
// A block holds four sub-blocks of 4 KB, one per pair of token columns; in sub-block p, k-step s,
// slot j (0..7) holds 16 bytes: the mma B fragment (b0, b1) of the bf16 high parts, then of the
// bf16 low parts, for token column 2 p + j/4 and k = 16 s + 2 (j%4) + {0,1} (+8 for b1).  Lane l of
// a warp reads slot l%8 of sub-block l/8.  A pass that carries few tokens fetches only the
// sub-blocks of the column pairs in use: activations go through the same copy engine as the
// weights, and for a CTA holding two weight tiles a full block per chunk would be half as many
// bytes again as the weights.
__device__ __forceinline__ size_t xfrag_index(int k, int col) {   // index in 2-byte units of the high part
    const int chunk = k / KC, ks = (k % KC) >> 4, kk = k & 15;
    const int slot = (col & 1) * 4 + ((kk & 7) >> 1);
    return (((((size_t)chunk * 4 + (col >> 1)) * KSTEPS + ks) * 8 + slot) << 3) + ((kk >> 3) << 1) + (kk & 1);
}
__device__ __forceinline__ void xfrag_store(__nv_bfloat16 *X, int k, int col, float v) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    const size_t i = xfrag_index(k, col);
    X[i] = hi;
    X[i + 4] = lo;
}
__host__ __device__ inline size_t xfrag_bytes(int K) { return (size_t)((K + KC - 1) / KC) * X_STAGE; }

// ---------------------------------------------------------------- GEMM phase

// One GEMM as seen by the whole grid: Y[n][col] = sum_k W[n][k] X[k][col].
//   pair == 1: N rows, tiles of 16 rows (the last may be ragged).
//   pair == 2: W holds two stacked matrices of `half` rows each (gate over up); a tile is rows
//              [16 t, 16 t + 16) of both, and the epilogue sees both accumulators.
// The weights are described by a rank-3 tensor map over the row-major [N][K] matrix, dimensions
// (64 elements, N rows, K/64 groups) with strides (2 B, 2K B, 128 B) and box (64, 16, 8): one box
// is a stage.  Rows past N and k groups past K read as zeros.  K must be a multiple of 64.
struct Gemm {
    const CUtensorMap *W;
    const CUtensorMap *W2 = nullptr;   // pair == 2 only: map of the second matrix when the two are separate tensors (null: stacked in W)
    const uint4 *X;
    int N, K, pair, half;
    int ctas;   // CTAs 0 .. ctas-1 share the tiles (see balanced_ctas); 0 = the whole grid
    // Exchange area for tiles split between two CTAs (null: whole tiles only): [grid][CONS_WARPS][8][32]
    // words of 8 bytes, each a partial sum (low half) tagged with the phase that wrote it (high half).
    // A word is written and read by one 8-byte access, so a reader that sees the tag sees the sum:
    // no fence is needed on either side (a fence in the middle of the stream stalls the publishing
    // warp, and with it the whole ring, for microseconds).  phase_id is unique per GEMM of a launch
    // and never 0; the area is zeroed before each launch.
    unsigned long long *part;
    unsigned phase_id;
    int cp0, ncp;   // column pairs cp0 .. cp0+ncp-1 of the activations are fetched
    __device__ __forceinline__ void columns(unsigned mask) {   // the pairs spanning the columns set in `mask`
        if (mask == 0) { cp0 = 0; ncp = 1; return; }
        cp0 = (__ffs(mask) - 1) >> 1;
        ncp = ((31 - __clz(mask)) >> 1) - cp0 + 1;
    }
    // k chunks whose activations share one 16 KB stage: 4 for one column pair, 2 for two, else 1.  (The
    // ring holds three stages; with one chunk per stage a CTA that owns two weight tiles would wait
    // for an activation copy every 96 KB of weights.)
    __device__ __forceinline__ int xchunks() const { return ncp == 1 ? 4 : ncp == 2 ? 2 : 1; }
    __host__ __device__ __forceinline__ int tiles() const { return pair == 2 ? half / TILE_N : (N + TILE_N - 1) / TILE_N; }
};

struct Rings { uint32_t wi, xi; };   // stage counters of one role (slot = i % N, parity = (i / N) & 1)

__host__ __device__ __forceinline__ void cta_tile_range(int T, int cta, int G, int &t0, int &t1) {
    if (cta >= G) { t0 = t1 = 0; return; }
    t0 = (int)((long long)T * cta / G);
    t1 = (int)((long long)T * (cta + 1) / G);
}
// ---------------------------------------------------------------- unit-balanced split of a GEMM
// With whole tiles some CTAs stream one tile more than the others (7 against 6 in the 8B gate-up
// GEMM) and the phase lasts as long as they do.  When g.part is set the work is instead measured in
// units of (tile, k chunk): CTA c takes the units [U c / C, U (c + 1) / C) of the tile-major order,
// so every CTA streams the same number of stages (+- one).  A tile cut by a CTA boundary is
// computed in two parts.  The CTA with its chunks from 0 (the head part, [0, kb)) meets them early
// in its k loop and publishes its partial sums as soon as they are complete; the CTA with the later
// chunks (the tail part, [ka, nch)) finishes them at the end of its loop, adds the published part
// (own + published, the published k-splits in index order: the sum does not depend on timing) and
// runs the epilogue.  All tiles of a CTA, partial ones included, form one group that shares every
// activation chunk; when the head part ends before the tail part begins they take turns in slot 0.
// GEMMs with fewer units per CTA than chunks per tile, or more tiles per CTA than consumer warps,
// keep whole tiles.  The plan is a function of the GEMM's shape and the grid only.
struct Plan {
    int split;       // 0: whole tiles [t0, t1) in groups of CONS_WARPS
    int t0, t1;
    // split: one group of n slots; slot s holds tile ta + s, except that
    int n, ta, tb;
    int s0_own_k0;   //   slot 0 multiplies its own tile from chunk s0_own_k0 on (0: a whole tile),
    int s0_pub_k1;   //   and before that the chunks below s0_pub_k1 of tile tb, to publish (0: none);
    int sl_k1;       //   the last slot (if not slot 0) multiplies chunks below sl_k1 only, to publish (nch: a whole tile)
};
__host__ __device__ __forceinline__ Plan make_plan(const Gemm &g, int cta, int G) {
    Plan p;
    p.split = 0;
    p.t0 = p.t1 = p.n = p.ta = p.tb = p.s0_own_k0 = p.s0_pub_k1 = 0;
    const int C = g.ctas > 0 ? g.ctas : G, T = g.tiles(), nch = (g.K + KC - 1) / KC;
    p.sl_k1 = nch;
    if (cta < 0 || cta >= C) return p;
    // 32-bit arithmetic throughout (a 64-bit division costs hundreds of cycles); GEMMs whose unit
    // count times the CTA count does not fit keep whole tiles
    const unsigned U = (unsigned)T * (unsigned)nch;
    const bool fits = (unsigned long long)T * nch * (unsigned)(C + 1) < 0x7fffffffull;
    const unsigned L = (U + C - 1) / C;      // most units of one CTA; a run of L units touches <= (L + nch - 2) / nch + 1 tiles
    if (!g.part || !fits || U / C < (unsigned)nch || (L + nch - 2) / nch + 1 > (unsigned)CONS_WARPS) {
        cta_tile_range(T, cta, C, p.t0, p.t1);
        return p;
    }
    p.split = 1;
    const unsigned u0 = U * (unsigned)cta / C, u1 = U * (unsigned)(cta + 1) / C;
    p.ta = (int)(u0 / nch);
    p.tb = (int)((u1 - 1) / nch);
    const int ka = (int)(u0 - p.ta * nch), kb = (int)((u1 - 1) - p.tb * nch) + 1;
    const bool has_tail = ka > 0, has_head = kb < nch;
    const bool shared = has_tail && has_head && kb <= ka;
    p.s0_own_k0 = ka;
    p.n = p.tb - p.ta + 1;
    if (shared) { p.s0_pub_k1 = kb; p.n -= 1; }
    else if (has_head) p.sl_k1 = kb;
    return p;
}
// the tile slot s of a split plan multiplies at chunk kc (-1: none)
__host__ __device__ __forceinline__ int plan_tile(const Plan &p, int s, int kc) {
    if (s == 0) return kc < p.s0_pub_k1 ? p.tb : (kc >= p.s0_own_k0 ? p.ta : -1);
    if (s == p.n - 1 && kc >= p.sl_k1) return -1;
    return p.ta + s;
}
// the k-splits of a group of ng slots
__host__ __device__ __forceinline__ int group_ks(int ng) {
    int TS = 1;
    while (TS < ng) TS <<= 1;
    return CONS_WARPS / TS;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long *p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// How many CTAs share the tiles of a GEMM: all of them.  (With its consumers attached one SM
// sustains about 45 GB/s through the ring, roughly its fair share of HBM with all 148 SMs
// streaming; giving equal tile counts to fewer CTAs was measured and lost more than the uneven
// split costs.)
__host__ __device__ inline int balanced_ctas(int T, int G) { (void)T; return G; }

// Weight producer warp: streams this CTA's tiles of the GEMM through the weight ring.
__device__ __forceinline__ void gemm_produce_w(const Shared &S, const Gemm &g, int cta, int G, Rings &r, uint64_t pol) {
    Smem *sm = S.sm;
    const int lane = threadIdx.x & 31;
    const Plan pl = make_plan(g, cta, G);
    const int nch = (g.K + KC - 1) / KC;
    if (lane == 0) trace(S, EV_WP_BEGIN, 0);
    auto stage = [&](int tile, int p, int kc) {
        const int slot = r.wi % NW;
        mbar_wait(S, &sm->w_empty[slot], ((r.wi / NW) & 1) ^ 1);
        if (lane == 0 && !aborted(S)) {
            mbar_expect_tx(&sm->w_full[slot], (uint32_t)W_STAGE);
            tma_load_3d(sm->w[slot], (p && g.W2) ? g.W2 : g.W, 0, tile * TILE_N + ((p && !g.W2) ? g.half : 0), kc * KG, &sm->w_full[slot], pol);
        }
        ++r.wi;
    };
    if (pl.split) {
        for (int kc = 0; kc < nch; ++kc)
            for (int s = 0; s < pl.n; ++s) {
                const int tile = plan_tile(pl, s, kc);
                if (tile < 0) continue;
                for (int p = 0; p < g.pair; ++p) stage(tile, p, kc);
            }
    } else {
        for (int g0 = pl.t0; g0 < pl.t1; g0 += CONS_WARPS) {
            const int ng = min(CONS_WARPS, pl.t1 - g0);
            for (int kc = 0; kc < nch; ++kc)
                for (int s = 0; s < ng; ++s)
                    for (int p = 0; p < g.pair; ++p) stage(g0 + s, p, kc);
        }
    }
    if (lane == 0) trace(S, EV_WP_END, 0);
}

// Activation producer warp: one stage per (tile group, k chunk).
// `after_first` runs once, after the first stage has been issued: work of the phase that is not
// needed before the epilogues (the normalisation factors) and must not delay the first copy.
template <class Hook>
__device__ __forceinline__ void gemm_produce_x(const Shared &S, const Gemm &g, int cta, int G, Rings &r, uint64_t pol, Hook &&after_first) {
    Smem *sm = S.sm;
    const int lane = threadIdx.x & 31;
    const Plan pl = make_plan(g, cta, G);
    const int nch = (g.K + KC - 1) / KC;
    const int XC = g.xchunks();
    const int ngroups = pl.split ? (pl.n > 0 ? 1 : 0) : (pl.t1 - pl.t0 + CONS_WARPS - 1) / CONS_WARPS;
    bool hooked = false;
    for (int gi = 0; gi < ngroups; ++gi) {
        for (int kc = 0; kc < nch; kc += XC) {
            const int nc = min(XC, nch - kc);
            const int slot = r.xi % NX;
            mbar_wait(S, &sm->x_empty[slot], ((r.xi / NX) & 1) ^ 1);
            if (lane == 0 && !aborted(S)) {
                const uint32_t bytes = (uint32_t)g.ncp * 4096u;
                mbar_expect_tx(&sm->x_full[slot], bytes * nc);
                for (int q = 0; q < nc; ++q)   // chunk kc+q: column pairs cp0.. at [q][pair - cp0] of the stage
                    bulk_g2s(sm->x[slot] + q * bytes, reinterpret_cast<const unsigned char *>(g.X) + (size_t)(kc + q) * X_STAGE + g.cp0 * 4096,
                             bytes, &sm->x_full[slot], pol);
            }
            ++r.xi;
            if (!hooked) { after_first(); hooked = true; }
        }
    }
    if (!hooked) after_first();
}
struct NoHook {
    __device__ __forceinline__ void operator()() const {}
};
__device__ __forceinline__ void gemm_produce_x(const Shared &S, const Gemm &g, int cta, int G, Rings &r, uint64_t pol) {
    gemm_produce_x(S, g, cta, G, r, pol, NoHook());
}

// The k-steps ks_id + KS_ j (j < 32 / KS_) of one full weight stage: fragment loads run PF steps
// ahead of the multiply-adds that use them.  Even j accumulate into acc[0] (high parts) and acc[2]
// (low parts), odd j into acc[1] and acc[3]: four independent accumulation chains.
template <int KS_>
__device__ __forceinline__ void stage_full(float (&acc)[4][4], const unsigned char *ws, const uint4 *xs, int ks_id, int a_hi, int a_sw) {
    constexpr int NJ = KSTEPS / KS_;
    constexpr int PF = NJ < 4 ? NJ : 4;
    uint32_t a[PF][4];
    uint4 b[PF];
#pragma unroll
    for (int j = 0; j < PF; ++j) {
        const int ks = ks_id + KS_ * j;
        ldmatrix_x4(a[j], ws + (ks >> 2) * 2048 + (((((ks & 3) << 1) | a_hi) ^ a_sw) << 4));
        b[j] = xs[ks * 8];
    }
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
        const int cur = j % PF;
        mma16816(acc[j & 1], a[cur], b[cur].x, b[cur].y);
        mma16816(acc[(j & 1) + 2], a[cur], b[cur].z, b[cur].w);
        if (j + PF < NJ) {
            const int ks = ks_id + KS_ * (j + PF);
            ldmatrix_x4(a[cur], ws + (ks >> 2) * 2048 + (((((ks & 3) << 1) | a_hi) ^ a_sw) << 4));
            b[cur] = xs[ks * 8];
        }
    }
}

// Consumer warps.  Within a group of up to eight tiles the warps are arranged as TS tile slots x
// KS k-splits (TS * KS = 8, TS the smallest power of two holding the group); a warp multiplies
// the stages of its slot whose k chunk is ks_id (mod KS).  The k-splits of a tile are summed in a
// fixed order through shared memory, then `epi(tile, acc)` runs in the slot's first warp with
//   acc[p][i]: fragment element i of matrix p: rows lane/4 (i<2) or lane/4+8, columns 2(lane%4)+(i&1).
// The arrangement depends only on the tile partition, never on which token columns are in use.
// `pre(tile)` runs in the same warp before the group's first stage (a place to start loads the epilogue will need).
template <int PAIR, class Pre, class Epi>
__device__ __forceinline__ void gemm_consume(const Shared &S, const Gemm &g, int cta, int G, Rings &r, Pre &&pre, Epi &&epi) {
    Smem *sm = S.sm;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nch = (g.K + KC - 1) / KC, XC = g.xchunks();
    bool first_group = true;
    // ldmatrix source of this lane inside a stage: row (lane%8) + 8 ((lane/8)%2), 16-byte chunk lane/16 of the k-step
    const int a_row = (lane & 7) + ((lane >> 3) & 1) * 8;
    const int a_off = a_row * 128, a_hi = lane >> 4, a_sw = a_row & 7;
    // One group of ng tile slots; slot s holds tile g0 + s.  Whole tiles: s0_own_k0 = s0_pub_k1 = 0,
    // sl_k1 = nch.  The group of a split plan: see Plan; ksp = k-splits of the CTA before (0: no tail part).
    auto group = [&](int g0, int ng, int s0_own_k0, int s0_pub_k1, int sl_k1, int ksp, bool last_group) {
        int TS = 1;
        while (TS < ng) TS <<= 1;
        const int KS = CONS_WARPS / TS;
        const int slot_id = warp % TS, ks_id = warp / TS;
        const bool mine = slot_id < ng;
        const bool pub_only = slot_id > 0 && slot_id == ng - 1 && sl_k1 < nch;
        // this warp's slot: chunks below my_pub_k1 go to the published part, chunks from my_own_k0 to its own tile
        const int my_pub_k1 = !mine ? 0 : slot_id == 0 ? s0_pub_k1 : pub_only ? sl_k1 : 0;
        const int my_own_k0 = (!mine || pub_only) ? nch : slot_id == 0 ? s0_own_k0 : 0;
        const int own_tile = (mine && !pub_only) ? g0 + slot_id : -1;
        const bool tail = own_tile >= 0 && my_own_k0 > 0;   // the head part of this tile comes from CTA cta - 1
        if (ks_id == 0 && own_tile >= 0) pre(own_tile);
        float acc[PAIR][4][4];   // [matrix][even/odd step x hi/lo][fragment]
#pragma unroll
        for (int p = 0; p < PAIR; ++p)
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[p][q][i] = 0.f;
        for (int kc = 0; kc < nch; ++kc) {
            const int ksteps = min(KC, g.K - kc * KC) >> 4;
            const int xslot = r.xi % NX;
            if (kc % XC == 0) mbar_wait(S, &sm->x_full[xslot], (r.xi / NX) & 1);
            if (threadIdx.x == 0 && kc == 0 && first_group) trace(S, EV_X0, 0);
            // this lane's column pair, if it was fetched (else any fetched pair: its column is not in use)
            const int xp = min(max((lane >> 3) - g.cp0, 0), g.ncp - 1);
            const uint4 *xs = reinterpret_cast<const uint4 *>(sm->x[xslot]) + ((kc % XC) * g.ncp + xp) * 256 + (lane & 7);
            // the k-splits of a slot take whole stages in turn, counted from the first chunk of the part
            // (chunk kc belongs to split (kc - first) mod KS): a warp then multiplies all 32 k-steps of
            // a stage, which amortises the per-stage waiting and set-up (splitting every stage among
            // the warps streamed 20-30 % slower)
            const int kbase = kc < my_pub_k1 ? 0 : my_own_k0;
            const bool my_turn = mine && ((kc - kbase) & (KS - 1)) == ks_id;
            for (int s = 0; s < ng; ++s) {
                if (s == 0 ? (kc >= s0_pub_k1 && kc < s0_own_k0) : (s == ng - 1 && kc >= sl_k1)) continue;   // no stage: outside the parts
#pragma unroll
                for (int p = 0; p < PAIR; ++p) {
                    const int wslot = r.wi % NW;
                    // Every warp waits for and releases every stage in order, although only its owner
                    // uses it.  An mbarrier tells phases apart by one parity bit: a warp that ran ahead
                    // of, or fell behind, the others by a ring would mistake one phase of a slot for
                    // another (releasing stages by their owners alone was tried: a lagging warp then
                    // waits for a refill that needs its own release).  With all eight arrivals per
                    // stage no warp is ever more than one ring away from any other.
                    mbar_wait(S, &sm->w_full[wslot], (r.wi / NW) & 1);
                    if (s == slot_id && my_turn) {
                        if (threadIdx.x == 0 && kc == 0 && first_group && p == 0) trace(S, EV_W0, 0);
                        const unsigned char *ws = sm->w[wslot] + a_off;
                        if (ksteps == KSTEPS) {   // full chunk: software-pipelined, fully unrolled
                            stage_full<1>(acc[p], ws, xs, 0, a_hi, a_sw);
                        } else {                  // short last chunk of K
                            int par = 0;
                            for (int ks = 0; ks < ksteps; ++ks) {
                                uint32_t a[4];
                                ldmatrix_x4(a, ws + (ks >> 2) * 2048 + (((((ks & 3) << 1) | a_hi) ^ a_sw) << 4));
                                const uint4 b = xs[ks * 8];
                                if (par == 0) { mma16816(acc[p][0], a, b.x, b.y); mma16816(acc[p][2], a, b.z, b.w); }
                                else { mma16816(acc[p][1], a, b.x, b.y); mma16816(acc[p][3], a, b.z, b.w); }
                                par ^= 1;
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm->w_empty[wslot]);
                    ++r.wi;
                }
            }
            if (kc % XC == XC - 1 || kc == nch - 1) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->x_empty[xslot]);
                ++r.xi;
            }
            if (kc + 1 == my_pub_k1) {
                // The head part of a split tile is complete: every k-split warp publishes its own sums
                // (no meeting inside the CTA in the middle of the stream) and starts over for the tail
                // part that may follow in this slot.
                unsigned long long *pb = g.part + (size_t)(cta * CONS_WARPS + ks_id) * 256;
#pragma unroll
                for (int p = 0; p < PAIR; ++p)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float v = (acc[p][0][i] + acc[p][1][i]) + (acc[p][2][i] + acc[p][3][i]);
                        st_relaxed_u64(pb + (p * 4 + i) * 32 + lane, ((unsigned long long)g.phase_id << 32) | __float_as_uint(v));
#pragma unroll
                        for (int q = 0; q < 4; ++q) acc[p][q][i] = 0.f;
                    }
            }
        }
        if (threadIdx.x == 0 && last_group) trace(S, EV_MAIN_END, 0);
        first_group = false;
        // fold the four partial accumulators in a fixed order: (even.hi + odd.hi) + (even.lo + odd.lo)
        float d[PAIR][4];
#pragma unroll
        for (int p = 0; p < PAIR; ++p)
#pragma unroll
            for (int i = 0; i < 4; ++i) d[p][i] = (acc[p][0][i] + acc[p][1][i]) + (acc[p][2][i] + acc[p][3][i]);
        // The head part published by CTA cta - 1, in ksp k-splits: this slot's k-split warp j fetches
        // the published splits j, j + KS, ... (all at once: one round trip) and adds them to its own
        // sums in index order; the fixed-order reduction below then covers both parts.
        if (tail) {
            unsigned long long t0 = 0;
            for (uint32_t it = 0;; ++it) {
                bool ok = true;
                float add[PAIR][4];
#pragma unroll
                for (int p = 0; p < PAIR; ++p)
#pragma unroll
                    for (int i = 0; i < 4; ++i) add[p][i] = 0.f;
                for (int q = ks_id; q < ksp; q += KS) {
                    const unsigned long long *pb = g.part + (size_t)((cta - 1) * CONS_WARPS + q) * 256;
#pragma unroll
                    for (int p = 0; p < PAIR; ++p)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const unsigned long long v = ld_relaxed_u64(pb + (p * 4 + i) * 32 + lane);
                            ok = ok && (unsigned)(v >> 32) == g.phase_id;
                            add[p][i] += __uint_as_float((unsigned)v);
                        }
                }
                if (__all_sync(0xffffffffu, ok)) {
#pragma unroll
                    for (int p = 0; p < PAIR; ++p)
#pragma unroll
                        for (int i = 0; i < 4; ++i) d[p][i] += add[p][i];
                    break;
                }
                if ((it & 15u) == 15u || S.wait_ns < SHORT_LIMIT_NS) {   // bounded like every other wait on another CTA
                    bool stop = aborted(S) || *(volatile int *)S.err != 0;
                    const unsigned long long t = gtime();
                    if (t0 == 0) t0 = t;
                    else if (t - t0 > S.wait_ns) { if (lane == 0) raise_error(S, ERR_TIMEOUT_GRID); stop = true; }
                    if (__any_sync(0xffffffffu, stop)) { *(volatile int *)&S.sm->abort = 1; break; }
                }
                __nanosleep(64);
            }
        }
        if (KS > 1) {
            float *red = reinterpret_cast<float *>(sm->scratch) + (size_t)warp * (PAIR * 128);
#pragma unroll
            for (int p = 0; p < PAIR; ++p)
#pragma unroll
                for (int i = 0; i < 4; ++i) red[(p * 4 + i) * 32 + lane] = d[p][i];
            bar_consumers();
            if (ks_id == 0) {
                for (int q = 1; q < KS; ++q) {
                    const float *o = reinterpret_cast<const float *>(sm->scratch) + (size_t)(q * TS + slot_id) * (PAIR * 128);
#pragma unroll
                    for (int p = 0; p < PAIR; ++p)
#pragma unroll
                        for (int i = 0; i < 4; ++i) d[p][i] += o[(p * 4 + i) * 32 + lane];
                }
            }
        }
        if (ks_id == 0 && own_tile >= 0) epi(own_tile, d);
        if (KS > 1) bar_consumers();
    };
    {
        const Plan pl = make_plan(g, cta, G);
        if (pl.split) {
            const int ksp = pl.s0_own_k0 > 0 ? group_ks(make_plan(g, cta - 1, G).n) : 0;
            if (pl.n > 0) group(pl.ta, pl.n, pl.s0_own_k0, pl.s0_pub_k1, pl.sl_k1, ksp, true);
        } else {
            for (int g0 = pl.t0; g0 < pl.t1; g0 += CONS_WARPS)
                group(g0, min(CONS_WARPS, pl.t1 - g0), 0, 0, nch, 0, g0 + CONS_WARPS >= pl.t1);
        }
    }
}

// The dynamic shared memory is requested SMEM_BYTES long; the structure starts at its first
// 1024-byte boundary.
constexpr size_t SMEM_BYTES = sizeof(Smem) + 1024;
static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a block may use");
__device__ __forceinline__ Smem *smem_base(unsigned char *raw) {
    const uint32_t a = s32(raw);
    return reinterpret_cast<Smem *>(raw + ((1024u - (a & 1023u)) & 1023u));
}

struct NoPre {
    __device__ __forceinline__ void operator()(int) const {}
};
template <int PAIR, class Epi>
__device__ __forceinline__ void gemm_consume(const Shared &S, const Gemm &g, int cta, int G, Rings &r, Epi &&epi) {
    gemm_consume<PAIR>(S, g, cta, G, r, NoPre(), epi);
}

// Shared-memory set-up by the whole block (call once, followed by __syncthreads()).
__device__ __forceinline__ void smem_init(Smem *sm) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < NW; ++i) { mbar_init(&sm->w_full[i], 1); mbar_init(&sm->w_empty[i], CONS_WARPS); }
        for (int i = 0; i < NX; ++i) { mbar_init(&sm->x_full[i], 1); mbar_init(&sm->x_empty[i], CONS_WARPS); }
        sm->abort = 0;
        sm->trace_n = 0;
        sm->vec_seq = 0;
        fence_mbar_init();
        fence_proxy_async();
    }
}

// After an error the producers stop issuing copies; give the ones already in flight time to land
// before the block's shared memory is released.
__device__ __forceinline__ void settle_on_abort(const Shared &S) {
    __syncthreads();
    if (!aborted(S)) return;
    const unsigned long long t0 = gtime();
    while (gtime() - t0 < 200000ull) __nanosleep(1000);
}

}  // namespace st
}  // namespace ada
