// Stand-alone launch of the weight-streaming GEMM phase (test and measurement hook): the same
// producer / consumer code as the persistent decode kernel, one phase, plain epilogues.
#pragma once

#include "stream.cuh"

namespace ada {

// fp32 activations X[cols][K] -> fragment layout (high/low bf16 split).
__global__ void k_xfrag_pack(const float *__restrict__ X, int K, int cols, __nv_bfloat16 *__restrict__ out) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    for (int c = 0; c < st::MAX_COLS; ++c) st::xfrag_store(out, k, c, c < cols ? X[(size_t)c * K + k] : 0.f);
}

// mode 0: Y[col][n] = sum_k W[n][k] X[col][k]                       (N rows)
// mode 1: Y[col][n] = silu(g) * u, g = W[n].X, u = W[half + n].X     (half = N/2 rows of each)
__global__ void __launch_bounds__(st::THREADS, 1)
k_gemm_probe(const CUtensorMap *__restrict__ W, int N, int K, int mode, const uint4 *__restrict__ X, float *__restrict__ Y,
             int ldy, int cols, int repeat, int *err, unsigned long long *part) {
    extern __shared__ unsigned char smem_raw[];
    st::Smem *sm = st::smem_base(smem_raw);
    st::smem_init(sm);
    __syncthreads();
    st::Shared S{sm, err, st::Trace{nullptr, nullptr, 0}, 0, st::WAIT_NS_DEFAULT};
    st::Gemm g;
    g.W = W; g.X = X; g.N = N; g.K = K; g.pair = mode == 1 ? 2 : 1; g.half = mode == 1 ? N / 2 : 0;
    g.ctas = st::balanced_ctas(g.tiles(), gridDim.x);
    g.cp0 = 0; g.ncp = (cols + 1) / 2;
    // tiles split between CTAs need a grid-wide meeting between products: only for a single product
    g.part = repeat == 1 ? part : nullptr; g.phase_id = 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    st::Rings r{0, 0};
    if (warp == st::CONS_WARPS) {
        const uint64_t pol = st::policy_evict_first();
        for (int it = 0; it < repeat; ++it) st::gemm_produce_w(S, g, cta, G, r, pol);
    } else if (warp == st::CONS_WARPS + 1) {
        const uint64_t pol = st::policy_evict_last();
        for (int it = 0; it < repeat; ++it) st::gemm_produce_x(S, g, cta, G, r, pol);
    } else {
        for (int it = 0; it < repeat; ++it) {
            if (mode == 0) {
                st::gemm_consume<1>(S, g, cta, G, r, [&](int tile, float (&d)[1][4]) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, c = 2 * (lane & 3) + (i & 1);
                        if (n < N && c < cols) Y[(size_t)c * ldy + n] = d[0][i];
                    }
                });
            } else {
                st::gemm_consume<2>(S, g, cta, G, r, [&](int tile, float (&d)[2][4]) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int n = tile * 16 + (lane >> 2) + (i >> 1) * 8, c = 2 * (lane & 3) + (i & 1);
                        const float gv = d[0][i], u = d[1][i];
                        if (n < g.half && c < cols) Y[(size_t)c * ldy + n] = gv / (1.0f + expf(-gv)) * u;
                    }
                });
            }
        }
    }
    st::settle_on_abort(S);
}

}  // namespace ada
