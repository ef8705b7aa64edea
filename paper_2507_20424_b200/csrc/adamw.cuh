// AdamW local step: stand-alone kernel and the distance pass with the step fused in.
#pragma once
#include "round_register.cuh"

namespace {

// ---------------------------------------------------------------- AdamW local step (fused and stand-alone)
// The ViT runs of the paper train with AdamW (lr 5e-4, weight decay 0.01).  Decoupled form:
//   x <- x (1 - lr wd);  m <- m + (1 - b1)(g - m);  v <- b2 v + (1 - b2) g^2;
//   x <- x - [lr / (1 - b1^t)] m / ( sqrt(v) / sqrt(1 - b2^t) + eps )
// The step-dependent factors are formed on the host in double and passed as floats.

struct AdamArgs {
    float *m1;   // exp_avg      [M, ld]
    float *m2;   // exp_avg_sq   [M, ld]
    const float *g;
    float decay, one_minus_b1, b2, one_minus_b2, step_size, inv_sqrt_bc2, eps;
};

__device__ __forceinline__ void adamw1(float &x, float &m1, float &m2, float g, const AdamArgs &p) {
    x = __fmul_rn(x, p.decay);
    m1 = __fmaf_rn(p.one_minus_b1, __fsub_rn(g, m1), m1);
    m2 = __fmaf_rn(p.b2, m2, __fmul_rn(p.one_minus_b2, __fmul_rn(g, g)));
    const float denom = __fmaf_rn(__fsqrt_rn(m2), p.inv_sqrt_bc2, p.eps);
    x = __fmaf_rn(-p.step_size, __fdiv_rn(m1, denom), x);
}
__device__ __forceinline__ void adamw4(float4 &x, float4 &m1, float4 &m2, float4 g, const AdamArgs &p) {
    adamw1(x.x, m1.x, m2.x, g.x, p);
    adamw1(x.y, m1.y, m2.y, g.y, p);
    adamw1(x.z, m1.z, m2.z, g.z, p);
    adamw1(x.w, m1.w, m2.w, g.w, p);
}

// Block shape of the kernels that fuse the AdamW step into the distance pass: four streams per
// row (x, both moments, g) need more registers per thread than the plain round, so the blocks
// are sized for 128 (M <= 8) or 255 (M > 8) registers and nothing spills.
template <int M>
struct AdamTuning {
    static constexpr int kThreads = 256;
    static constexpr int kBlocksPerSM = (M <= 8) ? 2 : 1;
    static constexpr int kWarps = kThreads / 32;
    static constexpr int kUnrollB = (M <= 4) ? 2 : 1;     // update pass: about 40-64 KB of loads in flight per SM
};

// Distance pass with the AdamW step applied first; leaves the same partial sums and header
// as distance_kernel, so the ordinary update pass completes the round.  Loads of G rows are
// issued together, ahead of their stores.
template <int M, int G>
__device__ __forceinline__ void adamw_distance_pass(const RoundArgs &a, const AdamArgs &p, double *s_red) {
    constexpr int T = AdamTuning<M>::kThreads;
    const long long ntiles = (a.nvec + T - 1) / T;
    float acc[M];
#pragma unroll
    for (int m = 0; m < M; ++m) acc[m] = 0.f;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const long long j = t * T + threadIdx.x;
        if (j < a.nvec) {
            float4 xv[M];
#pragma unroll
            for (int m0 = 0; m0 < M; m0 += G) {
                float4 av[G], bv[G], gv[G];
#pragma unroll
                for (int k = 0; k < G; ++k) {
                    if (m0 + k < M) {
                        const long long off = (m0 + k) * a.ld + j * 4;
                        xv[m0 + k] = ld_last_use(a.x + off);
                        av[k] = ld_last_use(p.m1 + off);
                        bv[k] = ld_last_use(p.m2 + off);
                        gv[k] = ld_last_use(p.g + off);
                    }
                }
#pragma unroll
                for (int k = 0; k < G; ++k) {
                    if (m0 + k < M) {
                        const long long off = (m0 + k) * a.ld + j * 4;
                        adamw4(xv[m0 + k], av[k], bv[k], gv[k], p);
                        st_keep(p.m1 + off, av[k]);
                        st_keep(p.m2 + off, bv[k]);
                        st_keep(a.x + off, xv[m0 + k]);
                    }
                }
            }
            const float4 ebar = shifted_mean<M>(xv);
#pragma unroll
            for (int m = 0; m < M; ++m) acc[m] = sq_acc(acc[m], deviation(xv[m], xv[0], ebar, m));
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {          // scalar tail columns
        const float inv_m = 1.0f / (float)M;
        for (long long i = a.nvec * 4; i < a.d; ++i) {
            float xs[M];
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const long long off = m * a.ld + i;
                float xi = a.x[off], ai = p.m1[off], bi = p.m2[off];
                adamw1(xi, ai, bi, p.g[off], p);
                p.m1[off] = ai;
                p.m2[off] = bi;
                a.x[off] = xi;
                xs[m] = xi;
            }
            float esum = 0.f;
#pragma unroll
            for (int m = 1; m < M; ++m) { xs[m] = __fsub_rn(xs[m], xs[0]); esum = __fadd_rn(esum, xs[m]); }
            const float ebar = __fmul_rn(esum, inv_m);
            acc[0] = __fmaf_rn(ebar, ebar, acc[0]);
#pragma unroll
            for (int m = 1; m < M; ++m) { float dv = __fsub_rn(xs[m], ebar); acc[m] = __fmaf_rn(dv, dv, acc[m]); }
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int m = 0; m < M; ++m) {
        double sum = warp_sum((double)acc[m]);
        if (lane == 0) s_red[warp * M + m] = sum;
    }
    __syncthreads();
    if (threadIdx.x < M) {
        double sum = 0.0;
        for (int w = 0; w < AdamTuning<M>::kWarps; ++w) sum += s_red[w * M + threadIdx.x];
        a.partials[(long long)blockIdx.x * M + threadIdx.x] = sum;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.hdr->status = DPPF_OK;
        a.hdr->magic = kMagic;
        a.hdr->grid = (int)gridDim.x;
        a.hdr->M = M;
        a.hdr->schedule = a.schedule;
    }
}

// Two-launch schedule (when a cooperative launch is refused, or on request): this kernel, then
// adamw_update_kernel on the same grid.  On its own the pass needs a few more registers than
// inside the persistent kernel, so its register budget is relaxed where that avoids spills.
template <int M>
__global__ void __launch_bounds__(AdamTuning<M>::kThreads, (M <= 6) ? AdamTuning<M>::kBlocksPerSM : 1)
adamw_distance_kernel(const RoundArgs a, const AdamArgs p) {
    __shared__ double s_red[AdamTuning<M>::kWarps * M];
    adamw_distance_pass<M, (M == 16) ? 1 : 2>(a, p, s_red);
}

template <int M>
__global__ void __launch_bounds__(AdamTuning<M>::kThreads, AdamTuning<M>::kBlocksPerSM)
adamw_update_kernel(const RoundArgs a, int nblocks_a) {
    __shared__ float s_c[M];
    __shared__ int s_ok;
    if (!finalise(a, M, nblocks_a, s_c, &s_ok)) return;
    update_pass<M, AdamTuning<M>::kUnrollB, AdamTuning<M>::kThreads>(a, s_c);
}

// One persistent cooperative launch: AdamW step + distance pass, grid barrier, update pass.
template <int M>
__global__ void __launch_bounds__(AdamTuning<M>::kThreads, AdamTuning<M>::kBlocksPerSM)
adamw_round_kernel(const RoundArgs a, const AdamArgs p) {
    __shared__ double s_red[AdamTuning<M>::kWarps * M];
    __shared__ float s_c[M];
    __shared__ int s_ok;
    adamw_distance_pass<M, 2>(a, p, s_red);
    cg::this_grid().sync();
    if (!finalise(a, M, (int)gridDim.x, s_c, &s_ok)) return;
    update_pass<M, AdamTuning<M>::kUnrollB, AdamTuning<M>::kThreads>(a, s_c);
}

__global__ void __launch_bounds__(kThreads) adamw_step_kernel(float *x, const AdamArgs p, long long d, long long ld,
                                                              long long nvec) {
    const long long row = (long long)blockIdx.y * ld;
    for (long long j = (long long)blockIdx.x * kThreads + threadIdx.x; j < nvec; j += (long long)gridDim.x * kThreads) {
        const long long off = row + j * 4;
        float4 xx = ld_last_use(x + off), aa = ld_last_use(p.m1 + off), bb = ld_last_use(p.m2 + off),
               gg = ld_last_use(p.g + off);
        adamw4(xx, aa, bb, gg, p);
        st_keep(p.m1 + off, aa);
        st_keep(p.m2 + off, bb);
        st_keep(x + off, xx);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (long long i = nvec * 4; i < d; ++i) {
            const long long off = row + i;
            float xi = x[off], ai = p.m1[off], bi = p.m2[off];
            adamw1(xi, ai, bi, p.g[off], p);
            p.m1[off] = ai;
            p.m2[off] = bi;
            x[off] = xi;
        }
    }
}

}  // namespace
