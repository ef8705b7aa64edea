// DPPF consensus round for one B200 (sm_100a): kernels and the C ABI of include/dppf.h.
//
// Data layout: x[M, ld] fp32, one row per worker, rows 128-byte aligned.  A "vector" is
// one float4 (four consecutive columns of one row); a thread always handles the same
// vector index in all M rows, so the average over workers (Algorithm 1, last line) is a
// purely per-thread quantity and is never written to memory.
//
// Round = distance pass + update pass (single-line pull-push update, Sec. 5):
//   distance pass  reads the M rows once, forms the deviations dev_m = x_m - x_A per
//                  column and accumulates sum(dev_m^2) per worker; each block leaves M
//                  fp64 partial sums in the workspace.
//   update pass    every block first adds the per-block partials in block order (the
//                  same order everywhere, so the result is identical in all blocks and
//                  from run to run), takes r_m = sqrt(.), c_m = alpha - lambda / r_m,
//                  then re-reads the rows, recomputes dev_m with the same instructions
//                  and writes x_m - c_m * dev_m  ( = x_m + (x_A - x_m) c_m ).
// The update pass walks the tiles in reverse so that it starts on the lines the
// distance pass touched last (still in L2) and ends where the next round begins.
//
// Deviations use a shifted mean: e_m = x_m - x_0, ebar = (sum_m e_m)/M, dev_0 = -ebar,
// dev_m = e_m - ebar.  Identical replicas give dev_m == 0 exactly for every M, which
// makes the zero-distance round leave x bit-for-bit unchanged.
#include "dppf.h"

#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <atomic>
#include <climits>
#include <cmath>
#include <cstdint>

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;            // threads per block: generic and local-step kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTemplateM = 16;        // worker counts with register-resident kernels
constexpr int kMaxBlocksSmallM = 2048;   // partial-sum slots reserved per worker, M <= 16
constexpr int kMaxBlocksLargeM = 512;    // ... and for the generic kernels
constexpr size_t kHeaderBytes = 256;
constexpr unsigned kMagic = 0x44505046u; // "DPPF"

struct WsHeader {
    int status;       // dppf_status seen by the kernels
    unsigned magic;   // written by the distance pass, checked by the update pass
    int grid;         // blocks that wrote partials
    int M;
};

struct RoundArgs {
    float *x;
    float *v;         // fused local step only
    const float *g;   // fused local step only
    long long d, ld, nvec;   // nvec = d / 4 full float4 groups per row
    float alpha, lambda, lr, mu, wd;
    float *norms_out; // may be null
    float *norms_stage; // fp32[M] inside the workspace (always written)
    WsHeader *hdr;
    double *partials; // [grid, M]
    int M;            // runtime copy (generic kernels)
};

// ---------------------------------------------------------------- memory access helpers

__device__ __forceinline__ float4 ld_keep(const float *p) {   // normal L2 priority, skip L1
    return __ldcg(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ float4 ld_last_use(const float *p) {  // evict-first: dead after this read
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void st_keep(float *p, float4 v) {
    __stcg(reinterpret_cast<float4 *>(p), v);
}

// ---------------------------------------------------------------- arithmetic helpers
// Explicitly rounded operations: the compiler may not re-associate or contract them, so
// the distance pass and the update pass see bit-identical deviations.

__device__ __forceinline__ float4 sub4(float4 a, float4 b) {
    return make_float4(__fsub_rn(a.x, b.x), __fsub_rn(a.y, b.y), __fsub_rn(a.z, b.z), __fsub_rn(a.w, b.w));
}
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float4 scale4(float4 a, float s) {
    return make_float4(__fmul_rn(a.x, s), __fmul_rn(a.y, s), __fmul_rn(a.z, s), __fmul_rn(a.w, s));
}
__device__ __forceinline__ float sq_acc(float acc, float4 d) {
    acc = __fmaf_rn(d.x, d.x, acc);
    acc = __fmaf_rn(d.y, d.y, acc);
    acc = __fmaf_rn(d.z, d.z, acc);
    acc = __fmaf_rn(d.w, d.w, acc);
    return acc;
}
// x - c * dev
__device__ __forceinline__ float4 apply4(float4 x, float4 dev, float c) {
    return make_float4(__fmaf_rn(-c, dev.x, x.x), __fmaf_rn(-c, dev.y, x.y),
                       __fmaf_rn(-c, dev.z, x.z), __fmaf_rn(-c, dev.w, x.w));
}
// Local optimiser step on one element: g~ = g + wd x ; v' = mu v + g~ ; x' = x - lr v'.
__device__ __forceinline__ void sgd1(float &x, float &v, float g, float lr, float mu, float wd) {
    float gt = __fmaf_rn(wd, x, g);
    v = __fmaf_rn(mu, v, gt);
    x = __fmaf_rn(-lr, v, x);
}
__device__ __forceinline__ void sgd4(float4 &x, float4 &v, float4 g, float lr, float mu, float wd) {
    sgd1(x.x, v.x, g.x, lr, mu, wd);
    sgd1(x.y, v.y, g.y, lr, mu, wd);
    sgd1(x.z, v.z, g.z, lr, mu, wd);
    sgd1(x.w, v.w, g.w, lr, mu, wd);
}

// Shifted mean of one vector over the M rows: ebar = (sum_{m>=1} (x_m - x_0)) / M, so that
// x_A = x_0 + ebar and the deviation of row m is dev_m = (x_m - x_0) - ebar (dev_0 = -ebar).
template <int M>
__device__ __forceinline__ float4 shifted_mean(const float4 (&xv)[M]) {
    const float inv_m = 1.0f / (float)M;
    float4 esum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int m = 1; m < M; ++m) esum = add4(esum, sub4(xv[m], xv[0]));
    return scale4(esum, inv_m);
}
__device__ __forceinline__ float4 deviation(float4 xm, float4 x0, float4 ebar, int m) {
    if (m == 0) return make_float4(-ebar.x, -ebar.y, -ebar.z, -ebar.w);
    return sub4(sub4(xm, x0), ebar);
}

__device__ __forceinline__ double warp_sum(double a) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    return a;   // butterfly: every lane holds the same bits
}

// Coefficient c_m = alpha - lambda / r_m of the single-line update.  Zero distance: the push
// direction is undefined and the pull acts on a zero vector, so the replica must stay as it
// is, bit for bit (including the sign of zeros).  That case is signalled by a NaN coefficient,
// which the update pass reads as "do not write this row".
__device__ __forceinline__ float coefficient(double S, float alpha, float lambda, float *r_out) {
    double r = sqrt(S);
    *r_out = (float)r;
    if (!(r > 0.0)) return __int_as_float(0x7fc00000);
    return (float)((double)alpha - (double)lambda / r);
}
__device__ __forceinline__ bool row_is_written(float c) { return c == c; }

// ---------------------------------------------------------------- register-resident kernels (M <= 16)

// Launch shape per worker count, from sweeps on B200.  The update pass mixes reads and
// writes and is fastest with about 40-48 KB of loads in flight per SM; more outstanding
// requests lower its DRAM efficiency, fewer cannot cover the latency.  The read-only distance
// pass wants about twice that, which it gets from a deeper unroll on the same grid.
//   bytes in flight per SM = kThreads * kBlocksPerSM * unroll * M * 16
template <int M>
struct Tuning {
    static constexpr int kThreads =
        (M <= 2) ? 320 : (M == 3) ? 384 : (M == 4) ? 320 : (M == 5) ? 288 : (M == 6) ? 224 :
        (M <= 8) ? 192 : (M == 9) ? 320 : (M == 10) ? 288 : (M <= 12) ? 256 : 224;
    static constexpr int kBlocksPerSM = (M <= 8) ? 2 : 1;
    static constexpr int kUnrollA = (M <= 2) ? 4 : (M <= 8) ? 2 : 1;      // distance pass
    static constexpr int kUnrollB = (M <= 2) ? 2 : 1;                     // update pass
    // With the local step fused in, the distance pass moves five streams per row (x, v, g in,
    // x, v out) and peaks at about half the resident threads (~60 KB of loads in flight per
    // SM); the update pass of that launch doubles its unroll to keep its own 40-48 KB.
    static constexpr int kBlocksPerSMFused = (kBlocksPerSM > 1) ? kBlocksPerSM / 2 : 1;
    static constexpr int kUnrollFused = 1;
    static constexpr int kUnrollBFused = kUnrollB * (kBlocksPerSM / kBlocksPerSMFused);
    static constexpr int kWarps = kThreads / 32;

};

// Scalar tail: columns 4*nvec .. d-1 (at most three), handled by one thread of block 0.
template <int M, bool kLocalStep>
__device__ __forceinline__ void tail_distance(const RoundArgs &a, float (&acc)[M]) {
    const float inv_m = 1.0f / (float)M;
    for (long long i = a.nvec * 4; i < a.d; ++i) {
        float xs[M];
#pragma unroll
        for (int m = 0; m < M; ++m) {
            float xi = a.x[m * a.ld + i];
            if (kLocalStep) {
                float vi = a.v[m * a.ld + i];
                sgd1(xi, vi, a.g[m * a.ld + i], a.lr, a.mu, a.wd);
                a.v[m * a.ld + i] = vi;
                a.x[m * a.ld + i] = xi;
            }
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

template <int M>
__device__ __forceinline__ void tail_update(const RoundArgs &a, const float *c) {
    const float inv_m = 1.0f / (float)M;
    for (long long i = a.nvec * 4; i < a.d; ++i) {
        float xs[M], dv[M];
#pragma unroll
        for (int m = 0; m < M; ++m) xs[m] = a.x[m * a.ld + i];
        float esum = 0.f;
#pragma unroll
        for (int m = 1; m < M; ++m) { dv[m] = __fsub_rn(xs[m], xs[0]); esum = __fadd_rn(esum, dv[m]); }
        const float ebar = __fmul_rn(esum, inv_m);
        dv[0] = -ebar;
#pragma unroll
        for (int m = 1; m < M; ++m) dv[m] = __fsub_rn(dv[m], ebar);
#pragma unroll
        for (int m = 0; m < M; ++m)
            if (row_is_written(c[m])) a.x[m * a.ld + i] = __fmaf_rn(-c[m], dv[m], xs[m]);
    }
}

// Distance pass body.  Tile t of the block = vectors [(t*U+u)*T + tid], u < U.
template <int M, bool kLocalStep>
__device__ __forceinline__ void distance_pass(const RoundArgs &a, double *s_red /* [warps][M] */) {
    constexpr int U = kLocalStep ? Tuning<M>::kUnrollFused : Tuning<M>::kUnrollA;
    constexpr int T = Tuning<M>::kThreads;
    const long long tile_vecs = (long long)T * U;
    const long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    float acc[M];
#pragma unroll
    for (int m = 0; m < M; ++m) acc[m] = 0.f;

    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
        float4 xv[U][M];
        bool live[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long j = (t * U + u) * T + threadIdx.x;
            live[u] = j < a.nvec;
            if (live[u]) {
                if (kLocalStep) {
                    // Rows in groups of four: all loads of a group are issued before its first
                    // store (x, v, g may not alias, but the compiler cannot know that and
                    // would otherwise order every row's loads behind the previous row's stores).
                    constexpr int G = 4;
#pragma unroll
                    for (int m0 = 0; m0 < M; m0 += G) {
                        float4 vv[G], gv[G];
#pragma unroll
                        for (int k = 0; k < G; ++k) {
                            if (m0 + k < M) {
                                const long long off = (m0 + k) * a.ld + j * 4;
                                xv[u][m0 + k] = ld_last_use(a.x + off);
                                vv[k] = ld_last_use(a.v + off);
                                gv[k] = ld_last_use(a.g + off);
                            }
                        }
#pragma unroll
                        for (int k = 0; k < G; ++k) {
                            if (m0 + k < M) {
                                const long long off = (m0 + k) * a.ld + j * 4;
                                sgd4(xv[u][m0 + k], vv[k], gv[k], a.lr, a.mu, a.wd);
                                st_keep(a.v + off, vv[k]);
                                st_keep(a.x + off, xv[u][m0 + k]);
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int m = 0; m < M; ++m) xv[u][m] = ld_keep(a.x + m * a.ld + j * 4);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (live[u]) {
                const float4 ebar = shifted_mean<M>(xv[u]);
#pragma unroll
                for (int m = 0; m < M; ++m) acc[m] = sq_acc(acc[m], deviation(xv[u][m], xv[u][0], ebar, m));
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) tail_distance<M, kLocalStep>(a, acc);

    // thread -> warp (butterfly, fp64) -> block (warp order) -> one fp64 partial per worker
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int m = 0; m < M; ++m) {
        double s = warp_sum((double)acc[m]);
        if (lane == 0) s_red[warp * M + m] = s;
    }
    __syncthreads();
    if (threadIdx.x < M) {
        double s = 0.0;
        for (int w = 0; w < Tuning<M>::kWarps; ++w) s += s_red[w * M + threadIdx.x];
        a.partials[(long long)blockIdx.x * M + threadIdx.x] = s;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.hdr->status = DPPF_OK;
        a.hdr->magic = kMagic;
        a.hdr->grid = (int)gridDim.x;
        a.hdr->M = M;
    }
}

// Cross-block sum in block order, identical in every block; fills s_c[M] and reports r_m.
// Returns false if the workspace header does not describe this launch.
__device__ __forceinline__ bool finalise(const RoundArgs &a, int M, int nblocks, float *s_c, int *s_ok) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0)
        *s_ok = (a.hdr->magic == kMagic && a.hdr->grid == nblocks && a.hdr->M == M) ? 1 : 0;
    const int nwarps = blockDim.x >> 5;
    for (int m = warp; m < M; m += nwarps) {
        double s = 0.0;
        for (int b = lane; b < nblocks; b += 32) s += __ldcg(a.partials + (long long)b * M + m);
        s = warp_sum(s);
        if (lane == 0) {
            float r;
            s_c[m] = coefficient(s, a.alpha, a.lambda, &r);
            if (blockIdx.x == 0) {
                a.norms_stage[m] = r;
                if (a.norms_out) a.norms_out[m] = r;
            }
        }
    }
    __syncthreads();
    if (!*s_ok && blockIdx.x == 0 && threadIdx.x == 0) a.hdr->status = DPPF_ERR_WORKSPACE;
    return *s_ok != 0;
}

template <int M, int U>
__device__ __forceinline__ void update_pass(const RoundArgs &a, const float *s_c) {
    constexpr int T = Tuning<M>::kThreads;
    const long long tile_vecs = (long long)T * U;
    const long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    const float *c = s_c;
    if (ntiles > blockIdx.x) {
        // last tile of this block's static sequence, then backwards
        long long t = blockIdx.x + (ntiles - 1 - blockIdx.x) / gridDim.x * gridDim.x;
        for (; t >= 0; t -= gridDim.x) {
            float4 xv[U][M];
            bool live[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long j = (t * U + u) * T + threadIdx.x;
                live[u] = j < a.nvec;
                if (live[u]) {
#pragma unroll
                    for (int m = 0; m < M; ++m) xv[u][m] = ld_last_use(a.x + m * a.ld + j * 4);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (live[u]) {
                    const long long j = (t * U + u) * T + threadIdx.x;
                    const float4 ebar = shifted_mean<M>(xv[u]);
#pragma unroll
                    for (int m = 0; m < M; ++m)
                        if (row_is_written(c[m]))
                            st_keep(a.x + m * a.ld + j * 4,
                                    apply4(xv[u][m], deviation(xv[u][m], xv[u][0], ebar, m), c[m]));
                }
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) tail_update<M>(a, c);
}

template <int M, bool kLocalStep>
__global__ void __launch_bounds__(Tuning<M>::kThreads, (kLocalStep ? Tuning<M>::kBlocksPerSMFused : Tuning<M>::kBlocksPerSM))
distance_kernel(const RoundArgs a) {
    __shared__ double s_red[Tuning<M>::kWarps * M];
    distance_pass<M, kLocalStep>(a, s_red);
}

template <int M, bool kAfterLocalStep>
__global__ void __launch_bounds__(Tuning<M>::kThreads, (kAfterLocalStep ? Tuning<M>::kBlocksPerSMFused : Tuning<M>::kBlocksPerSM))
update_kernel(const RoundArgs a, int nblocks_a) {
    __shared__ float s_c[M];
    __shared__ int s_ok;
    if (!finalise(a, M, nblocks_a, s_c, &s_ok)) return;
    update_pass<M, (kAfterLocalStep ? Tuning<M>::kUnrollBFused : Tuning<M>::kUnrollB)>(a, s_c);
}

// One persistent launch: distance pass, grid-wide barrier, update pass.  Launched with
// cudaLaunchCooperativeKernel, which refuses the launch unless all blocks are co-resident.
template <int M, bool kLocalStep>
__global__ void __launch_bounds__(Tuning<M>::kThreads, (kLocalStep ? Tuning<M>::kBlocksPerSMFused : Tuning<M>::kBlocksPerSM))
round_kernel(const RoundArgs a) {
    __shared__ double s_red[Tuning<M>::kWarps * M];
    __shared__ float s_c[M];
    __shared__ int s_ok;
    distance_pass<M, kLocalStep>(a, s_red);
    cg::this_grid().sync();
    if (!finalise(a, M, (int)gridDim.x, s_c, &s_ok)) return;
    update_pass<M, (kLocalStep ? Tuning<M>::kUnrollBFused : Tuning<M>::kUnrollB)>(a, s_c);
}

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

// Distance pass with the AdamW step applied first; leaves the same partial sums and header
// as distance_kernel, so update_kernel<M, false> completes the round.  Measured best with
// the plain round's residency and two rows of loads in flight per thread.
template <int M>
__global__ void __launch_bounds__(Tuning<M>::kThreads, Tuning<M>::kBlocksPerSM)
adamw_distance_kernel(const RoundArgs a, const AdamArgs p) {
    constexpr int T = Tuning<M>::kThreads;
    constexpr int G = 2;                               // rows whose loads are issued together
    __shared__ double s_red[Tuning<M>::kWarps * M];
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
        for (int w = 0; w < Tuning<M>::kWarps; ++w) sum += s_red[w * M + threadIdx.x];
        a.partials[(long long)blockIdx.x * M + threadIdx.x] = sum;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.hdr->status = DPPF_OK;
        a.hdr->magic = kMagic;
        a.hdr->grid = (int)gridDim.x;
        a.hdr->M = M;
    }
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

// ---------------------------------------------------------------- staged persistent kernel (default, M <= 16)
// One block per SM keeps a ring of up to kMaxStages shared-memory stages; a stage holds the same
// column chunk of all M rows (about 32 KB).  One thread fills stages with 1-D bulk async
// copies (cp.async.bulk, completion on an mbarrier); all threads then read the chunk from
// shared memory.  Both passes run in this one cooperative launch:
//   distance pass  chunks in ascending order, up to kPrefetchA chunks (~96 KB) in flight;
//   update pass    the same chunks in descending order with one chunk (~32 KB) in flight --
//                  the read/write mix is fastest with few outstanding loads -- results go
//                  straight from registers to global memory.
// The last kStages chunks of the distance pass are still in the ring when the update pass
// starts, so it consumes them without touching DRAM or L2 again.
// Every wait on an mbarrier is bounded; if one gives up the block marks its partial sums
// with a negative value, every block then sees the mark after the grid barrier, nobody
// writes x, and the status word reports DPPF_ERR_TIMEOUT.

constexpr int kStagedThreads = 256;
constexpr int kStagedWarps = kStagedThreads / 32;
constexpr int kMaxStages = 6;
constexpr int kPrefetchA = 3;
constexpr int kPrefetchB = 1;
constexpr int kSpinLimit = 1 << 22;   // mbarrier try_wait polls before a wait gives up (~ a second)

template <int M>
struct StagedShape {
    // columns per stage and row: a stage of about 32 KB (40 KB measured best for M = 8)
    static constexpr int kChunk = (M == 8) ? 1280 : ((8192 / M) / 128) * 128;
    static constexpr size_t kStageFloats = (size_t)M * kChunk;
    static constexpr int kFit = (int)((200 * 1024) / (kStageFloats * sizeof(float)));
    static constexpr int kStages = kFit < kMaxStages ? kFit : kMaxStages;
    static constexpr size_t kSmemBytes = (size_t)kStages * kStageFloats * sizeof(float);
    static_assert(kStages > kPrefetchA, "ring must be deeper than the prefetch distance");
};

__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long *bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long *bar, unsigned parity) {
    for (int spins = 0; spins < kSpinLimit; ++spins)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, unsigned bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

template <int M>
__global__ void __launch_bounds__(kStagedThreads, 1) round_kernel_staged(const RoundArgs a) {
    constexpr int CH = StagedShape<M>::kChunk;
    constexpr int kStages = StagedShape<M>::kStages;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *ring = reinterpret_cast<float *>(smem_raw);             // [kStages][M][CH]
    __shared__ unsigned long long full[kStages];
    __shared__ double s_red[kStagedWarps * M];
    __shared__ float s_c[M];
    __shared__ int s_ok;
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int st = 0; st < kStages; ++st) mbar_init(&full[st], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const long long d4 = a.nvec * 4;                                // columns covered by float4 groups
    const long long nchunks = (d4 + CH - 1) / CH;
    // this block's chunks, by local index k: chunk blockIdx.x + k * gridDim.x, ring stage k % kStages
    const long long n = (nchunks > blockIdx.x) ? (nchunks - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    unsigned phase = 0;                                             // bit st: parity of the next wait on stage st
    int failed = 0;

    auto chunk_cols = [&](long long k) -> int {
        const long long c0 = (blockIdx.x + k * gridDim.x) * CH;
        return (int)((d4 - c0 < CH) ? (d4 - c0) : CH);
    };
    auto issue = [&](long long k) {                                 // one thread: M row copies into one stage
        const int st = (int)(k % kStages);
        const long long c0 = (blockIdx.x + k * gridDim.x) * CH;
        const unsigned bytes = (unsigned)chunk_cols(k) * 4u;
        mbar_expect_tx(&full[st], bytes * M);
#pragma unroll
        for (int m = 0; m < M; ++m)
            bulk_load(ring + ((size_t)st * M + m) * CH, a.x + m * a.ld + c0, bytes, &full[st]);
    };

    // ---- distance pass
    double acc[M];
#pragma unroll
    for (int m = 0; m < M; ++m) acc[m] = 0.0;
    if (tid == 0)
        for (long long k = 0; k < kPrefetchA && k < n; ++k) issue(k);
    long long k_done = 0;                                           // chunks consumed so far
    for (long long k = 0; k < n; ++k) {
        if (tid == 0 && k + kPrefetchA < n) issue(k + kPrefetchA);
        const int st = (int)(k % kStages);
        int my_fail = mbar_wait_bounded(&full[st], (phase >> st) & 1u) ? 0 : 1;
        phase ^= 1u << st;
        if (!my_fail) {
            const int cols = chunk_cols(k);
            const float *sb = ring + (size_t)st * M * CH;
            float part[M];
#pragma unroll
            for (int m = 0; m < M; ++m) part[m] = 0.f;
            for (int q = tid * 4; q < cols; q += kStagedThreads * 4) {
                float4 xv[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
                const float4 ebar = shifted_mean<M>(xv);
#pragma unroll
                for (int m = 0; m < M; ++m) part[m] = sq_acc(part[m], deviation(xv[m], xv[0], ebar, m));
            }
#pragma unroll
            for (int m = 0; m < M; ++m) acc[m] += (double)part[m];
        }
        k_done = k + 1;
        if (__syncthreads_or(my_fail)) { failed = 1; break; }      // block-uniform decision
    }
    if (failed && tid == 0) {
        // give this block's copies still in flight a bounded chance to land before moving on
        const long long hi = (k_done - 1 + kPrefetchA < n - 1) ? k_done - 1 + kPrefetchA : n - 1;
        for (long long k = k_done; k <= hi; ++k) {
            const int st = (int)(k % kStages);
            mbar_wait_bounded(&full[st], (phase >> st) & 1u);
        }
    }
    if (blockIdx.x == 0 && tid == 0) {
        float tail[M];
#pragma unroll
        for (int m = 0; m < M; ++m) tail[m] = 0.f;
        tail_distance<M, false>(a, tail);
#pragma unroll
        for (int m = 0; m < M; ++m) acc[m] += (double)tail[m];
    }
    {
        const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
        for (int m = 0; m < M; ++m) {
            double sum = warp_sum(acc[m]);
            if (lane == 0) s_red[warp * M + m] = sum;
        }
        __syncthreads();
        if (tid < M) {
            double sum = 0.0;
            for (int w = 0; w < kStagedWarps; ++w) sum += s_red[w * M + tid];
            a.partials[(long long)blockIdx.x * M + tid] = failed ? -1.0 : sum;   // negative = "a wait gave up"
        }
        if (blockIdx.x == 0 && tid == 0) {
            a.hdr->status = DPPF_OK;
            a.hdr->magic = kMagic;
            a.hdr->grid = (int)gridDim.x;
            a.hdr->M = M;
        }
    }
    cg::this_grid().sync();

    // ---- every block: did any block give up?  (same answer everywhere)
    {
        int bad = 0;
        for (int i = tid; i < (int)gridDim.x * M; i += kStagedThreads) bad |= (__ldcg(a.partials + i) < 0.0) ? 1 : 0;
        if (__syncthreads_or(bad)) {
            if (blockIdx.x == 0 && tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;
            return;                                                 // x untouched
        }
    }
    if (!finalise(a, M, (int)gridDim.x, s_c, &s_ok)) return;

    // ---- update pass: local chunks n-1 .. 0; the newest min(n, kStages) are still in the ring
    const long long resident = (n < kStages) ? n : (long long)kStages;
    for (long long k = n - 1; k >= 0; --k) {
        if (tid == 0) {
            const long long kl = k - kPrefetchB;                    // its stage held chunk kl + kStages: already done
            if (kl >= 0 && kl < n - resident) issue(kl);
        }
        const int st = (int)(k % kStages);
        int my_fail = 0;
        if (k < n - resident) {
            my_fail = mbar_wait_bounded(&full[st], (phase >> st) & 1u) ? 0 : 1;
            phase ^= 1u << st;
        }
        if (!my_fail) {
            const int cols = chunk_cols(k);
            const long long c0 = (blockIdx.x + k * gridDim.x) * CH;
            const float *sb = ring + (size_t)st * M * CH;
            for (int q = tid * 4; q < cols; q += kStagedThreads * 4) {
                float4 xv[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
                const float4 ebar = shifted_mean<M>(xv);
#pragma unroll
                for (int m = 0; m < M; ++m)
                    if (row_is_written(s_c[m]))
                        st_keep(a.x + m * a.ld + c0 + q, apply4(xv[m], deviation(xv[m], xv[0], ebar, m), s_c[m]));
            }
        }
        if (__syncthreads_or(my_fail)) {
            if (tid == 0) {
                a.hdr->status = DPPF_ERR_TIMEOUT;                   // x is partly updated
                const long long kl = k - kPrefetchB;                // the one copy that may still be in flight
                if (k < n - resident && kl >= 0) mbar_wait_bounded(&full[(int)(kl % kStages)], (phase >> (int)(kl % kStages)) & 1u);
            }
            return;
        }
    }
    if (blockIdx.x == 0 && tid == 0) tail_update<M>(a, s_c);
}

// ---------------------------------------------------------------- general round (staged, M <= 16)
// Algorithm 1 with an arbitrary consensus variable x_C = sum_m w_m x_m (weights normalised
// on the host), the push taken from x_A or from x_C (the remark on LSGD), and optionally
// both terms of the regulariser's gradient (step (a) of the equation in Sec. 5):
//   y_m  = x_m + alpha (x_C - x_m)                       pull
//   u_m  = (y_m - P) / ||y_m - P||,  P = x_A or x_C      push direction of the pulled point
//   x_m+ = y_m + lambda u_m  [ - lambda (1/M) sum_j u_j ]
// Same two passes and the same traffic as the plain round: on one GPU the mean direction
// is a per-column register sum, so the second term needs no extra vector or pass.
// Everything is expressed relative to row 0 (e_m = x_m - x_0), like the shifted mean.

constexpr int kGeneralThreads = 256;   // 384/512/768 threads measured slower (registers)
constexpr int kGeneralWarps = kGeneralThreads / 32;

struct GeneralArgs {
    float *x;
    long long d, ld, nvec;
    float alpha, lambda;
    float wn[kMaxTemplateM];     // w_m / sum w
    int push_from_c, two_term;
    float *norms_out;            // ||x_m - x_A|| before the round, may be null
    float *push_norms_out;       // ||y_m - P||, may be null
    WsHeader *hdr;
    double *partials;            // [grid][2 M]: squared distances to x_A, then of the pulled points to P
};

template <int M>
struct GeneralColumn {
    // one column: xs[m] in; adds the two squared distances per worker
    static __device__ __forceinline__ void distances(const float (&xs)[M], const GeneralArgs &a, float (&pr)[M],
                                                     float (&pn)[M]) {
        float e[M], ea = 0.f, ec = 0.f;
        e[0] = 0.f;
#pragma unroll
        for (int m = 1; m < M; ++m) {
            e[m] = __fsub_rn(xs[m], xs[0]);
            ea = __fadd_rn(ea, e[m]);
            ec = __fmaf_rn(a.wn[m], e[m], ec);
        }
        ea = __fmul_rn(ea, 1.0f / (float)M);
        const float p = a.push_from_c ? ec : ea;
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const float dev = __fsub_rn(e[m], ea);
            pr[m] = __fmaf_rn(dev, dev, pr[m]);
            const float dy = __fmaf_rn(a.alpha, __fsub_rn(ec, e[m]), __fsub_rn(e[m], p));
            pn[m] = __fmaf_rn(dy, dy, pn[m]);
        }
    }
    // one column: xs[m] in, updated replicas out; g[m] = lambda / ||y_m - P|| (0: no direction)
    static __device__ __forceinline__ void update(float (&xs)[M], const GeneralArgs &a, const float *g) {
        float e[M], ea = 0.f, ec = 0.f;
        e[0] = 0.f;
#pragma unroll
        for (int m = 1; m < M; ++m) {
            e[m] = __fsub_rn(xs[m], xs[0]);
            ea = __fadd_rn(ea, e[m]);
            ec = __fmaf_rn(a.wn[m], e[m], ec);
        }
        ea = __fmul_rn(ea, 1.0f / (float)M);
        const float p = a.push_from_c ? ec : ea;
        float ub = 0.f;                                   // lambda * mean direction
        if (a.two_term) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const float dy = __fmaf_rn(a.alpha, __fsub_rn(ec, e[m]), __fsub_rn(e[m], p));
                ub = __fmaf_rn(g[m], dy, ub);
            }
            ub = __fmul_rn(ub, 1.0f / (float)M);
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const float pull = __fsub_rn(ec, e[m]);       // x_C - x_m
            const float dy = __fmaf_rn(a.alpha, pull, __fsub_rn(e[m], p));
            const float y = __fmaf_rn(a.alpha, pull, xs[m]);
            xs[m] = __fsub_rn(__fmaf_rn(g[m], dy, y), ub);
        }
    }
};

template <int M>
__global__ void __launch_bounds__(kGeneralThreads, 1) general_round_kernel(const GeneralArgs a) {
    constexpr int CH = StagedShape<M>::kChunk;
    constexpr int kStages = StagedShape<M>::kStages;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    float *ring = reinterpret_cast<float *>(smem_raw);
    __shared__ unsigned long long full[kStages];
    __shared__ double s_red[kGeneralWarps * 2 * M];
    __shared__ float s_g[M];
    __shared__ int s_flag;
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int st = 0; st < kStages; ++st) mbar_init(&full[st], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const long long d4 = a.nvec * 4;
    const long long nchunks = (d4 + CH - 1) / CH;
    const long long n = (nchunks > blockIdx.x) ? (nchunks - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    unsigned phase = 0;
    int failed = 0;
    auto chunk_cols = [&](long long k) -> int {
        const long long c0 = (blockIdx.x + k * gridDim.x) * CH;
        return (int)((d4 - c0 < CH) ? (d4 - c0) : CH);
    };
    auto issue = [&](long long k) {
        const int st = (int)(k % kStages);
        const long long c0 = (blockIdx.x + k * gridDim.x) * CH;
        const unsigned bytes = (unsigned)chunk_cols(k) * 4u;
        mbar_expect_tx(&full[st], bytes * M);
#pragma unroll
        for (int m = 0; m < M; ++m)
            bulk_load(ring + ((size_t)st * M + m) * CH, a.x + m * a.ld + c0, bytes, &full[st]);
    };

    // ---- distance pass: sum (x_m - x_A)^2 and sum (y_m - P)^2 per worker
    double acc[2 * M];
#pragma unroll
    for (int m = 0; m < 2 * M; ++m) acc[m] = 0.0;
    if (tid == 0)
        for (long long k = 0; k < kPrefetchA && k < n; ++k) issue(k);
    long long k_done = 0;
    for (long long k = 0; k < n; ++k) {
        if (tid == 0 && k + kPrefetchA < n) issue(k + kPrefetchA);
        const int st = (int)(k % kStages);
        int my_fail = mbar_wait_bounded(&full[st], (phase >> st) & 1u) ? 0 : 1;
        phase ^= 1u << st;
        if (!my_fail) {
            const int cols = chunk_cols(k);
            const float *sb = ring + (size_t)st * M * CH;
            float pr[M], pn[M];
#pragma unroll
            for (int m = 0; m < M; ++m) pr[m] = pn[m] = 0.f;
            for (int q = tid * 4; q < cols; q += kGeneralThreads * 4) {
                float4 xv[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
                float xs[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xs[m] = xv[m].x;
                GeneralColumn<M>::distances(xs, a, pr, pn);
#pragma unroll
                for (int m = 0; m < M; ++m) xs[m] = xv[m].y;
                GeneralColumn<M>::distances(xs, a, pr, pn);
#pragma unroll
                for (int m = 0; m < M; ++m) xs[m] = xv[m].z;
                GeneralColumn<M>::distances(xs, a, pr, pn);
#pragma unroll
                for (int m = 0; m < M; ++m) xs[m] = xv[m].w;
                GeneralColumn<M>::distances(xs, a, pr, pn);
            }
#pragma unroll
            for (int m = 0; m < M; ++m) {
                acc[m] += (double)pr[m];
                acc[M + m] += (double)pn[m];
            }
        }
        k_done = k + 1;
        if (__syncthreads_or(my_fail)) { failed = 1; break; }
    }
    if (failed && tid == 0) {
        const long long hi = (k_done - 1 + kPrefetchA < n - 1) ? k_done - 1 + kPrefetchA : n - 1;
        for (long long k = k_done; k <= hi; ++k) {
            const int st = (int)(k % kStages);
            mbar_wait_bounded(&full[st], (phase >> st) & 1u);
        }
    }
    if (blockIdx.x == 0 && tid == 0) {                    // scalar tail columns
        float pr[M], pn[M];
#pragma unroll
        for (int m = 0; m < M; ++m) pr[m] = pn[m] = 0.f;
        for (long long i = d4; i < a.d; ++i) {
            float xs[M];
#pragma unroll
            for (int m = 0; m < M; ++m) xs[m] = a.x[m * a.ld + i];
            GeneralColumn<M>::distances(xs, a, pr, pn);
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
            acc[m] += (double)pr[m];
            acc[M + m] += (double)pn[m];
        }
    }
    {
        const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
        for (int m = 0; m < 2 * M; ++m) {
            double sum = warp_sum(acc[m]);
            if (lane == 0) s_red[warp * 2 * M + m] = sum;
        }
        __syncthreads();
        if (tid < 2 * M) {
            double sum = 0.0;
            for (int w = 0; w < kGeneralWarps; ++w) sum += s_red[w * 2 * M + tid];
            a.partials[(long long)blockIdx.x * 2 * M + tid] = failed ? -1.0 : sum;
        }
        if (blockIdx.x == 0 && tid == 0) {
            a.hdr->status = DPPF_OK;
            a.hdr->magic = kMagic;
            a.hdr->grid = (int)gridDim.x;
            a.hdr->M = M;
        }
    }
    cg::this_grid().sync();

    {   // did any block give up?
        int bad = 0;
        for (int i = tid; i < (int)gridDim.x * 2 * M; i += kGeneralThreads) bad |= (__ldcg(a.partials + i) < 0.0) ? 1 : 0;
        if (__syncthreads_or(bad)) {
            if (blockIdx.x == 0 && tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;
            return;
        }
    }
    {   // cross-block sums in block order (identical in every block)
        const int lane = tid & 31, warp = tid >> 5;
        if (tid == 0) s_flag = 0;
        __syncthreads();
        for (int j = warp; j < 2 * M; j += kGeneralWarps) {
            double sum = 0.0;
            for (int b = lane; b < (int)gridDim.x; b += 32) sum += __ldcg(a.partials + (long long)b * 2 * M + j);
            sum = warp_sum(sum);
            if (lane == 0) {
                const double nrm = sqrt(sum);
                if (j < M) {
                    if (nrm > 0.0) s_flag = 1;            // some replica differs from the average
                    if (blockIdx.x == 0 && a.norms_out) a.norms_out[j] = (float)nrm;
                } else {
                    s_g[j - M] = (nrm > 0.0) ? (float)((double)a.lambda / nrm) : 0.f;
                    if (blockIdx.x == 0 && a.push_norms_out) a.push_norms_out[j - M] = (float)nrm;
                }
            }
        }
        __syncthreads();
        if (!s_flag) return;                              // identical replicas: nothing moves, x untouched
    }

    // ---- update pass, chunks in reverse, newest chunks reused from the ring
    const long long resident = (n < kStages) ? n : (long long)kStages;
    for (long long k = n - 1; k >= 0; --k) {
        if (tid == 0) {
            const long long kl = k - kPrefetchB;
            if (kl >= 0 && kl < n - resident) issue(kl);
        }
        const int st = (int)(k % kStages);
        int my_fail = 0;
        if (k < n - resident) {
            my_fail = mbar_wait_bounded(&full[st], (phase >> st) & 1u) ? 0 : 1;
            phase ^= 1u << st;
        }
        if (!my_fail) {
            const int cols = chunk_cols(k);
            const long long c0 = (blockIdx.x + k * gridDim.x) * CH;
            const float *sb = ring + (size_t)st * M * CH;
            for (int q = tid * 4; q < cols; q += kGeneralThreads * 4) {
                float4 xv[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
                float xs[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xs[m] = xv[m].x;
                GeneralColumn<M>::update(xs, a, s_g);
#pragma unroll
                for (int m = 0; m < M; ++m) { xv[m].x = xs[m]; xs[m] = xv[m].y; }
                GeneralColumn<M>::update(xs, a, s_g);
#pragma unroll
                for (int m = 0; m < M; ++m) { xv[m].y = xs[m]; xs[m] = xv[m].z; }
                GeneralColumn<M>::update(xs, a, s_g);
#pragma unroll
                for (int m = 0; m < M; ++m) { xv[m].z = xs[m]; xs[m] = xv[m].w; }
                GeneralColumn<M>::update(xs, a, s_g);
#pragma unroll
                for (int m = 0; m < M; ++m) {
                    xv[m].w = xs[m];
                    st_keep(a.x + m * a.ld + c0 + q, xv[m]);
                }
            }
        }
        if (__syncthreads_or(my_fail)) {
            if (tid == 0) {
                a.hdr->status = DPPF_ERR_TIMEOUT;
                const long long kl = k - kPrefetchB;
                if (k < n - resident && kl >= 0) mbar_wait_bounded(&full[(int)(kl % kStages)], (phase >> (int)(kl % kStages)) & 1u);
            }
            return;
        }
    }
    if (blockIdx.x == 0 && tid == 0) {
        for (long long i = d4; i < a.d; ++i) {
            float xs[M];
#pragma unroll
            for (int m = 0; m < M; ++m) xs[m] = a.x[m * a.ld + i];
            GeneralColumn<M>::update(xs, a, s_g);
#pragma unroll
            for (int m = 0; m < M; ++m) a.x[m * a.ld + i] = xs[m];
        }
    }
}

// ---------------------------------------------------------------- generic kernels (16 < M <= 1024)
// Rows are streamed twice per vector (second time from L1/L2); per-worker sums live in
// shared memory, one fp32 slot per (warp, worker), so no thread needs M registers.

template <bool kLocalStep>
__global__ void __launch_bounds__(kThreads) distance_kernel_generic(const RoundArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *s_acc = reinterpret_cast<float *>(smem_raw);               // [kWarps][M]
    const int M = a.M, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float inv_m = 1.0f / (float)M;
    for (int i = threadIdx.x; i < kWarps * M; i += kThreads) s_acc[i] = 0.f;
    __syncthreads();
    float *my_acc = s_acc + warp * M;
    const long long ntiles = (a.nvec + kThreads - 1) / kThreads;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const long long j = t * kThreads + threadIdx.x;
        const bool live = j < a.nvec;
        float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), esum = x0;
        if (live) {
            for (int m = 0; m < M; ++m) {
                const long long off = m * a.ld + j * 4;
                float4 xr = *reinterpret_cast<const float4 *>(a.x + off);
                if (kLocalStep) {
                    float4 vr = ld_last_use(a.v + off), gr = ld_last_use(a.g + off);
                    sgd4(xr, vr, gr, a.lr, a.mu, a.wd);
                    st_keep(a.v + off, vr);
                    *reinterpret_cast<float4 *>(a.x + off) = xr;
                }
                if (m == 0) x0 = xr; else esum = add4(esum, sub4(xr, x0));
            }
        }
        const float4 ebar = scale4(esum, inv_m);
        for (int m = 0; m < M; ++m) {
            float q = 0.f;
            if (live) {
                float4 dv;
                if (m == 0) dv = make_float4(-ebar.x, -ebar.y, -ebar.z, -ebar.w);
                else dv = sub4(sub4(*reinterpret_cast<const float4 *>(a.x + m * a.ld + j * 4), x0), ebar);
                q = sq_acc(0.f, dv);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
            if (lane == 0) my_acc[m] += q;
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {      // scalar tail columns
        for (long long i = a.nvec * 4; i < a.d; ++i) {
            float x0s = 0.f, esum = 0.f;
            for (int m = 0; m < M; ++m) {
                float xi = a.x[m * a.ld + i];
                if (kLocalStep) {
                    float vi = a.v[m * a.ld + i];
                    sgd1(xi, vi, a.g[m * a.ld + i], a.lr, a.mu, a.wd);
                    a.v[m * a.ld + i] = vi;
                    a.x[m * a.ld + i] = xi;
                }
                if (m == 0) x0s = xi; else esum = __fadd_rn(esum, __fsub_rn(xi, x0s));
            }
            const float ebar = __fmul_rn(esum, inv_m);
            for (int m = 0; m < M; ++m) {
                float dv = (m == 0) ? -ebar : __fsub_rn(__fsub_rn(a.x[m * a.ld + i], x0s), ebar);
                my_acc[m] = __fmaf_rn(dv, dv, my_acc[m]);
            }
        }
    }
    __syncthreads();
    for (int m = threadIdx.x; m < M; m += kThreads) {
        double s = 0.0;
        for (int w = 0; w < kWarps; ++w) s += (double)s_acc[w * M + m];
        a.partials[(long long)blockIdx.x * M + m] = s;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.hdr->status = DPPF_OK;
        a.hdr->magic = kMagic;
        a.hdr->grid = (int)gridDim.x;
        a.hdr->M = M;
    }
}

__global__ void __launch_bounds__(kThreads) update_kernel_generic(const RoundArgs a, int nblocks_a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *s_c = reinterpret_cast<float *>(smem_raw);                 // [M]
    __shared__ int s_ok;
    const int M = a.M;
    const float inv_m = 1.0f / (float)M;
    if (!finalise(a, M, nblocks_a, s_c, &s_ok)) return;
    const long long ntiles = (a.nvec + kThreads - 1) / kThreads;
    if (ntiles > blockIdx.x) {
        long long t = blockIdx.x + (ntiles - 1 - blockIdx.x) / gridDim.x * gridDim.x;
        for (; t >= 0; t -= gridDim.x) {
            const long long j = t * kThreads + threadIdx.x;
            if (j >= a.nvec) continue;
            float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), esum = x0;
            for (int m = 0; m < M; ++m) {
                float4 xr = *reinterpret_cast<const float4 *>(a.x + m * a.ld + j * 4);
                if (m == 0) x0 = xr; else esum = add4(esum, sub4(xr, x0));
            }
            const float4 ebar = scale4(esum, inv_m);
            for (int m = M - 1; m >= 0; --m) {       // row 0 last: the others still need x0 (in a register)
                float *p = a.x + m * a.ld + j * 4;
                float4 xr = (m == 0) ? x0 : *reinterpret_cast<const float4 *>(p);
                float4 dv = (m == 0) ? make_float4(-ebar.x, -ebar.y, -ebar.z, -ebar.w) : sub4(sub4(xr, x0), ebar);
                if (row_is_written(s_c[m])) st_keep(p, apply4(xr, dv, s_c[m]));
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (long long i = a.nvec * 4; i < a.d; ++i) {
            float x0s = a.x[i], esum = 0.f;
            for (int m = 1; m < M; ++m) esum = __fadd_rn(esum, __fsub_rn(a.x[m * a.ld + i], x0s));
            const float ebar = __fmul_rn(esum, inv_m);
            for (int m = M - 1; m >= 0; --m) {
                float xi = a.x[m * a.ld + i];
                float dv = (m == 0) ? -ebar : __fsub_rn(__fsub_rn(xi, x0s), ebar);
                if (row_is_written(s_c[m])) a.x[m * a.ld + i] = __fmaf_rn(-s_c[m], dv, xi);
            }
        }
    }
}

// ---------------------------------------------------------------- stand-alone local step

__global__ void __launch_bounds__(kThreads) local_step_kernel(float *x, float *v, const float *g, long long d,
                                                              long long ld, long long nvec, float lr, float mu,
                                                              float wd) {
    const long long row = (long long)blockIdx.y * ld;
    float *xr = x + row, *vr = v + row;
    const float *gr = g + row;
    for (long long j = (long long)blockIdx.x * kThreads + threadIdx.x; j < nvec; j += (long long)gridDim.x * kThreads) {
        float4 xx = ld_last_use(xr + j * 4), vv = ld_last_use(vr + j * 4), gg = ld_last_use(gr + j * 4);
        sgd4(xx, vv, gg, lr, mu, wd);
        st_keep(vr + j * 4, vv);
        st_keep(xr + j * 4, xx);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (long long i = nvec * 4; i < d; ++i) {
            float xi = xr[i], vi = vr[i];
            sgd1(xi, vi, gr[i], lr, mu, wd);
            vr[i] = vi;
            xr[i] = xi;
        }
    }
}

// Zero distances for the one-worker case (x_A == x_1).
__global__ void zero_norms_kernel(float *norms_out, float *norms_stage, WsHeader *hdr) {
    if (threadIdx.x == 0) {
        norms_stage[0] = 0.f;
        if (norms_out) norms_out[0] = 0.f;
        hdr->status = DPPF_OK;
        hdr->magic = 0;
    }
}

// ---------------------------------------------------------------- host side

struct DeviceInfo {
    std::atomic<int> sms{0};
    std::atomic<int> coop{-1};
};
DeviceInfo g_dev[64];   // immutable facts about each device, filled on first use

int sm_count(int dev) {
    int n = g_dev[dev].sms.load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return -1;
        g_dev[dev].sms.store(n, std::memory_order_relaxed);
    }
    return n;
}

bool coop_supported(int dev) {
    int c = g_dev[dev].coop.load(std::memory_order_relaxed);
    if (c < 0) {
        if (cudaDeviceGetAttribute(&c, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) c = 0;
        g_dev[dev].coop.store(c, std::memory_order_relaxed);
    }
    return c != 0;
}

int max_blocks_for(int M) { return M <= kMaxTemplateM ? kMaxBlocksSmallM : kMaxBlocksLargeM; }

size_t norms_stage_offset(int M) {
    size_t partial_bytes = (size_t)max_blocks_for(M) * (size_t)M * sizeof(double);
    return kHeaderBytes + partial_bytes;
}

size_t workspace_bytes(int M) {
    return norms_stage_offset(M) + (((size_t)M * sizeof(float) + 255) / 256) * 256;
}

bool finite_all(std::initializer_list<float> vals) {
    for (float f : vals)
        if (!std::isfinite(f)) return false;
    return true;
}

bool aligned128(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 127u) == 0; }

bool overlap(const void *a, size_t abytes, const void *b, size_t bbytes) {
    uintptr_t pa = reinterpret_cast<uintptr_t>(a), pb = reinterpret_cast<uintptr_t>(b);
    return pa < pb + bbytes && pb < pa + abytes;
}

int check_layout(const void *x, int M, int64_t d, int64_t ld) {
    if (!x || M < 1 || M > DPPF_MAX_WORKERS || d < 1 || ld < d) return DPPF_ERR_INVALID_ARG;
    if (ld > (int64_t)1 << 40) return DPPF_ERR_INVALID_ARG;
    if (ld % 32 != 0 || !aligned128(x)) return DPPF_ERR_ALIGNMENT;
    return DPPF_OK;
}

// Per-(M, kernel kind) resident blocks per SM, cached per device.
std::atomic<int> g_occ[64][kMaxTemplateM + 1][3];   // kind 0/1: register kernels, 2: staged

template <typename K>
int blocks_per_sm(K kernel, int dev, int M, int kind, int threads, size_t dyn_smem) {
    int n = g_occ[dev][M][kind].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, dyn_smem) != cudaSuccess || n <= 0)
            return -1;
        g_occ[dev][M][kind].store(n, std::memory_order_relaxed);
    }
    return n;
}

template <int M>
int launch_round_m(RoundArgs a, bool fused, int path, int dev, cudaStream_t s) {
    if (path == DPPF_PATH_STAGED && !fused && coop_supported(dev)) {
        constexpr size_t smem = StagedShape<M>::kSmemBytes;
        if (g_occ[dev][M][2].load(std::memory_order_relaxed) == 0 &&
            cudaFuncSetAttribute(round_kernel_staged<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess) {
            cudaGetLastError();
            return DPPF_ERR_CUDA;
        }
        if (blocks_per_sm(round_kernel_staged<M>, dev, M, 2, kStagedThreads, smem) >= 1) {
            const int sms = sm_count(dev);
            if (sms <= 0) return DPPF_ERR_CUDA;
            const long long nchunks = (a.nvec * 4 + StagedShape<M>::kChunk - 1) / StagedShape<M>::kChunk;
            long long grid = sms;                       // one block per SM
            if (grid > nchunks) grid = nchunks;
            if (grid < 1) grid = 1;
            void *params[] = {&a};
            if (cudaLaunchCooperativeKernel((const void *)round_kernel_staged<M>, dim3((unsigned)grid),
                                            dim3(kStagedThreads), params, smem, s) != cudaSuccess) {
                cudaGetLastError();
                return DPPF_ERR_CUDA;
            }
            return DPPF_OK;
        }
        path = DPPF_PATH_COOPERATIVE;                   // ring does not fit: register kernel instead
    }
    if (path == DPPF_PATH_STAGED) path = DPPF_PATH_COOPERATIVE;
    constexpr int T = Tuning<M>::kThreads;
    // grid never exceeds the tile count of the pass with the largest tiles
    const int u_a = fused ? Tuning<M>::kUnrollFused : Tuning<M>::kUnrollA;
    const int u_b = fused ? Tuning<M>::kUnrollBFused : Tuning<M>::kUnrollB;
    const long long tile_vecs = (long long)T * (u_a > u_b ? u_a : u_b);
    long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (ntiles < 1) ntiles = 1;
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;

    // Both schedules use the same grid (the tuned blocks per SM, never more than the
    // persistent kernel can keep resident), so they split the sum of squares into the same
    // per-block partials and give bit-identical results.
    int per_sm = fused ? blocks_per_sm(round_kernel<M, true>, dev, M, 1, T, 0)
                       : blocks_per_sm(round_kernel<M, false>, dev, M, 0, T, 0);
    if (per_sm <= 0) return DPPF_ERR_CUDA;
    const int tuned = fused ? Tuning<M>::kBlocksPerSMFused : Tuning<M>::kBlocksPerSM;
    if (per_sm > tuned) per_sm = tuned;
    long long grid = (long long)sms * per_sm;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM) grid = kMaxBlocksSmallM;

    if (path == DPPF_PATH_COOPERATIVE && coop_supported(dev)) {
        void *params[] = {&a};
        const void *fn = fused ? (const void *)round_kernel<M, true> : (const void *)round_kernel<M, false>;
        if (cudaLaunchCooperativeKernel(fn, dim3((unsigned)grid), dim3(T), params, 0, s) != cudaSuccess) {
            cudaGetLastError();
            return DPPF_ERR_CUDA;
        }
        return DPPF_OK;
    }
    if (fused) {
        distance_kernel<M, true><<<(unsigned)grid, T, 0, s>>>(a);
        update_kernel<M, true><<<(unsigned)grid, T, 0, s>>>(a, (int)grid);
    } else {
        distance_kernel<M, false><<<(unsigned)grid, T, 0, s>>>(a);
        update_kernel<M, false><<<(unsigned)grid, T, 0, s>>>(a, (int)grid);
    }
    if (cudaGetLastError() != cudaSuccess) return DPPF_ERR_CUDA;
    return DPPF_OK;
}

int launch_round_generic(RoundArgs a, bool fused, int dev, cudaStream_t s) {
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    long long ntiles = (a.nvec + kThreads - 1) / kThreads;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * 2;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksLargeM) grid = kMaxBlocksLargeM;
    const size_t smem_a = (size_t)kWarps * a.M * sizeof(float), smem_b = (size_t)a.M * sizeof(float);
    if (smem_a > 48 * 1024) {
        cudaError_t e = fused ? cudaFuncSetAttribute(distance_kernel_generic<true>,
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_a)
                              : cudaFuncSetAttribute(distance_kernel_generic<false>,
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_a);
        if (e != cudaSuccess) return DPPF_ERR_CUDA;
    }
    if (fused) distance_kernel_generic<true><<<(unsigned)grid, kThreads, smem_a, s>>>(a);
    else distance_kernel_generic<false><<<(unsigned)grid, kThreads, smem_a, s>>>(a);
    update_kernel_generic<<<(unsigned)grid, kThreads, smem_b, s>>>(a, (int)grid);
    if (cudaGetLastError() != cudaSuccess) return DPPF_ERR_CUDA;
    return DPPF_OK;
}

int launch_local_step(float *x, float *v, const float *g, int M, int64_t d, int64_t ld, float lr, float mu,
                      float wd, int dev, cudaStream_t s) {
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    const long long nvec = d / 4;
    long long bx = (nvec + kThreads - 1) / kThreads;
    const long long cap = ((long long)sms * 4 + M - 1) / M;   // about four blocks per SM over all rows
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    local_step_kernel<<<dim3((unsigned)bx, (unsigned)M), kThreads, 0, s>>>(x, v, g, d, ld, nvec, lr, mu, wd);
    if (cudaGetLastError() != cudaSuccess) return DPPF_ERR_CUDA;
    return DPPF_OK;
}

int resolve_path(int path, int M, bool fused) {
    if (M > kMaxTemplateM) return DPPF_PATH_TWO_KERNEL;
    if (fused && path == DPPF_PATH_STAGED) return DPPF_PATH_COOPERATIVE;   // no staged kernel with the local step
    // one launch per round; staging through shared memory pays off up to eight rows
    if (path == DPPF_PATH_AUTO) return (fused || M > 8) ? DPPF_PATH_COOPERATIVE : DPPF_PATH_STAGED;
    return path;
}

int run_round(float *x, float *v, const float *g, int M, int64_t d, int64_t ld, float lr, float mu, float wd,
              float alpha, float lambda, float *norms_out, void *ws, size_t ws_bytes, int path, bool fused,
              cudaStream_t s) {
    int rc = check_layout(x, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (path != DPPF_PATH_AUTO && path != DPPF_PATH_TWO_KERNEL && path != DPPF_PATH_COOPERATIVE &&
        path != DPPF_PATH_STAGED)
        return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    const size_t bytes = (size_t)M * (size_t)ld * sizeof(float);
    if (fused) {
        if ((rc = check_layout(v, M, d, ld)) != DPPF_OK) return rc;
        if ((rc = check_layout(g, M, d, ld)) != DPPF_OK) return rc;
        if (!finite_all({lr, mu, wd})) return DPPF_ERR_INVALID_ARG;
        if (overlap(x, bytes, v, bytes) || overlap(x, bytes, g, bytes) || overlap(v, bytes, g, bytes)) return DPPF_ERR_INVALID_ARG;
    }
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    if (overlap(x, bytes, ws, workspace_bytes(M))) return DPPF_ERR_INVALID_ARG;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;

    RoundArgs a;
    a.x = x; a.v = v; a.g = g;
    a.d = d; a.ld = ld; a.nvec = d / 4;
    a.alpha = alpha; a.lambda = lambda; a.lr = lr; a.mu = mu; a.wd = wd;
    a.norms_out = norms_out;
    a.hdr = reinterpret_cast<WsHeader *>(ws);
    a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
    a.norms_stage = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + norms_stage_offset(M));
    a.M = M;

    if (M == 1) {   // x_A == x_1: distance 0, replica unchanged
        if (fused && (rc = launch_local_step(x, v, g, M, d, ld, lr, mu, wd, dev, s)) != DPPF_OK) return rc;
        zero_norms_kernel<<<1, 32, 0, s>>>(norms_out, a.norms_stage, a.hdr);
        return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
    }
    path = resolve_path(path, M, fused);
    switch (M) {
#define DPPF_CASE(MM) case MM: return launch_round_m<MM>(a, fused, path, dev, s);
        DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: return launch_round_generic(a, fused, dev, s);
    }
}

// ---------------------------------------------------------------- built-in scratch
// Scratch for dppf_consensus_static: one workspace image (header, per-block partial sums for
// up to DPPF_STATIC_MAX_WORKERS workers, distance staging) that lives in the module's own
// global memory.  Each GPU that loads the library carries these bytes until the process ends.
constexpr size_t kStaticWsBytes =
    kHeaderBytes + (size_t)kMaxBlocksSmallM * DPPF_STATIC_MAX_WORKERS * sizeof(double) + 256;
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

// Device address of g_static_ws on each device.  In host code the name g_static_ws is only a
// handle for the runtime, not an address a kernel can use; the real address comes from
// cudaGetSymbolAddress, asked once per device while that device is current.
std::atomic<void *> g_static_ws_addr[64];

int static_ws_address(int dev, void **out) {
    void *p = g_static_ws_addr[dev].load(std::memory_order_acquire);
    if (p == nullptr) {
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return DPPF_ERR_CUDA;
        }
        g_static_ws_addr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return DPPF_OK;
}


// ---------------------------------------------------------------- general round: host side
std::atomic<int> g_general_ready[64][kMaxTemplateM + 1];

template <int M>
int launch_general_m(const GeneralArgs &a, int dev, cudaStream_t s) {
    if (!coop_supported(dev)) return DPPF_ERR_CUDA;
    constexpr size_t smem = StagedShape<M>::kSmemBytes;
    if (g_general_ready[dev][M].load(std::memory_order_relaxed) == 0) {
        if (cudaFuncSetAttribute(general_round_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess) {
            cudaGetLastError();
            return DPPF_ERR_CUDA;
        }
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, general_round_kernel<M>, kGeneralThreads, smem) !=
                cudaSuccess || n < 1)
            return DPPF_ERR_CUDA;
        g_general_ready[dev][M].store(1, std::memory_order_relaxed);
    }
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    const long long nchunks = (a.nvec * 4 + StagedShape<M>::kChunk - 1) / StagedShape<M>::kChunk;
    long long grid = sms;
    if (grid > nchunks) grid = nchunks;
    if (grid < 1) grid = 1;
    GeneralArgs args = a;
    void *params[] = {&args};
    if (cudaLaunchCooperativeKernel((const void *)general_round_kernel<M>, dim3((unsigned)grid),
                                    dim3(kGeneralThreads), params, smem, s) != cudaSuccess) {
        cudaGetLastError();
        return DPPF_ERR_CUDA;
    }
    return DPPF_OK;
}


// ---------------------------------------------------------------- AdamW: host side
int make_adam_args(float *m1, float *m2, const float *g, float lr, float beta1, float beta2, float eps, float wd,
                   int step, AdamArgs *out) {
    if (!finite_all({lr, beta1, beta2, eps, wd}) || step < 1) return DPPF_ERR_INVALID_ARG;
    if (!(beta1 >= 0.f && beta1 < 1.f && beta2 >= 0.f && beta2 < 1.f)) return DPPF_ERR_INVALID_ARG;
    const double bc1 = 1.0 - std::pow((double)beta1, (double)step);
    const double bc2 = 1.0 - std::pow((double)beta2, (double)step);
    out->m1 = m1; out->m2 = m2; out->g = g;
    out->decay = (float)(1.0 - (double)lr * (double)wd);
    out->one_minus_b1 = (float)(1.0 - (double)beta1);
    out->b2 = beta2;
    out->one_minus_b2 = (float)(1.0 - (double)beta2);
    out->step_size = (float)((double)lr / bc1);
    out->inv_sqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
    out->eps = eps;
    return DPPF_OK;
}

int check_adam_buffers(const float *x, const float *m1, const float *m2, const float *g, int M, int64_t d, int64_t ld) {
    int rc;
    if ((rc = check_layout(x, M, d, ld)) != DPPF_OK) return rc;
    if ((rc = check_layout(m1, M, d, ld)) != DPPF_OK) return rc;
    if ((rc = check_layout(m2, M, d, ld)) != DPPF_OK) return rc;
    if ((rc = check_layout(g, M, d, ld)) != DPPF_OK) return rc;
    const size_t bytes = (size_t)M * (size_t)ld * sizeof(float);
    const void *bufs[4] = {x, m1, m2, g};
    for (int i = 0; i < 4; ++i)
        for (int j = i + 1; j < 4; ++j)
            if (overlap(bufs[i], bytes, bufs[j], bytes)) return DPPF_ERR_INVALID_ARG;
    return DPPF_OK;
}

int launch_adamw_step(float *x, const AdamArgs &p, int M, int64_t d, int64_t ld, int dev, cudaStream_t s) {
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    const long long nvec = d / 4;
    long long bx = (nvec + kThreads - 1) / kThreads;
    const long long cap = ((long long)sms * 3 + M - 1) / M;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    adamw_step_kernel<<<dim3((unsigned)bx, (unsigned)M), kThreads, 0, s>>>(x, p, d, ld, nvec);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
}

template <int M>
int launch_adamw_round_m(const RoundArgs &a, const AdamArgs &p, int dev, cudaStream_t s) {
    constexpr int T = Tuning<M>::kThreads;
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    const long long tile_vecs = (long long)T * Tuning<M>::kUnrollB;
    long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * Tuning<M>::kBlocksPerSM;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM) grid = kMaxBlocksSmallM;
    adamw_distance_kernel<M><<<(unsigned)grid, T, 0, s>>>(a, p);
    update_kernel<M, false><<<(unsigned)grid, T, 0, s>>>(a, (int)grid);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
}

}  // namespace

// ---------------------------------------------------------------- C ABI

extern "C" {

size_t dppf_workspace_bytes(int M, int64_t d) {
    if (M < 1 || M > DPPF_MAX_WORKERS || d < 1) return 0;
    return workspace_bytes(M);
}

int dppf_consensus_ex(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, float *norms_out,
                      void *ws, size_t ws_bytes, int path, void *cuda_stream) {
    return run_round(x, nullptr, nullptr, M, d, ld, 0.f, 0.f, 0.f, alpha, lambda, norms_out, ws, ws_bytes, path,
                     false, static_cast<cudaStream_t>(cuda_stream));
}

int dppf_consensus(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, float *norms_out, void *ws,
                   size_t ws_bytes, void *cuda_stream) {
    return dppf_consensus_ex(x, M, d, ld, alpha, lambda, norms_out, ws, ws_bytes, DPPF_PATH_AUTO, cuda_stream);
}

int dppf_local_step(float *x, float *v, const float *g, int M, int64_t d, int64_t ld, float lr, float momentum,
                    float weight_decay, void *cuda_stream) {
    int rc;
    if ((rc = check_layout(x, M, d, ld)) != DPPF_OK) return rc;
    if ((rc = check_layout(v, M, d, ld)) != DPPF_OK) return rc;
    if ((rc = check_layout(g, M, d, ld)) != DPPF_OK) return rc;
    if (!finite_all({lr, momentum, weight_decay})) return DPPF_ERR_INVALID_ARG;
    const size_t bytes = (size_t)M * (size_t)ld * sizeof(float);
    if (overlap(x, bytes, v, bytes) || overlap(x, bytes, g, bytes) || overlap(v, bytes, g, bytes)) return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    return launch_local_step(x, v, g, M, d, ld, lr, momentum, weight_decay, dev,
                             static_cast<cudaStream_t>(cuda_stream));
}

int dppf_local_step_and_consensus_ex(float *x, float *v, const float *g, int M, int64_t d, int64_t ld, float lr,
                                     float momentum, float weight_decay, float alpha, float lambda,
                                     float *norms_out, void *ws, size_t ws_bytes, int path, void *cuda_stream) {
    return run_round(x, v, g, M, d, ld, lr, momentum, weight_decay, alpha, lambda, norms_out, ws, ws_bytes, path,
                     true, static_cast<cudaStream_t>(cuda_stream));
}

int dppf_local_step_and_consensus(float *x, float *v, const float *g, int M, int64_t d, int64_t ld, float lr,
                                  float momentum, float weight_decay, float alpha, float lambda, float *norms_out,
                                  void *ws, size_t ws_bytes, void *cuda_stream) {
    return dppf_local_step_and_consensus_ex(x, v, g, M, d, ld, lr, momentum, weight_decay, alpha, lambda,
                                            norms_out, ws, ws_bytes, DPPF_PATH_AUTO, cuda_stream);
}

int dppf_consensus_host(float *x_host, int M, int64_t d, int64_t ld, float alpha, float lambda, float *norms_host,
                        float *x_dev, void *ws, size_t ws_bytes, void *cuda_stream) {
    if (!x_host) return DPPF_ERR_INVALID_ARG;
    int rc = check_layout(x_dev, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t pitch = (size_t)ld * sizeof(float), width = (size_t)d * sizeof(float);
    if (cudaMemcpy2DAsync(x_dev, pitch, x_host, pitch, width, (size_t)M, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return DPPF_ERR_CUDA;
    rc = dppf_consensus(x_dev, M, d, ld, alpha, lambda, nullptr, ws, ws_bytes, cuda_stream);
    if (rc != DPPF_OK) return rc;
    if (cudaMemcpy2DAsync(x_host, pitch, x_dev, pitch, width, (size_t)M, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return DPPF_ERR_CUDA;
    if (norms_host) {
        const float *stage =
            reinterpret_cast<const float *>(static_cast<unsigned char *>(ws) + norms_stage_offset(M));
        if (cudaMemcpyAsync(norms_host, stage, (size_t)M * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return DPPF_ERR_CUDA;
    }
    return DPPF_OK;
}

int dppf_device_status(const void *ws, void *cuda_stream) {
    if (!ws) return DPPF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    int status = DPPF_OK;
    if (cudaMemcpyAsync(&status, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return DPPF_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return DPPF_ERR_CUDA;
    return status;
}

const char *dppf_status_string(int status) {
    switch (status) {
        case DPPF_OK: return "DPPF_OK";
        case DPPF_ERR_INVALID_ARG: return "DPPF_ERR_INVALID_ARG";
        case DPPF_ERR_ALIGNMENT: return "DPPF_ERR_ALIGNMENT";
        case DPPF_ERR_WORKSPACE: return "DPPF_ERR_WORKSPACE";
        case DPPF_ERR_CUDA: return "DPPF_ERR_CUDA";
        case DPPF_ERR_TIMEOUT: return "DPPF_ERR_TIMEOUT";
        default: return "DPPF_ERR_UNKNOWN";
    }
}

int dppf_launch_count(int M, int64_t d, int path, int fused) {
    if (M < 1 || M > DPPF_MAX_WORKERS || d < 1) return 0;
    if (M == 1) return fused ? 2 : 1;                       // [local step], zero norms
    return resolve_path(path, M, fused != 0) == DPPF_PATH_TWO_KERNEL ? 2 : 1;
}

int dppf_consensus_static(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, float *norms_out,
                          void *cuda_stream) {
    if (M > DPPF_STATIC_MAX_WORKERS) return DPPF_ERR_WORKSPACE;   // built-in scratch holds 16 workers at most
    if (M < 1) return DPPF_ERR_INVALID_ARG;
    if (workspace_bytes(M) > kStaticWsBytes) return DPPF_ERR_WORKSPACE;
    int rc = check_layout(x, M, d, ld);      // reject bad arguments before any CUDA call
    if (rc != DPPF_OK) return rc;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    void *ws = nullptr;
    if ((rc = static_ws_address(dev, &ws)) != DPPF_OK) return rc;
    return run_round(x, nullptr, nullptr, M, d, ld, 0.f, 0.f, 0.f, alpha, lambda, norms_out, ws, kStaticWsBytes,
                     DPPF_PATH_AUTO, false, static_cast<cudaStream_t>(cuda_stream));
}

int dppf_consensus_general(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, const float *weights_host,
                           int push_from, int two_term, float *norms_out, float *push_norms_out, void *ws,
                           size_t ws_bytes, void *cuda_stream) {
    int rc = check_layout(x, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (M > kMaxTemplateM) return DPPF_ERR_INVALID_ARG;
    if (push_from != DPPF_PUSH_FROM_AVERAGE && push_from != DPPF_PUSH_FROM_CONSENSUS) return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = (size_t)M * (size_t)ld * sizeof(float);
    if (overlap(x, bytes, ws, workspace_bytes(M))) return DPPF_ERR_INVALID_ARG;
    GeneralArgs a;
    double wsum = 0.0;
    for (int m = 0; m < M; ++m) {
        const float w = weights_host ? weights_host[m] : 1.0f;
        if (!std::isfinite(w)) return DPPF_ERR_INVALID_ARG;
        wsum += (double)w;
    }
    if (!(wsum != 0.0) || !std::isfinite(wsum)) return DPPF_ERR_INVALID_ARG;
    for (int m = 0; m < kMaxTemplateM; ++m)
        a.wn[m] = (m < M) ? (float)((double)(weights_host ? weights_host[m] : 1.0f) / wsum) : 0.f;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    a.x = x; a.d = d; a.ld = ld; a.nvec = d / 4;
    a.alpha = alpha; a.lambda = lambda;
    a.push_from_c = (push_from == DPPF_PUSH_FROM_CONSENSUS) ? 1 : 0;
    a.two_term = two_term ? 1 : 0;
    a.norms_out = norms_out; a.push_norms_out = push_norms_out;
    a.hdr = reinterpret_cast<WsHeader *>(ws);
    a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    switch (M) {
#define DPPF_CASE(MM) case MM: return launch_general_m<MM>(a, dev, s);
        DPPF_CASE(1) DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: return DPPF_ERR_INVALID_ARG;
    }
}

int dppf_adamw_step(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M, int64_t d, int64_t ld,
                    float lr, float beta1, float beta2, float eps, float weight_decay, int step, void *cuda_stream) {
    int rc = check_adam_buffers(x, exp_avg, exp_avg_sq, g, M, d, ld);
    if (rc != DPPF_OK) return rc;
    AdamArgs p;
    if ((rc = make_adam_args(exp_avg, exp_avg_sq, g, lr, beta1, beta2, eps, weight_decay, step, &p)) != DPPF_OK) return rc;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    return launch_adamw_step(x, p, M, d, ld, dev, static_cast<cudaStream_t>(cuda_stream));
}

int dppf_adamw_step_and_consensus(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M, int64_t d,
                                  int64_t ld, float lr, float beta1, float beta2, float eps, float weight_decay,
                                  int step, float alpha, float lambda, float *norms_out, void *ws, size_t ws_bytes,
                                  void *cuda_stream) {
    int rc = check_adam_buffers(x, exp_avg, exp_avg_sq, g, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (M > kMaxTemplateM) return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    AdamArgs p;
    if ((rc = make_adam_args(exp_avg, exp_avg_sq, g, lr, beta1, beta2, eps, weight_decay, step, &p)) != DPPF_OK) return rc;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = (size_t)M * (size_t)ld * sizeof(float);
    if (overlap(x, bytes, ws, workspace_bytes(M))) return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    RoundArgs a;
    a.x = x; a.v = nullptr; a.g = g;
    a.d = d; a.ld = ld; a.nvec = d / 4;
    a.alpha = alpha; a.lambda = lambda; a.lr = 0.f; a.mu = 0.f; a.wd = 0.f;
    a.norms_out = norms_out;
    a.hdr = reinterpret_cast<WsHeader *>(ws);
    a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
    a.norms_stage = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + norms_stage_offset(M));
    a.M = M;
    if (M == 1) {
        if ((rc = launch_adamw_step(x, p, M, d, ld, dev, s)) != DPPF_OK) return rc;
        zero_norms_kernel<<<1, 32, 0, s>>>(norms_out, a.norms_stage, a.hdr);
        return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
    }
    switch (M) {
#define DPPF_CASE(MM) case MM: return launch_adamw_round_m<MM>(a, p, dev, s);
        DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: return DPPF_ERR_INVALID_ARG;
    }
}

// ---- host-side scalars of a run (no device work)

float dppf_lambda_schedule(int kind, float lambda, int64_t t, int64_t T) {
    if (kind == DPPF_SCHEDULE_FIXED) return lambda;
    if (T <= 0 || t < 0 || (kind != DPPF_SCHEDULE_DECREASING && kind != DPPF_SCHEDULE_INCREASING))
        return std::nanf("");
    const double c = std::cos(3.14159265358979323846 * (double)t / (double)T);
    const double f = (kind == DPPF_SCHEDULE_DECREASING) ? 0.5 * (1.0 + c) : 0.5 * (1.0 - c);
    return (float)((double)lambda * f);
}

float dppf_lr_cosine(float lr_max, int64_t t, int64_t T) {
    if (T <= 0 || t < 0) return std::nanf("");
    return (float)((double)lr_max * 0.5 * (1.0 + std::cos(3.14159265358979323846 * (double)t / (double)T)));
}

int64_t dppf_qsr_period(int64_t tau_base, float beta, float lr_t) {
    if (tau_base < 1 || !std::isfinite(beta) || !std::isfinite(lr_t) || !(lr_t > 0.f)) return -1;
    const double q = (double)beta / (double)lr_t;
    const double sq = std::floor(q * q);
    if (!(sq < 9.0e18)) return INT64_MAX;
    const int64_t tau = (int64_t)sq;
    return tau > tau_base ? tau : tau_base;
}

int dppf_round_metrics(const float *norms_host, int M, float alpha, float lambda, float *mean_distance,
                       float *pull_strength, float *push_strength) {
    if (!norms_host || M < 1 || !finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    double sum = 0.0;
    for (int m = 0; m < M; ++m) {
        if (!(norms_host[m] >= 0.f)) return DPPF_ERR_INVALID_ARG;
        sum += (double)norms_host[m];
        if (pull_strength) pull_strength[m] = (float)((double)alpha * (double)norms_host[m]);
    }
    if (mean_distance) *mean_distance = (float)(sum / (double)M);
    if (push_strength) *push_strength = lambda;
    return DPPF_OK;
}

}  // extern "C"
