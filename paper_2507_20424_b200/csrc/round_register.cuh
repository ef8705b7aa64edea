// Register-resident round kernels (M <= 16): distance pass, finalise, update pass; two-launch and cooperative schedules.
#pragma once
#include "common.cuh"

namespace {

// ---------------------------------------------------------------- register-resident kernels (M <= 16)

// Launch shape per worker count, from sweeps on B200.  The update pass mixes reads and
// writes and is fastest with about 40-48 KB of loads in flight per SM; more outstanding
// requests lower its DRAM efficiency, fewer cannot cover the latency.  The read-only distance
// pass wants about twice that, which it gets from a deeper unroll on the same grid.
//   bytes in flight per SM = kThreads * kBlocksPerSM * unroll * M * 16
template <int M>
struct Tuning {
    static constexpr int kThreads =
        (M <= 2) ? 320 : (M == 3) ? 384 : (M == 4) ? 320 : (M == 5) ? 256 : (M == 6) ? 224 :
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
        a.hdr->schedule = a.schedule;
    }
}

// Cross-block sum in block order, identical in every block; fills s_c[M] and reports r_m.
// Returns false if the workspace header does not describe this launch.  With a.hdr == nullptr
// the partials are the caller's own M sums (nblocks == 1) and there is no header to check.
__device__ __forceinline__ bool finalise(const RoundArgs &a, int M, int nblocks, float *s_c, int *s_ok) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0)
        *s_ok = (!a.hdr || (a.hdr->magic == kMagic && a.hdr->grid == nblocks && a.hdr->M == M)) ? 1 : 0;
    const int nwarps = blockDim.x >> 5;
    for (int m = warp; m < M; m += nwarps) {
        double s = 0.0;
        for (int b = lane; b < nblocks; b += 32) s += __ldcg(a.partials + (long long)b * M + m);
        s = warp_sum(s);
        if (lane == 0) {
            float r;
            s_c[m] = coefficient(s, a.alpha, a.lambda, &r);
            if (blockIdx.x == 0) {
                if (a.norms_stage) a.norms_stage[m] = r;
                if (a.norms_out) a.norms_out[m] = r;
            }
        }
    }
    __syncthreads();
    if (!*s_ok && blockIdx.x == 0 && threadIdx.x == 0) a.hdr->status = DPPF_ERR_WORKSPACE;
    return *s_ok != 0;
}

template <int M, int U, int T = Tuning<M>::kThreads>
__device__ __forceinline__ void update_pass(const RoundArgs &a, const float *s_c) {
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

// Per-worker totals of the per-block partial sums, in block order (the order finalise uses):
// what a column shard contributes to the squared distances.  One block of up to 16 warps.
__global__ void sum_partials_kernel(const double *partials, int nblocks, int M, double *sums_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int m = warp; m < M; m += nwarps) {
        double s = 0.0;
        for (int b = lane; b < nblocks; b += 32) s += __ldcg(partials + (long long)b * M + m);
        s = warp_sum(s);
        if (lane == 0) sums_out[m] = s;
    }
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

}  // namespace
