// One worker's share of a round when every GPU holds ONE replica (the paper's own deployment).
#pragma once
#include "round_register.cuh"

namespace {

// ---------------------------------------------------------------- worker-per-GPU round
// In Algorithm 1 each worker obtains the consensus variable with one collective per round and
// then pulls and pushes its own replica.  Given this worker's x[d] and the all-reduced
// parameters (x_A = scale * reduced, scale = 1/M after a sum, 1 after a mean), the kernel
// measures r = ||x - x_A|| and applies the single-line update of Sec. 5,
//   x <- x + (x_A - x)(alpha - lambda / r),
// in one cooperative launch: distance pass, grid barrier, update pass (5 d 4 bytes: x and
// the reduced vector are read twice, x is written once).  r == 0 leaves x untouched.
// Arguments travel in a RoundArgs: x = the replica, g = the reduced vector, lr = scale, M = 1.
constexpr int kWorkerThreads = 256;
constexpr int kWorkerBlocksPerSM = 3;
constexpr int kWorkerUnroll = 2;

__device__ __forceinline__ float4 worker_deviation(float4 x, float4 red, float scale) {
    return sub4(x, scale4(red, scale));                               // x - x_A
}

__device__ __forceinline__ void worker_distance_pass(const RoundArgs &a, double *s_red) {
    constexpr int T = kWorkerThreads, U = kWorkerUnroll;
    const long long tile_vecs = (long long)T * U;
    const long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    float acc = 0.f;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
        float4 xv[U], rv[U];
        bool live[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long j = (t * U + u) * T + threadIdx.x;
            live[u] = j < a.nvec;
            if (live[u]) {
                xv[u] = ld_keep(a.x + j * 4);
                rv[u] = ld_keep(a.g + j * 4);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (live[u]) acc = sq_acc(acc, worker_deviation(xv[u], rv[u], a.lr));
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (long long i = a.nvec * 4; i < a.d; ++i) {
            const float dv = __fsub_rn(a.x[i], __fmul_rn(a.g[i], a.lr));
            acc = __fmaf_rn(dv, dv, acc);
        }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const double s = warp_sum((double)acc);
    if (lane == 0) s_red[warp] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double sum = 0.0;
        for (int w = 0; w < kWorkerThreads / 32; ++w) sum += s_red[w];
        a.partials[blockIdx.x] = sum;
        if (blockIdx.x == 0) {
            a.hdr->status = DPPF_OK;
            a.hdr->magic = kMagic;
            a.hdr->grid = (int)gridDim.x;
            a.hdr->M = 1;
            a.hdr->schedule = a.schedule;
        }
    }
}

__device__ __forceinline__ void worker_update_pass(const RoundArgs &a, float c) {
    constexpr int T = kWorkerThreads, U = kWorkerUnroll;
    const long long tile_vecs = (long long)T * U;
    const long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (!row_is_written(c)) return;                                   // zero distance: replica unchanged
    if (ntiles > blockIdx.x) {
        long long t = blockIdx.x + (ntiles - 1 - blockIdx.x) / gridDim.x * gridDim.x;
        for (; t >= 0; t -= gridDim.x) {
            float4 xv[U], rv[U];
            bool live[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long j = (t * U + u) * T + threadIdx.x;
                live[u] = j < a.nvec;
                if (live[u]) {
                    xv[u] = ld_last_use(a.x + j * 4);
                    rv[u] = ld_last_use(a.g + j * 4);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (live[u]) {
                    const long long j = (t * U + u) * T + threadIdx.x;
                    st_keep(a.x + j * 4, apply4(xv[u], worker_deviation(xv[u], rv[u], a.lr), c));
                }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (long long i = a.nvec * 4; i < a.d; ++i) {
            const float dv = __fsub_rn(a.x[i], __fmul_rn(a.g[i], a.lr));
            a.x[i] = __fmaf_rn(-c, dv, a.x[i]);
        }
}

// One persistent cooperative launch.
__global__ void __launch_bounds__(kWorkerThreads, kWorkerBlocksPerSM) worker_round_kernel(const RoundArgs a) {
    __shared__ double s_red[kWorkerThreads / 32];
    __shared__ float s_c[1];
    __shared__ int s_ok;
    worker_distance_pass(a, s_red);
    cg::this_grid().sync();
    if (!finalise(a, 1, (int)gridDim.x, s_c, &s_ok)) return;
    worker_update_pass(a, s_c[0]);
}

// Two-launch schedule (when a cooperative launch is refused).
__global__ void __launch_bounds__(kWorkerThreads, kWorkerBlocksPerSM) worker_distance_kernel(const RoundArgs a) {
    __shared__ double s_red[kWorkerThreads / 32];
    worker_distance_pass(a, s_red);
}
__global__ void __launch_bounds__(kWorkerThreads, kWorkerBlocksPerSM) worker_update_kernel(const RoundArgs a, int nblocks_a) {
    __shared__ float s_c[1];
    __shared__ int s_ok;
    if (!finalise(a, 1, nblocks_a, s_c, &s_ok)) return;
    worker_update_pass(a, s_c[0]);
}

}  // namespace
