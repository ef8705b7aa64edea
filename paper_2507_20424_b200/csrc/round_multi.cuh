// Several consensus rounds in one persistent launch: the update pass of round k also forms the
// squared distances round k+1 needs.
#pragma once
#include "round_register.cuh"
#include "chunk_ring.cuh"

namespace {

// ---------------------------------------------------------------- n rounds, one launch
// The single-line pull-push update (Sec. 5) applied n times, every round from its own
// pre-round average (proof of Theorem 1, first display).  While the update pass of round k
// holds the M new values of a column in registers, their average and squared deviations are
// per-column functions of exactly those values, so the pass also accumulates the sums of
// squares of round k+1:
//   pass 0        read x once, distances of round 1
//   pass k, k>=1  read x, write the round-k update, distances of round k+1 (not in the last pass)
// n rounds move (1 + 2n) M d 4 bytes instead of 3n M d 4 and need one launch.
// Passes alternate direction over the block's chunks, so each pass starts on what the previous
// one touched last; the newest ring stages are consumed from shared memory (updated values are
// written back into the ring for that).  A block whose chunks all fit in the ring never reloads.
// Between passes: per-block fp64 partials -> grid barrier -> every block adds them in block
// order.  The partials alternate between two buffers, because a fast block may write those of
// pass k+1 while a slow one still adds up pass k.
// A bounded wait that gives up ends the call as in the single-round kernel: the block marks its
// partials negative, everybody meets at the grid barrier, sees the mark and returns together
// (x untouched if that was pass 0, partly updated otherwise).

constexpr int kMaxRoundsPerLaunch = 256;   // lambda of every round travels in the launch arguments

struct RoundsArgs {
    float *x;
    long long d, ld, nvec;
    float alpha;
    int n_rounds;                 // 1 .. kMaxRoundsPerLaunch
    int spin_first, spin_later;   // mbarrier polls before a wait gives up: pass 0 / later passes
    float *norms_all;             // [n_rounds, M] pre-update distances of every round, may be null
    float *norms_stage;           // fp32[M] inside the workspace: distances of the last round
    WsHeader *hdr;
    double *partials;             // two buffers of [grid, M], the second at partials + partials_half
    long long partials_half;
    int schedule;                 // DPPF_PATH_* being launched, recorded in the workspace header
    float lambdas[kMaxRoundsPerLaunch];
};

// One chunk in shared memory: optional update with coefficients c (written to x and, if asked,
// back into the ring), optional accumulation of the squared deviations of the values left behind.
template <int M, bool kUpdate>
__device__ __forceinline__ void chunk_body(float *sb, float *xg /* x + col0 */, long long ld, int cols,
                                           const float *c, bool write_back, bool accumulate, double (&acc)[M]) {
    constexpr int CH = StagedShape<M>::kChunk;
    float part[M];
#pragma unroll
    for (int m = 0; m < M; ++m) part[m] = 0.f;
    for (int q = threadIdx.x * 4; q < cols; q += kStagedThreads * 4) {
        float4 xv[M];
#pragma unroll
        for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
        if (kUpdate) {
            const float4 ebar = shifted_mean<M>(xv);
            const float4 x0 = xv[0];
#pragma unroll
            for (int m = 0; m < M; ++m) {
                if (row_is_written(c[m])) {
                    xv[m] = apply4(xv[m], deviation(xv[m], x0, ebar, m), c[m]);
                    st_keep(xg + m * ld + q, xv[m]);
                }
            }
            if (write_back) {
#pragma unroll
                for (int m = 0; m < M; ++m) *reinterpret_cast<float4 *>(sb + m * CH + q) = xv[m];
            }
        }
        if (accumulate) {
            const float4 ebar = shifted_mean<M>(xv);
#pragma unroll
            for (int m = 0; m < M; ++m) part[m] = sq_acc(part[m], deviation(xv[m], xv[0], ebar, m));
        }
    }
#pragma unroll
    for (int m = 0; m < M; ++m) acc[m] += (double)part[m];
}

template <int M>
__global__ void __launch_bounds__(kStagedThreads, 1) rounds_kernel_staged(const RoundsArgs a) {
    constexpr int kStages = StagedShape<M>::kStages;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long full[kStages];
    __shared__ double s_red[kStagedWarps * M];
    __shared__ float s_c[M];
    const int tid = threadIdx.x;
    ChunkRing<M> ring;
    ring.base[0] = a.x;
    ring.init(smem_raw, full, a.ld, a.nvec);
    const int n = ring.n;

    // tail columns (d % 4 of them) go through the scalar routines, which take the single-round arguments
    RoundArgs tail_args;
    tail_args.x = a.x; tail_args.v = nullptr; tail_args.g = nullptr;
    tail_args.d = a.d; tail_args.ld = a.ld; tail_args.nvec = a.nvec;
    tail_args.alpha = a.alpha; tail_args.lambda = 0.f; tail_args.lr = tail_args.mu = tail_args.wd = 0.f;

    const int R = a.n_rounds;
    for (int p = 0; p <= R; ++p) {
        const bool first = (p == 0), last = (p == R), fwd = !(p & 1);
        double acc[M];
#pragma unroll
        for (int m = 0; m < M; ++m) acc[m] = 0.0;
        int failed;
        if (first) {
            failed = ring_pass<StagedShape<M>::kPrefetchA>(ring, a.spin_first, fwd, 0, [&](float *sb, int k, int) {
                chunk_body<M, false>(sb, nullptr, 0, ring.cols(k), s_c, false, true, acc);
            });
        } else if (last) {
            failed = ring_pass<StagedShape<M>::kPrefetchB>(ring, a.spin_later, fwd, ring.resident(), [&](float *sb, int k, int) {
                chunk_body<M, true>(sb, a.x + ring.col0(k), a.ld, ring.cols(k), s_c, false, false, acc);
            });
        } else {
            failed = ring_pass<StagedShape<M>::kPrefetchB>(ring, a.spin_later, fwd, ring.resident(), [&](float *sb, int k, int i) {
                // chunks this pass handles last are the first of the next pass: keep them current in the ring
                const bool write_back = i >= n - kStages;
                chunk_body<M, true>(sb, a.x + ring.col0(k), a.ld, ring.cols(k), s_c, write_back, true, acc);
                if (write_back) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            });
        }
        if (blockIdx.x == 0 && tid == 0 && !failed) {
            if (!first) tail_update<M>(tail_args, s_c);
            if (!last) {
                float tail[M];
#pragma unroll
                for (int m = 0; m < M; ++m) tail[m] = 0.f;
                tail_distance<M, false>(tail_args, tail);
#pragma unroll
                for (int m = 0; m < M; ++m) acc[m] += (double)tail[m];
            }
        }
        if (last) {
            if (failed && tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;   // x is partly updated
            break;
        }
        double *partials = a.partials + (p & 1) * a.partials_half;
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
                partials[(long long)blockIdx.x * M + tid] = failed ? -1.0 : sum;   // negative = "a wait gave up"
            }
            if (first && blockIdx.x == 0 && tid == 0) {
                a.hdr->status = DPPF_OK;
                a.hdr->magic = kMagic;
                a.hdr->grid = (int)gridDim.x;
                a.hdr->M = M;
                a.hdr->schedule = a.schedule;
            }
        }
        cg::this_grid().sync();

        // every block: did any block give up?  (same answer everywhere)
        {
            int bad = 0;
            for (int i = tid; i < (int)gridDim.x * M; i += kStagedThreads) bad |= (__ldcg(partials + i) < 0.0) ? 1 : 0;
            if (__syncthreads_or(bad)) {
                if (blockIdx.x == 0 && tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;
                return;
            }
        }
        // distances and coefficients of round p + 1, identical in every block
        {
            const int lane = tid & 31, warp = tid >> 5;
            for (int m = warp; m < M; m += kStagedWarps) {
                double s = 0.0;
                for (int b = lane; b < (int)gridDim.x; b += 32) s += __ldcg(partials + (long long)b * M + m);
                s = warp_sum(s);
                if (lane == 0) {
                    float r;
                    s_c[m] = coefficient(s, a.alpha, a.lambdas[p], &r);
                    if (blockIdx.x == 0) {
                        if (p == R - 1) a.norms_stage[m] = r;
                        if (a.norms_all) a.norms_all[(long long)p * M + m] = r;
                    }
                }
            }
            __syncthreads();
        }
    }
}

// ---------------------------------------------------------------- n rounds, register-resident
// Same schedule of passes with 128-bit loads straight into registers, for when the ring cannot
// be used.  Per-thread fp32 sums per pass, fp64 from the warp upwards.
template <int M, int U, bool kUpdate>
__device__ __forceinline__ void register_pass(const RoundsArgs &a, const float *c, bool fwd, bool accumulate,
                                              float (&acc)[M]) {
    constexpr int T = Tuning<M>::kThreads;
    const long long tile_vecs = (long long)T * U;
    const long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    const long long nloc = (ntiles > blockIdx.x) ? (ntiles - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    for (long long i = 0; i < nloc; ++i) {
        const long long t = blockIdx.x + (fwd ? i : nloc - 1 - i) * gridDim.x;
        float4 xv[U][M];
        bool live[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long j = (t * U + u) * T + threadIdx.x;
            live[u] = j < a.nvec;
            if (live[u]) {
#pragma unroll
                for (int m = 0; m < M; ++m)
                    xv[u][m] = kUpdate ? ld_last_use(a.x + m * a.ld + j * 4) : ld_keep(a.x + m * a.ld + j * 4);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (live[u]) {
                const long long j = (t * U + u) * T + threadIdx.x;
                if (kUpdate) {
                    const float4 ebar = shifted_mean<M>(xv[u]);
                    const float4 x0 = xv[u][0];
#pragma unroll
                    for (int m = 0; m < M; ++m)
                        if (row_is_written(c[m])) {
                            xv[u][m] = apply4(xv[u][m], deviation(xv[u][m], x0, ebar, m), c[m]);
                            st_keep(a.x + m * a.ld + j * 4, xv[u][m]);
                        }
                }
                if (accumulate) {
                    const float4 ebar = shifted_mean<M>(xv[u]);
#pragma unroll
                    for (int m = 0; m < M; ++m) acc[m] = sq_acc(acc[m], deviation(xv[u][m], xv[u][0], ebar, m));
                }
            }
        }
    }
}

template <int M>
__global__ void __launch_bounds__(Tuning<M>::kThreads, Tuning<M>::kBlocksPerSM) rounds_kernel(const RoundsArgs a) {
    __shared__ double s_red[Tuning<M>::kWarps * M];
    __shared__ float s_c[M];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    RoundArgs tail_args;
    tail_args.x = a.x; tail_args.v = nullptr; tail_args.g = nullptr;
    tail_args.d = a.d; tail_args.ld = a.ld; tail_args.nvec = a.nvec;
    tail_args.alpha = a.alpha; tail_args.lambda = 0.f; tail_args.lr = tail_args.mu = tail_args.wd = 0.f;
    const int R = a.n_rounds;
    for (int p = 0; p <= R; ++p) {
        const bool first = (p == 0), last = (p == R), fwd = !(p & 1);
        float acc[M];
#pragma unroll
        for (int m = 0; m < M; ++m) acc[m] = 0.f;
        if (first) register_pass<M, Tuning<M>::kUnrollA, false>(a, s_c, fwd, true, acc);
        else register_pass<M, Tuning<M>::kUnrollB, true>(a, s_c, fwd, !last, acc);
        if (blockIdx.x == 0 && tid == 0) {
            if (!first) tail_update<M>(tail_args, s_c);
            if (!last) tail_distance<M, false>(tail_args, acc);
        }
        if (last) break;
        double *partials = a.partials + (p & 1) * a.partials_half;
#pragma unroll
        for (int m = 0; m < M; ++m) {
            double s = warp_sum((double)acc[m]);
            if (lane == 0) s_red[warp * M + m] = s;
        }
        __syncthreads();
        if (tid < M) {
            double s = 0.0;
            for (int w = 0; w < Tuning<M>::kWarps; ++w) s += s_red[w * M + tid];
            partials[(long long)blockIdx.x * M + tid] = s;
        }
        if (first && blockIdx.x == 0 && tid == 0) {
            a.hdr->status = DPPF_OK;
            a.hdr->magic = kMagic;
            a.hdr->grid = (int)gridDim.x;
            a.hdr->M = M;
            a.hdr->schedule = a.schedule;
        }
        cg::this_grid().sync();
        for (int m = warp; m < M; m += Tuning<M>::kWarps) {
            double s = 0.0;
            for (int b = lane; b < (int)gridDim.x; b += 32) s += __ldcg(partials + (long long)b * M + m);
            s = warp_sum(s);
            if (lane == 0) {
                float r;
                s_c[m] = coefficient(s, a.alpha, a.lambdas[p], &r);
                if (blockIdx.x == 0) {
                    if (p == R - 1) a.norms_stage[m] = r;
                    if (a.norms_all) a.norms_all[(long long)p * M + m] = r;
                }
            }
        }
        __syncthreads();
    }
}

}  // namespace
