// DPPF consensus round for one B200 (sm_100a): host side and the C ABI of include/dppf.h.
// Kernels live in the .cuh files included below (one translation unit):
//   common.cuh          constants, argument structs, cache-hinted accesses, rounded arithmetic
//   round_register.cuh  register-resident round kernels (two-launch and cooperative schedules)
//   adamw.cuh           AdamW local step, stand-alone and fused into the distance pass
//   chunk_ring.cuh      shared-memory chunk ring of the staged kernels (bulk async copies, bounded waits)
//   round_staged.cuh    staged persistent round kernel, one round per launch
//   round_multi.cuh     several rounds in one launch (update pass of round k + distances of round k+1)
//   round_fused_staged.cuh  SGD-momentum local step + round, x, v, g staged through shared memory
//   round_general.cuh   general round (weighted consensus variable, push reference, two-term push)
//   round_generic.cuh   any worker count up to 1024, stand-alone SGD-momentum local step
//   round_worker.cuh    one worker's update from the all-reduced parameters (one replica per GPU)
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

#include "common.cuh"
#include "round_register.cuh"
#include "adamw.cuh"
#include "chunk_ring.cuh"
#include "round_staged.cuh"
#include "round_multi.cuh"
#include "round_fused_staged.cuh"
#include "round_general.cuh"
#include "round_generic.cuh"
#include "round_worker.cuh"

namespace {

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

// Poll limits of the bounded waits of the staged kernels (distance pass / later passes).  Only
// the testing hook dppf_debug_set_poll_limits changes them.
std::atomic<int> g_spin_first{kSpinLimit}, g_spin_later{kSpinLimit};

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

// Bytes from the first element of row 0 to the last element of row M-1 (a column shard of a
// wider buffer ends before its last row's stride does).
size_t extent_bytes(int M, int64_t d, int64_t ld) {
    return ((size_t)(M - 1) * (size_t)ld + (size_t)d) * sizeof(float);
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

std::atomic<int> g_fused_ready[64][9];

// Staged fused round (M <= 8).  DPPF_ERR_CUDA + *refused when it cannot be launched cooperatively.
template <int M>
int launch_fused_staged_m(const RoundArgs &a, int dev, cudaStream_t s, bool *refused) {
    *refused = true;
    if constexpr (M <= 8) {
        using RingA = ChunkRing<M, FusedShape<M>::kArrays, FusedShape<M>::kChunk, FusedShape<M>::kStages>;
        constexpr size_t smem = RingA::kSmemBytes > StagedShape<M>::kSmemBytes ? RingA::kSmemBytes
                                                                               : StagedShape<M>::kSmemBytes;
        const int sms = sm_count(dev);
        if (sms <= 0 || !coop_supported(dev)) return DPPF_ERR_CUDA;
        if (g_fused_ready[dev][M].load(std::memory_order_relaxed) == 0) {
            int n = 0;
            if (cudaFuncSetAttribute(fused_round_kernel_staged<M>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem) != cudaSuccess ||
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fused_round_kernel_staged<M>, kStagedThreads,
                                                              smem) != cudaSuccess || n < 1) {
                cudaGetLastError();
                return DPPF_ERR_CUDA;
            }
            g_fused_ready[dev][M].store(1, std::memory_order_relaxed);
        }
        const long long nchunks = (a.nvec * 4 + RingA::CH - 1) / RingA::CH;
        long long grid = sms;
        if (grid > nchunks) grid = nchunks;
        if (grid < 1) grid = 1;
        RoundArgs aa = a;
        aa.schedule = DPPF_PATH_STAGED;
        void *params[] = {&aa};
        if (cudaLaunchCooperativeKernel((const void *)fused_round_kernel_staged<M>, dim3((unsigned)grid),
                                        dim3(kStagedThreads), params, smem, s) == cudaSuccess) {
            *refused = false;
            return DPPF_OK;
        }
        cudaGetLastError();
    }
    return DPPF_ERR_CUDA;
}

template <int M>
int launch_rounds_m(RoundsArgs &a, int path, int dev, cudaStream_t s, bool *refused);
RoundsArgs one_round_args(const RoundArgs &a);

template <int M>
int launch_round_m(RoundArgs a, bool fused, int path, int dev, cudaStream_t s) {
    if (path == DPPF_PATH_STAGED && fused && M <= 8) {
        bool refused = false;
        const int rc = launch_fused_staged_m<M>(a, dev, s, &refused);
        if (rc == DPPF_OK || !refused) return rc;
        path = DPPF_PATH_COOPERATIVE;
    }
    if (path == DPPF_PATH_STAGED && !fused && M > 8) {
        // above eight rows the multi-round kernel (row copies issued by one lane each) is the faster
        // staged kernel; a single round is its two-pass special case
        RoundsArgs ra = one_round_args(a);
        bool refused = false;
        const int rc = launch_rounds_m<M>(ra, DPPF_PATH_STAGED, dev, s, &refused);
        if (rc == DPPF_OK || !refused) return rc;
        path = DPPF_PATH_TWO_KERNEL;
    }
    if constexpr (M <= 8) if (path == DPPF_PATH_STAGED && !fused && coop_supported(dev)) {
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
            a.schedule = DPPF_PATH_STAGED;
            void *params[] = {&a};
            if (cudaLaunchCooperativeKernel((const void *)round_kernel_staged<M>, dim3((unsigned)grid),
                                            dim3(kStagedThreads), params, smem, s) == cudaSuccess)
                return DPPF_OK;
            cudaGetLastError();                         // e.g. not all blocks can be co-resident right now
            path = DPPF_PATH_TWO_KERNEL;                // (SMs shared with another client): two plain launches
        } else {
            path = DPPF_PATH_COOPERATIVE;               // ring does not fit: register kernel instead
        }
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
        a.schedule = DPPF_PATH_COOPERATIVE;
        void *params[] = {&a};
        const void *fn = fused ? (const void *)round_kernel<M, true> : (const void *)round_kernel<M, false>;
        if (cudaLaunchCooperativeKernel(fn, dim3((unsigned)grid), dim3(T), params, 0, s) == cudaSuccess)
            return DPPF_OK;
        cudaGetLastError();                             // cooperative launch refused: fall back to two launches
    }
    a.schedule = DPPF_PATH_TWO_KERNEL;
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
    a.schedule = DPPF_PATH_TWO_KERNEL;
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
    if (fused && path == DPPF_PATH_STAGED && M > 8) return DPPF_PATH_COOPERATIVE;   // staged fused kernel: M <= 8
    // one launch per round, rows staged through shared memory
    if (path == DPPF_PATH_AUTO) return (fused && M > 8) ? DPPF_PATH_COOPERATIVE : DPPF_PATH_STAGED;
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
    const size_t bytes = extent_bytes(M, d, ld);
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
    a.spin_first = g_spin_first.load(std::memory_order_relaxed);
    a.spin_later = g_spin_later.load(std::memory_order_relaxed);
    a.schedule = DPPF_PATH_TWO_KERNEL;

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

// ---------------------------------------------------------------- the two passes as separate calls
template <int M>
int distance_only_m(const RoundArgs &a, int dev, cudaStream_t s) {
    constexpr int T = Tuning<M>::kThreads;
    const int sms = sm_count(dev);
    if (sms <= 0) return -1;
    const long long tile_vecs = (long long)T * Tuning<M>::kUnrollA;
    long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * Tuning<M>::kBlocksPerSM;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM) grid = kMaxBlocksSmallM;
    distance_kernel<M, false><<<(unsigned)grid, T, 0, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? (int)grid : -1;
}

// Distance pass alone; returns the number of blocks that wrote partial sums, -1 on failure.
int launch_distance_only(const RoundArgs &a, int M, int dev, cudaStream_t s) {
    switch (M) {
#define DPPF_CASE(MM) case MM: return distance_only_m<MM>(a, dev, s);
        DPPF_CASE(1) DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: break;
    }
    const int sms = sm_count(dev);
    if (sms <= 0) return -1;
    long long ntiles = (a.nvec + kThreads - 1) / kThreads;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * 2;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksLargeM) grid = kMaxBlocksLargeM;
    const size_t smem_a = (size_t)kWarps * a.M * sizeof(float);
    if (smem_a > 48 * 1024 &&
        cudaFuncSetAttribute(distance_kernel_generic<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem_a) != cudaSuccess)
        return -1;
    distance_kernel_generic<false><<<(unsigned)grid, kThreads, smem_a, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? (int)grid : -1;
}

template <int M>
int update_only_m(const RoundArgs &a, int dev, cudaStream_t s) {
    constexpr int T = Tuning<M>::kThreads;
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    const long long tile_vecs = (long long)T * Tuning<M>::kUnrollB;
    long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * Tuning<M>::kBlocksPerSM;
    if (grid > ntiles) grid = ntiles;
    update_kernel<M, false><<<(unsigned)grid, T, 0, s>>>(a, 1);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
}

// Update pass alone, from M caller-provided sums of squares (a.partials, a.hdr == nullptr).
int launch_update_only(const RoundArgs &a, int M, int dev, cudaStream_t s) {
    switch (M) {
#define DPPF_CASE(MM) case MM: return update_only_m<MM>(a, dev, s);
        DPPF_CASE(1) DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: break;
    }
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    long long ntiles = (a.nvec + kThreads - 1) / kThreads;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * 2;
    if (grid > ntiles) grid = ntiles;
    update_kernel_generic<<<(unsigned)grid, kThreads, (size_t)a.M * sizeof(float), s>>>(a, 1);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
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


// ---------------------------------------------------------------- several rounds per launch: host side
std::atomic<int> g_rounds_ready[64][kMaxTemplateM + 1][2];   // [][][0] staged, [1] register: blocks per SM

RoundsArgs one_round_args(const RoundArgs &a) {
    RoundsArgs r;
    r.x = a.x; r.d = a.d; r.ld = a.ld; r.nvec = a.nvec;
    r.alpha = a.alpha;
    r.n_rounds = 1;
    r.spin_first = a.spin_first;
    r.spin_later = a.spin_later;
    r.norms_all = a.norms_out;
    r.norms_stage = a.norms_stage;
    r.hdr = a.hdr;
    r.partials = a.partials;
    r.partials_half = (long long)(kMaxBlocksSmallM / 2) * a.M;
    r.lambdas[0] = a.lambda;
    return r;
}

// One launch of up to kMaxRoundsPerLaunch rounds.  DPPF_ERR_CUDA + *refused = true when the
// runtime will not launch cooperatively (caller falls back to single rounds).
template <int M>
int launch_rounds_m(RoundsArgs &a, int path, int dev, cudaStream_t s, bool *refused) {
    *refused = false;
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    if (!coop_supported(dev)) { *refused = true; return DPPF_ERR_CUDA; }
    void *params[] = {&a};
    a.schedule = (path == DPPF_PATH_STAGED) ? DPPF_PATH_STAGED : DPPF_PATH_COOPERATIVE;
    if (path == DPPF_PATH_STAGED) {
        constexpr size_t smem = StagedShape<M>::kSmemBytes;
        if (g_rounds_ready[dev][M][0].load(std::memory_order_relaxed) == 0) {
            int n = 0;
            if (cudaFuncSetAttribute(rounds_kernel_staged<M>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem) != cudaSuccess ||
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, rounds_kernel_staged<M>, kStagedThreads, smem) !=
                    cudaSuccess || n < 1) {
                cudaGetLastError();
                *refused = true;
                return DPPF_ERR_CUDA;
            }
            g_rounds_ready[dev][M][0].store(n, std::memory_order_relaxed);
        }
        const long long nchunks = (a.nvec * 4 + StagedShape<M>::kChunk - 1) / StagedShape<M>::kChunk;
        long long grid = sms;                           // one block per SM
        if (grid > nchunks) grid = nchunks;
        if (grid > kMaxBlocksSmallM / 2) grid = kMaxBlocksSmallM / 2;
        if (grid < 1) grid = 1;
        if (cudaLaunchCooperativeKernel((const void *)rounds_kernel_staged<M>, dim3((unsigned)grid),
                                        dim3(kStagedThreads), params, smem, s) == cudaSuccess)
            return DPPF_OK;
        cudaGetLastError();
        *refused = true;
        return DPPF_ERR_CUDA;
    }
    constexpr int T = Tuning<M>::kThreads;
    int per_sm = g_rounds_ready[dev][M][1].load(std::memory_order_relaxed);
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rounds_kernel<M>, T, 0) != cudaSuccess ||
            per_sm < 1) {
            cudaGetLastError();
            *refused = true;
            return DPPF_ERR_CUDA;
        }
        g_rounds_ready[dev][M][1].store(per_sm, std::memory_order_relaxed);
    }
    if (per_sm > Tuning<M>::kBlocksPerSM) per_sm = Tuning<M>::kBlocksPerSM;
    const int u = Tuning<M>::kUnrollA > Tuning<M>::kUnrollB ? Tuning<M>::kUnrollA : Tuning<M>::kUnrollB;
    long long ntiles = (a.nvec + (long long)T * u - 1) / ((long long)T * u);
    long long grid = (long long)sms * per_sm;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM / 2) grid = kMaxBlocksSmallM / 2;
    if (grid < 1) grid = 1;
    if (cudaLaunchCooperativeKernel((const void *)rounds_kernel<M>, dim3((unsigned)grid), dim3(T), params, 0, s) ==
        cudaSuccess)
        return DPPF_OK;
    cudaGetLastError();
    *refused = true;
    return DPPF_ERR_CUDA;
}

int launch_rounds(RoundsArgs &a, int M, int path, int dev, cudaStream_t s, bool *refused) {
    switch (M) {
#define DPPF_CASE(MM) case MM: return launch_rounds_m<MM>(a, path, dev, s, refused);
        DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: *refused = true; return DPPF_ERR_CUDA;
    }
}

// ---------------------------------------------------------------- general round: host side
std::atomic<int> g_general_ready[64][kMaxTemplateM + 1];

template <int M>
int launch_general_m(const GeneralArgs &a, int path, int dev, cudaStream_t s) {
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    GeneralArgs args = a;
    if (path != DPPF_PATH_TWO_KERNEL && coop_supported(dev)) {
        constexpr size_t smem = StagedShape<M>::kSmemBytes;
        bool ready = g_general_ready[dev][M].load(std::memory_order_relaxed) != 0;
        if (!ready) {
            int n = 0;
            ready = cudaFuncSetAttribute(general_round_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem) == cudaSuccess &&
                    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, general_round_kernel<M>, GeneralShape<M>::kThreads,
                                                                  smem) == cudaSuccess && n >= 1;
            if (ready) g_general_ready[dev][M].store(1, std::memory_order_relaxed);
            else cudaGetLastError();
        }
        if (ready) {
            const long long nchunks = (a.nvec * 4 + StagedShape<M>::kChunk - 1) / StagedShape<M>::kChunk;
            long long grid = sms;
            if (grid > nchunks) grid = nchunks;
            if (grid > kMaxBlocksSmallM / 2) grid = kMaxBlocksSmallM / 2;
            if (grid < 1) grid = 1;
            args.schedule = DPPF_PATH_STAGED;
            void *params[] = {&args};
            if (cudaLaunchCooperativeKernel((const void *)general_round_kernel<M>, dim3((unsigned)grid),
                                            dim3(GeneralShape<M>::kThreads), params, smem, s) == cudaSuccess)
                return DPPF_OK;
            cudaGetLastError();                         // refused (blocks cannot all be resident now): two launches
        }
    }
    constexpr int T = Tuning<M>::kThreads;
    long long ntiles = (a.nvec + T - 1) / T;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * Tuning<M>::kBlocksPerSM;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM / 2) grid = kMaxBlocksSmallM / 2;   // the partials hold 2M sums per block
    args.grid_a = (int)grid;
    args.schedule = DPPF_PATH_TWO_KERNEL;
    general_distance_kernel<M><<<(unsigned)grid, T, 0, s>>>(args);
    general_update_kernel<M><<<(unsigned)grid, T, 0, s>>>(args);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
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
    const size_t bytes = extent_bytes(M, d, ld);
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

std::atomic<int> g_adamw_occ[64][kMaxTemplateM + 1];
std::atomic<int> g_worker_occ[64];

template <int M>
int launch_adamw_round_m(const RoundArgs &a, const AdamArgs &p, int path, int dev, cudaStream_t s) {
    constexpr int T = AdamTuning<M>::kThreads;
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    int per_sm = g_adamw_occ[dev][M].load(std::memory_order_relaxed);
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, adamw_round_kernel<M>, T, 0) != cudaSuccess ||
            per_sm < 1) {
            cudaGetLastError();
            return DPPF_ERR_CUDA;
        }
        g_adamw_occ[dev][M].store(per_sm, std::memory_order_relaxed);
    }
    if (per_sm > AdamTuning<M>::kBlocksPerSM) per_sm = AdamTuning<M>::kBlocksPerSM;
    const long long tile_vecs = (long long)T * AdamTuning<M>::kUnrollB;
    long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (ntiles < 1) ntiles = 1;
    long long grid = (long long)sms * per_sm;            // the same grid for both schedules: same partial sums
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM) grid = kMaxBlocksSmallM;
    if (path != DPPF_PATH_TWO_KERNEL && coop_supported(dev)) {
        RoundArgs aa = a;
        aa.schedule = DPPF_PATH_COOPERATIVE;
        AdamArgs pp = p;
        void *params[] = {&aa, &pp};
        if (cudaLaunchCooperativeKernel((const void *)adamw_round_kernel<M>, dim3((unsigned)grid), dim3(T), params, 0,
                                        s) == cudaSuccess)
            return DPPF_OK;
        cudaGetLastError();                              // refused: two plain launches
    }
    RoundArgs a2 = a;
    a2.schedule = DPPF_PATH_TWO_KERNEL;
    adamw_distance_kernel<M><<<(unsigned)grid, T, 0, s>>>(a2, p);
    adamw_update_kernel<M><<<(unsigned)grid, T, 0, s>>>(a2, (int)grid);
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
    const size_t bytes = extent_bytes(M, d, ld);
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

int dppf_device_schedule(const void *ws, void *cuda_stream) {
    if (!ws) return DPPF_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    WsHeader h;
    if (cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return -1;
    if (cudaStreamSynchronize(s) != cudaSuccess) return -1;
    return h.schedule;
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
    if (fused == 2) return (M > kMaxTemplateM) ? 0 : (path == DPPF_PATH_TWO_KERNEL ? 2 : 1);   // AdamW fused
    return resolve_path(path, M, fused != 0) == DPPF_PATH_TWO_KERNEL ? 2 : 1;
}

// ---- a round split at its reduction (column shards of the replicas on several GPUs)

int dppf_distance_partials(const float *x, int M, int64_t d, int64_t ld, double *sums_out, void *ws,
                           size_t ws_bytes, void *cuda_stream) {
    int rc = check_layout(x, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (!sums_out || (reinterpret_cast<uintptr_t>(sums_out) & 7u)) return DPPF_ERR_INVALID_ARG;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = extent_bytes(M, d, ld);
    if (overlap(x, bytes, ws, workspace_bytes(M)) || overlap(x, bytes, sums_out, (size_t)M * sizeof(double)) ||
        overlap(ws, workspace_bytes(M), sums_out, (size_t)M * sizeof(double)))
        return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    RoundArgs a;
    a.x = const_cast<float *>(x); a.v = nullptr; a.g = nullptr;     // the distance pass only reads x
    a.d = d; a.ld = ld; a.nvec = d / 4;
    a.alpha = 0.f; a.lambda = 0.f; a.lr = a.mu = a.wd = 0.f;
    a.norms_out = nullptr;
    a.hdr = reinterpret_cast<WsHeader *>(ws);
    a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
    a.norms_stage = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + norms_stage_offset(M));
    a.M = M;
    a.spin_first = a.spin_later = kSpinLimit;
    a.schedule = DPPF_PATH_TWO_KERNEL;
    const int grid = launch_distance_only(a, M, dev, s);
    if (grid <= 0) return DPPF_ERR_CUDA;
    const int warps = M < 16 ? M : 16;
    sum_partials_kernel<<<1, 32 * warps, 0, s>>>(a.partials, grid, M, sums_out);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
}

int dppf_update_from_sums(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, const double *sums,
                          float *norms_out, void *cuda_stream) {
    int rc = check_layout(x, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (!sums || (reinterpret_cast<uintptr_t>(sums) & 7u)) return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    const size_t bytes = extent_bytes(M, d, ld);
    if (overlap(x, bytes, sums, (size_t)M * sizeof(double))) return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    RoundArgs a;
    a.x = x; a.v = nullptr; a.g = nullptr;
    a.d = d; a.ld = ld; a.nvec = d / 4;
    a.alpha = alpha; a.lambda = lambda; a.lr = a.mu = a.wd = 0.f;
    a.norms_out = norms_out;
    a.hdr = nullptr;                                   // the sums are the caller's: no header, no staging
    a.partials = const_cast<double *>(sums);
    a.norms_stage = nullptr;
    a.M = M;
    a.spin_first = a.spin_later = kSpinLimit;
    a.schedule = DPPF_PATH_TWO_KERNEL;
    return launch_update_only(a, M, dev, s);
}

// ---- one replica per GPU: this worker's pull-push update from the all-reduced parameters

int dppf_worker_update(float *x, const float *x_reduced, float scale, int64_t d, float alpha, float lambda,
                       float *norm_out, void *ws, size_t ws_bytes, void *cuda_stream) {
    int rc = check_layout(x, 1, d, (d + 31) / 32 * 32);
    if (rc != DPPF_OK) return rc;
    if (!x_reduced) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(x_reduced)) return DPPF_ERR_ALIGNMENT;
    if (!finite_all({scale, alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(1)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = (size_t)d * sizeof(float);
    if (overlap(x, bytes, x_reduced, bytes) || overlap(x, bytes, ws, workspace_bytes(1)) ||
        overlap(x_reduced, bytes, ws, workspace_bytes(1)))
        return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int sms = sm_count(dev);
    if (sms <= 0) return DPPF_ERR_CUDA;
    RoundArgs a;
    a.x = x; a.v = nullptr; a.g = x_reduced;
    a.d = d; a.ld = d; a.nvec = d / 4;
    a.alpha = alpha; a.lambda = lambda; a.lr = scale; a.mu = a.wd = 0.f;
    a.norms_out = norm_out;
    a.hdr = reinterpret_cast<WsHeader *>(ws);
    a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
    a.norms_stage = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + norms_stage_offset(1));
    a.M = 1;
    a.spin_first = a.spin_later = kSpinLimit;
    const long long tile_vecs = (long long)kWorkerThreads * kWorkerUnroll;
    long long ntiles = (a.nvec + tile_vecs - 1) / tile_vecs;
    if (ntiles < 1) ntiles = 1;
    int per_sm = g_worker_occ[dev].load(std::memory_order_relaxed);
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, worker_round_kernel, kWorkerThreads, 0) !=
                cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            return DPPF_ERR_CUDA;
        }
        g_worker_occ[dev].store(per_sm, std::memory_order_relaxed);
    }
    if (per_sm > kWorkerBlocksPerSM) per_sm = kWorkerBlocksPerSM;
    long long grid = (long long)sms * per_sm;
    if (grid > ntiles) grid = ntiles;
    if (grid > kMaxBlocksSmallM) grid = kMaxBlocksSmallM;
    if (coop_supported(dev)) {
        a.schedule = DPPF_PATH_COOPERATIVE;
        void *params[] = {&a};
        if (cudaLaunchCooperativeKernel((const void *)worker_round_kernel, dim3((unsigned)grid), dim3(kWorkerThreads),
                                        params, 0, s) == cudaSuccess)
            return DPPF_OK;
        cudaGetLastError();
    }
    a.schedule = DPPF_PATH_TWO_KERNEL;
    worker_distance_kernel<<<(unsigned)grid, kWorkerThreads, 0, s>>>(a);
    worker_update_kernel<<<(unsigned)grid, kWorkerThreads, 0, s>>>(a, (int)grid);
    return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
}

int dppf_consensus_rounds_ex(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                             const float *lambdas_host, int n_rounds, float *norms_out, void *ws, size_t ws_bytes,
                             int path, void *cuda_stream) {
    int rc = check_layout(x, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (n_rounds < 1) return DPPF_ERR_INVALID_ARG;
    if (path != DPPF_PATH_AUTO && path != DPPF_PATH_TWO_KERNEL && path != DPPF_PATH_COOPERATIVE &&
        path != DPPF_PATH_STAGED)
        return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha})) return DPPF_ERR_INVALID_ARG;
    if (lambdas_host) {
        for (int k = 0; k < n_rounds; ++k)
            if (!std::isfinite(lambdas_host[k])) return DPPF_ERR_INVALID_ARG;
    } else if (!finite_all({lambda})) {
        return DPPF_ERR_INVALID_ARG;
    }
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = extent_bytes(M, d, ld);
    if (overlap(x, bytes, ws, workspace_bytes(M))) return DPPF_ERR_INVALID_ARG;
    if (norms_out && overlap(x, bytes, norms_out, (size_t)n_rounds * M * sizeof(float))) return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    if (path == DPPF_PATH_AUTO) path = DPPF_PATH_STAGED;
    bool single_rounds = (M == 1 || M > kMaxTemplateM || path == DPPF_PATH_TWO_KERNEL);
    int done = 0;
    while (!single_rounds && done < n_rounds) {
        RoundsArgs a;
        a.x = x; a.d = d; a.ld = ld; a.nvec = d / 4;
        a.alpha = alpha;
        a.n_rounds = (n_rounds - done < kMaxRoundsPerLaunch) ? n_rounds - done : kMaxRoundsPerLaunch;
        a.spin_first = g_spin_first.load(std::memory_order_relaxed);
        a.spin_later = g_spin_later.load(std::memory_order_relaxed);
        a.norms_all = norms_out ? norms_out + (size_t)done * M : nullptr;
        a.norms_stage = reinterpret_cast<float *>(static_cast<unsigned char *>(ws) + norms_stage_offset(M));
        a.hdr = reinterpret_cast<WsHeader *>(ws);
        a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
        a.partials_half = (long long)(kMaxBlocksSmallM / 2) * M;
        for (int k = 0; k < a.n_rounds; ++k) a.lambdas[k] = lambdas_host ? lambdas_host[done + k] : lambda;
        bool refused = false;
        rc = launch_rounds(a, M, path, dev, s, &refused);
        if (rc == DPPF_OK) { done += a.n_rounds; continue; }
        if (!refused) return rc;
        single_rounds = true;       // cooperative launch not possible right now: one round per call below
    }
    for (; done < n_rounds; ++done) {
        rc = run_round(x, nullptr, nullptr, M, d, ld, 0.f, 0.f, 0.f, alpha, lambdas_host ? lambdas_host[done] : lambda,
                       norms_out ? norms_out + (size_t)done * M : nullptr, ws, ws_bytes,
                       path == DPPF_PATH_TWO_KERNEL ? DPPF_PATH_TWO_KERNEL : DPPF_PATH_AUTO, false, s);
        if (rc != DPPF_OK) return rc;
    }
    return DPPF_OK;
}

int dppf_consensus_rounds(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                          const float *lambdas_host, int n_rounds, float *norms_out, void *ws, size_t ws_bytes,
                          void *cuda_stream) {
    return dppf_consensus_rounds_ex(x, M, d, ld, alpha, lambda, lambdas_host, n_rounds, norms_out, ws, ws_bytes,
                                    DPPF_PATH_AUTO, cuda_stream);
}

int dppf_debug_set_poll_limits(int first_pass_polls, int later_pass_polls) {
    g_spin_first.store(first_pass_polls < 0 ? kSpinLimit : first_pass_polls, std::memory_order_relaxed);
    g_spin_later.store(later_pass_polls < 0 ? kSpinLimit : later_pass_polls, std::memory_order_relaxed);
    return DPPF_OK;
}

int dppf_consensus_static(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, float *norms_out,
                          void *cuda_stream) {
    if (M > DPPF_STATIC_MAX_WORKERS) return DPPF_ERR_WORKSPACE;   // built-in scratch holds 16 workers at most
    if (M < 1) return DPPF_ERR_INVALID_ARG;
    if (workspace_bytes(M) > kStaticWsBytes) return DPPF_ERR_WORKSPACE;
    int rc = check_layout(x, M, d, ld);      // reject bad arguments before any CUDA call
    if (rc != DPPF_OK) return rc;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    void *ws = nullptr;
    if ((rc = static_ws_address(dev, &ws)) != DPPF_OK) return rc;
    return run_round(x, nullptr, nullptr, M, d, ld, 0.f, 0.f, 0.f, alpha, lambda, norms_out, ws, kStaticWsBytes,
                     DPPF_PATH_AUTO, false, static_cast<cudaStream_t>(cuda_stream));
}

int dppf_static_device_status(void *cuda_stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DPPF_ERR_CUDA;
    void *ws = nullptr;
    const int rc = static_ws_address(dev, &ws);
    if (rc != DPPF_OK) return rc;
    return dppf_device_status(ws, cuda_stream);
}

int dppf_consensus_general_ex(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda,
                              const float *weights_host, int push_from, int two_term, float *norms_out,
                              float *push_norms_out, void *ws, size_t ws_bytes, int path, void *cuda_stream) {
    int rc = check_layout(x, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (M > kMaxTemplateM) return DPPF_ERR_INVALID_ARG;
    if (path != DPPF_PATH_AUTO && path != DPPF_PATH_TWO_KERNEL && path != DPPF_PATH_STAGED) return DPPF_ERR_INVALID_ARG;
    if (push_from != DPPF_PUSH_FROM_AVERAGE && push_from != DPPF_PUSH_FROM_CONSENSUS) return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = extent_bytes(M, d, ld);
    if (overlap(x, bytes, ws, workspace_bytes(M))) return DPPF_ERR_INVALID_ARG;
    GeneralArgs a;
    double wsum = 0.0;
    bool uniform = true;
    for (int m = 0; m < M; ++m) {
        const float w = weights_host ? weights_host[m] : 1.0f;
        if (!std::isfinite(w)) return DPPF_ERR_INVALID_ARG;
        if (weights_host && w != weights_host[0]) uniform = false;
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
    a.uniform = uniform ? 1 : 0;
    a.spin_first = g_spin_first.load(std::memory_order_relaxed);
    a.spin_later = g_spin_later.load(std::memory_order_relaxed);
    a.grid_a = 0;
    a.norms_out = norms_out; a.push_norms_out = push_norms_out;
    a.hdr = reinterpret_cast<WsHeader *>(ws);
    a.partials = reinterpret_cast<double *>(static_cast<unsigned char *>(ws) + kHeaderBytes);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    switch (M) {
#define DPPF_CASE(MM) case MM: return launch_general_m<MM>(a, path, dev, s);
        DPPF_CASE(1) DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: return DPPF_ERR_INVALID_ARG;
    }
}

int dppf_consensus_general(float *x, int M, int64_t d, int64_t ld, float alpha, float lambda, const float *weights_host,
                           int push_from, int two_term, float *norms_out, float *push_norms_out, void *ws,
                           size_t ws_bytes, void *cuda_stream) {
    return dppf_consensus_general_ex(x, M, d, ld, alpha, lambda, weights_host, push_from, two_term, norms_out,
                                     push_norms_out, ws, ws_bytes, DPPF_PATH_AUTO, cuda_stream);
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

int dppf_adamw_step_and_consensus_ex(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M, int64_t d,
                                     int64_t ld, float lr, float beta1, float beta2, float eps, float weight_decay,
                                     int step, float alpha, float lambda, float *norms_out, void *ws,
                                     size_t ws_bytes, int path, void *cuda_stream) {
    int rc = check_adam_buffers(x, exp_avg, exp_avg_sq, g, M, d, ld);
    if (rc != DPPF_OK) return rc;
    if (M > kMaxTemplateM) return DPPF_ERR_INVALID_ARG;
    if (path != DPPF_PATH_AUTO && path != DPPF_PATH_TWO_KERNEL && path != DPPF_PATH_COOPERATIVE) return DPPF_ERR_INVALID_ARG;
    if (!finite_all({alpha, lambda})) return DPPF_ERR_INVALID_ARG;
    AdamArgs p;
    if ((rc = make_adam_args(exp_avg, exp_avg_sq, g, lr, beta1, beta2, eps, weight_decay, step, &p)) != DPPF_OK) return rc;
    if (!ws) return DPPF_ERR_INVALID_ARG;
    if (!aligned128(ws)) return DPPF_ERR_ALIGNMENT;
    if (ws_bytes < workspace_bytes(M)) return DPPF_ERR_WORKSPACE;
    const size_t bytes = extent_bytes(M, d, ld);
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
    a.spin_first = g_spin_first.load(std::memory_order_relaxed);
    a.spin_later = g_spin_later.load(std::memory_order_relaxed);
    if (M == 1) {
        if ((rc = launch_adamw_step(x, p, M, d, ld, dev, s)) != DPPF_OK) return rc;
        zero_norms_kernel<<<1, 32, 0, s>>>(norms_out, a.norms_stage, a.hdr);
        return cudaGetLastError() == cudaSuccess ? DPPF_OK : DPPF_ERR_CUDA;
    }
    switch (M) {
#define DPPF_CASE(MM) case MM: return launch_adamw_round_m<MM>(a, p, path, dev, s);
        DPPF_CASE(2) DPPF_CASE(3) DPPF_CASE(4) DPPF_CASE(5) DPPF_CASE(6) DPPF_CASE(7) DPPF_CASE(8)
        DPPF_CASE(9) DPPF_CASE(10) DPPF_CASE(11) DPPF_CASE(12) DPPF_CASE(13) DPPF_CASE(14) DPPF_CASE(15)
        DPPF_CASE(16)
#undef DPPF_CASE
        default: return DPPF_ERR_INVALID_ARG;
    }
}

int dppf_adamw_step_and_consensus(float *x, float *exp_avg, float *exp_avg_sq, const float *g, int M, int64_t d,
                                  int64_t ld, float lr, float beta1, float beta2, float eps, float weight_decay,
                                  int step, float alpha, float lambda, float *norms_out, void *ws, size_t ws_bytes,
                                  void *cuda_stream) {
    return dppf_adamw_step_and_consensus_ex(x, exp_avg, exp_avg_sq, g, M, d, ld, lr, beta1, beta2, eps, weight_decay,
                                            step, alpha, lambda, norms_out, ws, ws_bytes, DPPF_PATH_AUTO, cuda_stream);
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
