// Staged persistent round kernel: rows streamed through a shared-memory ring by bulk async copies.
#pragma once
#include "round_register.cuh"
#include "chunk_ring.cuh"

namespace {

// ---------------------------------------------------------------- staged persistent kernel, one round (default for M <= 8)
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

template <int M>
__global__ void __launch_bounds__(kStagedThreads, 1) round_kernel_staged(const RoundArgs a) {
    constexpr int CH = StagedShape<M>::kChunk;
    constexpr int kStages = StagedShape<M>::kStages;
    constexpr int kPrefetchA = StagedShape<M>::kPrefetchA, kPrefetchB = StagedShape<M>::kPrefetchB;
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
    long long k_done = 0;                                           // chunks this thread saw land
    long long k_fail = 0;                                           // iteration in which the block gave up
    for (long long k = 0; k < n; ++k) {
        k_fail = k;
        if (tid == 0 && k + kPrefetchA < n) issue(k + kPrefetchA);
        const int st = (int)(k % kStages);
        int my_fail = mbar_wait_bounded(&full[st], (phase >> st) & 1u, a.spin_first) ? 0 : 1;
        if (!my_fail) {
            phase ^= 1u << st;
            k_done = k + 1;
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
        if (__syncthreads_or(my_fail)) { failed = 1; break; }      // block-uniform decision
    }
    if (failed && tid == 0) {
        // copies still in flight (from the first chunk this thread did not see land) get the full
        // poll budget before the block moves on
        const long long hi = (k_fail + kPrefetchA < n - 1) ? k_fail + kPrefetchA : n - 1;
        for (long long k = k_done; k <= hi; ++k) {
            const int st = (int)(k % kStages);
            mbar_wait_bounded(&full[st], (phase >> st) & 1u, kSpinLimit);
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
            a.hdr->schedule = a.schedule;
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
            my_fail = mbar_wait_bounded(&full[st], (phase >> st) & 1u, a.spin_later) ? 0 : 1;
            if (!my_fail) phase ^= 1u << st;
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
                // the copies that may still be in flight: chunk k (unless this thread saw it land) and k - 1
                if (my_fail) mbar_wait_bounded(&full[st], (phase >> st) & 1u, kSpinLimit);
                const long long kl = k - kPrefetchB;
                if (kl >= 0 && kl < n - resident)
                    mbar_wait_bounded(&full[(int)(kl % kStages)], (phase >> (int)(kl % kStages)) & 1u, kSpinLimit);
            }
            return;
        }
    }
    if (blockIdx.x == 0 && tid == 0) tail_update<M>(a, s_c);
}

}  // namespace
