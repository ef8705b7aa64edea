// Shared-memory chunk ring of the staged kernels: stage shapes, mbarrier and bulk-copy wrappers,
// the ring itself and one pass over a block's chunks.
#pragma once
#include "common.cuh"

namespace {

// One block per SM keeps a ring of shared-memory stages; a stage holds the same column chunk of
// all M rows.  Stages are filled by 1-D bulk async copies (cp.async.bulk, completion counted
// in bytes on the stage's mbarrier); all threads of the block then read the chunk from shared
// memory.  Bulk copies need 16-byte alignment: rows are 128-byte aligned, chunk starts are
// multiples of 128 columns and lengths multiples of 4 columns.  No multicast, no clusters.
// Every wait on an mbarrier is bounded by a poll count.

constexpr int kStagedThreads = 256;
constexpr int kStagedWarps = kStagedThreads / 32;
constexpr int kMaxStages = 6;
constexpr int kSpinLimit = 1 << 22;   // mbarrier try_wait polls before a wait gives up (~ a second)

template <int M>
struct StagedShape {
    // columns per stage and row: a stage of about 32 KB (40 KB measured best for M = 8); above eight
    // rows the row copies of such a stage get short, and 64 KB stages (three of them) measure faster
    static constexpr int kChunk = (M > 8) ? ((16384 / M) / 128) * 128 : (M == 8) ? 1280 : ((8192 / M) / 128) * 128;
    static constexpr size_t kStageFloats = (size_t)M * kChunk;
    static constexpr int kFit = (int)((200 * 1024) / (kStageFloats * sizeof(float)));
    static constexpr int kStages = kFit < kMaxStages ? kFit : kMaxStages;
    static constexpr size_t kSmemBytes = (size_t)kStages * kStageFloats * sizeof(float);
    // chunks in flight ahead of the one being consumed: about 96 KB in the read-only distance
    // pass, one chunk in passes that also write (mixed traffic is fastest with few loads outstanding)
    static constexpr int kPrefetchA = (kStages > 3) ? 3 : kStages - 1;
    static constexpr int kPrefetchB = 1;
    static_assert(kStages > kPrefetchA && kPrefetchA >= kPrefetchB, "ring must be deeper than the prefetch distance");
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
// Bounded wait: false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long *bar, unsigned parity, int limit) {
    for (int spins = 0; spins < limit; ++spins)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, unsigned bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

// Ring of kStages stages; a stage holds the same chunk of kChunk columns of the M rows of each of
// kArrays arrays that share one layout (x alone, or x with optimiser state and gradients).
template <int M, int kArrays = 1, int kChunk = StagedShape<M>::kChunk, int kStages_ = StagedShape<M>::kStages>
struct ChunkRing {
    static constexpr int CH = kChunk;
    static constexpr int kStages = kStages_;
    static constexpr int kRows = kArrays * M;          // row copies per stage
    static constexpr size_t kStageFloats = (size_t)kRows * CH;
    static constexpr size_t kSmemBytes = (size_t)kStages * kStageFloats * sizeof(float);
    float *ring;                   // [kStages][kArrays][M][CH]
    unsigned long long *full;      // one mbarrier per stage
    const float *base[kArrays];
    long long ld, d4;              // row stride; columns covered by float4 groups
    int n;                         // chunks of this block; local chunk k = global chunk blockIdx.x + k gridDim.x,
                                   // always staged in ring stage k % kStages
    unsigned phase;                // bit st: parity of the next wait on stage st

    // to be called by all threads of the block, once; set base[] before
    __device__ __forceinline__ void init(void *smem, unsigned long long *bars, long long ld_, long long nvec) {
        ring = reinterpret_cast<float *>(smem);
        full = bars;
        ld = ld_;
        d4 = nvec * 4;
        const long long nchunks = (d4 + CH - 1) / CH;
        n = (nchunks > blockIdx.x) ? (int)((nchunks - 1 - blockIdx.x) / gridDim.x + 1) : 0;
        phase = 0;
        if (threadIdx.x == 0) {
            for (int st = 0; st < kStages; ++st) mbar_init(&full[st], 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
    }
    __device__ __forceinline__ int resident() const { return (n < kStages) ? n : kStages; }
    __device__ __forceinline__ long long col0(int k) const { return ((long long)k * gridDim.x + blockIdx.x) * CH; }
    __device__ __forceinline__ int cols(int k) const {
        const long long c0 = col0(k);
        return (int)((d4 - c0 < CH) ? (d4 - c0) : CH);
    }
    __device__ __forceinline__ float *stage(int st) const { return ring + (size_t)st * kStageFloats; }
    // called by all of warp 0: lane 0 announces the bytes, then one row copy per lane
    __device__ __forceinline__ void issue(int k, int st) {
        const unsigned bytes = (unsigned)cols(k) * 4u;
        const int lane = threadIdx.x;
        if (lane == 0) mbar_expect_tx(&full[st], bytes * kRows);
        __syncwarp();
        const long long c0 = col0(k);
#pragma unroll
        for (int r0 = 0; r0 < kRows; r0 += 32) {
            const int r = r0 + lane;
            if (r < kRows) {
                const int arr = r / M, m = r - arr * M;
                const float *src = base[0];
#pragma unroll
                for (int i = 1; i < kArrays; ++i)
                    if (arr == i) src = base[i];
                bulk_load(ring + (size_t)st * kStageFloats + (size_t)r * CH, src + m * ld + c0, bytes, &full[st]);
            }
        }
    }
    __device__ __forceinline__ bool wait(int st, int limit) {
        if (mbar_wait_bounded(&full[st], (phase >> st) & 1u, limit)) {
            phase ^= 1u << st;
            return true;
        }
        return false;
    }
};

// One pass over the block's chunks, forward (local chunks 0..n-1) or backward, with kPrefetch
// chunks requested ahead of the one being consumed.  The first `resident` chunks of the pass are
// taken from the ring as the previous pass left them (its last chunks, in the opposite direction).
// body(stage pointer, local chunk k, order index i) runs in all threads on each landed chunk; a
// body that writes the stage must end with fence.proxy.async (the stage is refilled by the
// async proxy later).  `limit` bounds every wait in polls.  If a wait gives up, the block stops
// the pass, thread 0 waits (full budget) for the copies still in flight, and 1 is returned in
// every thread; otherwise 0.
template <int kPrefetch, typename Ring, typename Body>
__device__ __forceinline__ int ring_pass(Ring &ring, int limit, bool fwd, int resident, Body body) {
    constexpr int kStages = Ring::kStages;
    static_assert(kPrefetch >= 1 && kPrefetch < kStages, "prefetch distance must leave a free stage");
    const int tid = threadIdx.x, n = ring.n;
    int failed = 0;
    // (k, st): chunk consumed now and its stage; (kj, stj): order index jn, the next one to fetch
    const int dk = fwd ? 1 : -1;
    int k = fwd ? 0 : n - 1, st = (n > 0) ? k % kStages : 0;
    int jn = resident, kj = fwd ? jn : n - 1 - jn, stj = (kj >= 0) ? kj % kStages : 0;
    int next_wait = resident;                        // oldest order index not yet seen to land (this thread)
    auto advance = [&](int &kk, int &ss) {
        kk += dk;
        ss += dk;
        if (ss == kStages) ss = 0;
        if (ss < 0) ss = kStages - 1;
    };
    if (tid < 32)
        while (jn < n && jn < kPrefetch) {
            ring.issue(kj, stj);
            advance(kj, stj);
            ++jn;
        }
    for (int i = 0; i < n; ++i) {
        if (tid < 32 && jn < n && jn <= i + kPrefetch) {   // stage stj held order index jn - kStages: consumed
            ring.issue(kj, stj);
            advance(kj, stj);
            ++jn;
        }
        int my_fail = 0;
        if (i >= resident) {
            my_fail = ring.wait(st, limit) ? 0 : 1;
            if (!my_fail) next_wait = i + 1;
        }
        if (!my_fail) body(ring.stage(st), k, i);
        if (__syncthreads_or(my_fail)) { failed = 1; break; }  // block-uniform decision
        advance(k, st);
    }
    if (failed && tid == 0)
        for (int j = next_wait; j < jn; ++j) ring.wait((fwd ? j : n - 1 - j) % kStages, kSpinLimit);
    return failed;
}

}  // namespace
