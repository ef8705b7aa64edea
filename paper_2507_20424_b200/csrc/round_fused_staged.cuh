// Last local SGD-momentum step fused with the round, rows staged through shared memory (M <= 8).
#pragma once
#include "round_multi.cuh"

namespace {

// ---------------------------------------------------------------- staged fused round
// Pass A streams x together with the momentum buffer v and the gradients g through a ring of
// stages of about 48 KB (three arrays x M rows), applies the local step (Algorithm 1, local
// update line), stores the stepped x and v and accumulates the squared distances of the stepped
// replicas; one chunk is requested ahead of the one in work (measured best: this pass reads
// three streams and writes two).  After the grid barrier pass B is the staged update pass of the
// plain round on x alone, over the same shared memory with the plain round's stage shape.  Same
// arithmetic, instruction for instruction, as the register-resident fused kernel.  (The AdamW
// step was measured in this form too and lost to its register kernel: its square roots and
// divisions want more warps per SM than one 256-thread block.)
template <int M>
struct FusedShape {
    static constexpr int kArrays = 3;                 // x, v, g
    static constexpr int kChunk = (M <= 4) ? 1024 : ((12288 / (kArrays * M)) / 128) * 128;
    static constexpr size_t kStageBytes = (size_t)kArrays * M * kChunk * sizeof(float);
    static constexpr int kFit = (int)((200 * 1024) / kStageBytes);
    static constexpr int kStages = kFit < kMaxStages ? kFit : kMaxStages;
    static constexpr int kPrefetch = 1;
    static_assert(kChunk >= 128 && kStages >= 2, "stage shape");
};

template <int M>
__global__ void __launch_bounds__(kStagedThreads, 1) fused_round_kernel_staged(const RoundArgs a) {
    constexpr int A = FusedShape<M>::kArrays;
    using RingA = ChunkRing<M, A, FusedShape<M>::kChunk, FusedShape<M>::kStages>;
    using RingB = ChunkRing<M>;
    constexpr int CHA = RingA::CH;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long full_a[RingA::kStages], full_b[RingB::kStages];
    __shared__ double s_red[kStagedWarps * M];
    __shared__ float s_c[M];
    __shared__ int s_ok;
    const int tid = threadIdx.x;
    RingA ra;
    ra.base[0] = a.x;
    ra.base[1] = a.v;
    ra.base[2] = a.g;
    ra.init(smem_raw, full_a, a.ld, a.nvec);
    RingB rb;
    rb.base[0] = a.x;
    rb.init(smem_raw, full_b, a.ld, a.nvec);

    // ---- pass A: local step + distances of the stepped replicas
    double acc[M];
#pragma unroll
    for (int m = 0; m < M; ++m) acc[m] = 0.0;
    int failed = ring_pass<FusedShape<M>::kPrefetch>(ra, a.spin_first, true, 0, [&](float *sb, int k, int) {
        const int cols = ra.cols(k);
        const long long c0 = ra.col0(k);
        float part[M];
#pragma unroll
        for (int m = 0; m < M; ++m) part[m] = 0.f;
        for (int q = tid * 4; q < cols; q += kStagedThreads * 4) {
            float4 xv[M];
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const long long off = m * a.ld + c0 + q;
                xv[m] = *reinterpret_cast<const float4 *>(sb + (0 * M + m) * CHA + q);
                float4 vv = *reinterpret_cast<const float4 *>(sb + (1 * M + m) * CHA + q);
                const float4 gv = *reinterpret_cast<const float4 *>(sb + (2 * M + m) * CHA + q);
                sgd4(xv[m], vv, gv, a.lr, a.mu, a.wd);
                st_keep(a.v + off, vv);
                st_keep(a.x + off, xv[m]);
            }
            const float4 ebar = shifted_mean<M>(xv);
#pragma unroll
            for (int m = 0; m < M; ++m) part[m] = sq_acc(part[m], deviation(xv[m], xv[0], ebar, m));
        }
#pragma unroll
        for (int m = 0; m < M; ++m) acc[m] += (double)part[m];
    });
    if (blockIdx.x == 0 && tid == 0 && !failed) {
        float tail[M];
#pragma unroll
        for (int m = 0; m < M; ++m) tail[m] = 0.f;
        tail_distance<M, true>(a, tail);
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
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // ring B reuses the memory ring A was read from
    cg::this_grid().sync();
    {
        int bad = 0;
        for (int i = tid; i < (int)gridDim.x * M; i += kStagedThreads) bad |= (__ldcg(a.partials + i) < 0.0) ? 1 : 0;
        if (__syncthreads_or(bad)) {
            if (blockIdx.x == 0 && tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;
            return;                                     // the step is partly applied, the round is not
        }
    }
    if (!finalise(a, M, (int)gridDim.x, s_c, &s_ok)) return;

    // ---- pass B: pull-push update of the stepped replicas, chunks in reverse
    double unused[M];
    failed = ring_pass<StagedShape<M>::kPrefetchB>(rb, a.spin_later, false, 0, [&](float *sb, int k, int) {
        chunk_body<M, true>(sb, a.x + rb.col0(k), a.ld, rb.cols(k), s_c, false, false, unused);
    });
    if (failed) {
        if (tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;
        return;
    }
    if (blockIdx.x == 0 && tid == 0) tail_update<M>(a, s_c);
}

}  // namespace
