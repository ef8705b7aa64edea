// General round (arbitrary consensus variable, push from x_A or x_C, two-term push) on the staged pipeline.
#pragma once
#include "round_register.cuh"
#include "chunk_ring.cuh"

namespace {

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

// Threads per block of the cooperative kernel: this round is arithmetic-heavy, so a chunk's float4
// columns should split evenly over the threads (M = 8: 1280 columns = 320 float4 = 320 threads,
// not 256 + a quarter-filled second sweep), within the register budget of the worker count.
template <int M>
struct GeneralShape {
    static constexpr int kVecs = StagedShape<M>::kChunk / 4;
    static constexpr int kMaxThreads = (M <= 4) ? 256 : (M <= 8) ? 384 : 256;
    static constexpr int kSweeps = (kVecs + kMaxThreads - 1) / kMaxThreads;
    static constexpr int kThreads = (((kVecs + kSweeps - 1) / kSweeps) + 31) / 32 * 32;
    static constexpr int kWarps = kThreads / 32;
};

struct GeneralArgs {
    float *x;
    long long d, ld, nvec;
    float alpha, lambda;
    float wn[kMaxTemplateM];     // w_m / sum w
    int push_from_c, two_term;
    int uniform;                 // all weights equal: x_C is x_A, bit for bit
    int spin_first, spin_later;  // mbarrier polls before a wait gives up (distance / update pass)
    float *norms_out;            // ||x_m - x_A|| before the round, may be null
    float *push_norms_out;       // ||y_m - P||, may be null
    WsHeader *hdr;
    double *partials;            // [grid][2 M]: squared distances to x_A, then of the pulled points to P
    int grid_a;                  // two-launch schedule: blocks of the distance launch
    int schedule;                // DPPF_PATH_* being launched, recorded in the workspace header
};

// The per-column arithmetic is written once for fp32 and for packed fp32x2: on sm_100 one
// add/mul/fma instruction handles two columns (float2), which halves the floating-point
// instruction count of this arithmetic-heavy round; each lane is rounded exactly like the scalar
// operation, so both forms give the same bits.
__device__ __forceinline__ float vsplat(float s, float) { return s; }
__device__ __forceinline__ float2 vsplat(float s, float2) { return make_float2(s, s); }
__device__ __forceinline__ float vadd(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float2 vadd(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float vsub(float a, float b) { return __fsub_rn(a, b); }
__device__ __forceinline__ float2 vsub(float2 a, float2 b) { return __fadd2_rn(a, make_float2(-b.x, -b.y)); }
__device__ __forceinline__ float vmul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float2 vmul(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float vfma(float a, float b, float c) { return __fmaf_rn(a, b, c); }
__device__ __forceinline__ float2 vfma(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }

template <int M>
struct GeneralColumn {
    // one column (V = float) or two (V = float2): xs[m] in; adds the two squared distances per worker
    template <typename V>
    static __device__ __forceinline__ void distances(const V (&xs)[M], const GeneralArgs &a, V (&pr)[M], V (&pn)[M]) {
        const V zero = vsplat(0.f, V()), alpha = vsplat(a.alpha, V());
        V e[M], ea = zero, ec = zero;
        e[0] = zero;
#pragma unroll
        for (int m = 1; m < M; ++m) {
            e[m] = vsub(xs[m], xs[0]);
            ea = vadd(ea, e[m]);
            ec = vfma(vsplat(a.wn[m], V()), e[m], ec);
        }
        ea = vmul(ea, vsplat(1.0f / (float)M, V()));
        if (a.uniform) ec = ea;                           // equal weights: the consensus variable IS the average
        const V p = a.push_from_c ? ec : ea;
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const V dev = vsub(e[m], ea);
            pr[m] = vfma(dev, dev, pr[m]);
            const V dy = vfma(alpha, vsub(ec, e[m]), vsub(e[m], p));
            pn[m] = vfma(dy, dy, pn[m]);
        }
    }
    // one or two columns: xs[m] in, updated replicas out; g[m] = lambda / ||y_m - P|| (0: no direction)
    template <typename V>
    static __device__ __forceinline__ void update(V (&xs)[M], const GeneralArgs &a, const float *g) {
        const V zero = vsplat(0.f, V()), alpha = vsplat(a.alpha, V());
        V e[M], ea = zero, ec = zero;
        e[0] = zero;
#pragma unroll
        for (int m = 1; m < M; ++m) {
            e[m] = vsub(xs[m], xs[0]);
            ea = vadd(ea, e[m]);
            ec = vfma(vsplat(a.wn[m], V()), e[m], ec);
        }
        ea = vmul(ea, vsplat(1.0f / (float)M, V()));
        if (a.uniform) ec = ea;                           // equal weights: the consensus variable IS the average
        const V p = a.push_from_c ? ec : ea;
        V ub = zero;                                      // lambda * mean direction
        if (a.two_term) {
#pragma unroll
            for (int m = 0; m < M; ++m) {
                const V dy = vfma(alpha, vsub(ec, e[m]), vsub(e[m], p));
                ub = vfma(vsplat(g[m], V()), dy, ub);
            }
            ub = vmul(ub, vsplat(1.0f / (float)M, V()));
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
            const V pull = vsub(ec, e[m]);                // x_C - x_m
            const V dy = vfma(alpha, pull, vsub(e[m], p));
            const V y = vfma(alpha, pull, xs[m]);
            xs[m] = vsub(vfma(vsplat(g[m], V()), dy, y), ub);
        }
    }
};

// Four columns of all rows at once (one float4 per row) as two packed pairs.
template <int M>
__device__ __forceinline__ void general_distances4(const float4 (&xv)[M], const GeneralArgs &a, float2 (&pr)[M],
                                                   float2 (&pn)[M]) {
    float2 xs[M];
#pragma unroll
    for (int m = 0; m < M; ++m) xs[m] = make_float2(xv[m].x, xv[m].y);
    GeneralColumn<M>::distances(xs, a, pr, pn);
#pragma unroll
    for (int m = 0; m < M; ++m) xs[m] = make_float2(xv[m].z, xv[m].w);
    GeneralColumn<M>::distances(xs, a, pr, pn);
}
template <int M>
__device__ __forceinline__ void general_update4(float4 (&xv)[M], const GeneralArgs &a, const float *g) {
    float2 lo[M], hi[M];
#pragma unroll
    for (int m = 0; m < M; ++m) {
        lo[m] = make_float2(xv[m].x, xv[m].y);
        hi[m] = make_float2(xv[m].z, xv[m].w);
    }
    GeneralColumn<M>::update(lo, a, g);
    GeneralColumn<M>::update(hi, a, g);
#pragma unroll
    for (int m = 0; m < M; ++m) xv[m] = make_float4(lo[m].x, lo[m].y, hi[m].x, hi[m].y);
}

// Scalar tail columns (d % 4 of them), one thread.
template <int M>
__device__ __forceinline__ void general_tail_distances(const GeneralArgs &a, double (&acc)[2 * M]) {
    float pr[M], pn[M];
#pragma unroll
    for (int m = 0; m < M; ++m) pr[m] = pn[m] = 0.f;
    for (long long i = a.nvec * 4; i < a.d; ++i) {
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
template <int M>
__device__ __forceinline__ void general_tail_update(const GeneralArgs &a, const float *g) {
    for (long long i = a.nvec * 4; i < a.d; ++i) {
        float xs[M];
#pragma unroll
        for (int m = 0; m < M; ++m) xs[m] = a.x[m * a.ld + i];
        GeneralColumn<M>::update(xs, a, g);
#pragma unroll
        for (int m = 0; m < M; ++m) a.x[m * a.ld + i] = xs[m];
    }
}

// Block reduction of the 2M per-thread sums into the block's slot of the partials; `failed`
// marks the slot negative ("a wait gave up").  Block 0 also stamps the header.
template <int M, int kWarpsPerBlock>
__device__ __forceinline__ void general_write_partials(const GeneralArgs &a, const double (&acc)[2 * M], double *s_red,
                                                       int failed) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int m = 0; m < 2 * M; ++m) {
        double sum = warp_sum(acc[m]);
        if (lane == 0) s_red[warp * 2 * M + m] = sum;
    }
    __syncthreads();
    if (tid < 2 * M) {
        double sum = 0.0;
        for (int w = 0; w < kWarpsPerBlock; ++w) sum += s_red[w * 2 * M + tid];
        a.partials[(long long)blockIdx.x * 2 * M + tid] = failed ? -1.0 : sum;
    }
    if (blockIdx.x == 0 && tid == 0) {
        a.hdr->status = DPPF_OK;
        a.hdr->magic = kMagic;
        a.hdr->grid = (int)gridDim.x;
        a.hdr->M = M;
        a.hdr->schedule = a.schedule;
    }
}

// Cross-block sums in block order (identical in every block): fills s_g[m] = lambda / ||y_m - P||
// (0: no direction), reports both sets of distances, sets *s_flag if any replica differs from the
// average.  Returns false (in all threads) if nothing is to be written: identical replicas, or a
// negative mark among the partials (then the status word becomes DPPF_ERR_TIMEOUT).
template <int M>
__device__ __forceinline__ bool general_finalise(const GeneralArgs &a, int nblocks, float *s_g, int *s_flag) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    int bad = 0;
    for (int i = tid; i < nblocks * 2 * M; i += blockDim.x) bad |= (__ldcg(a.partials + i) < 0.0) ? 1 : 0;
    if (__syncthreads_or(bad)) {
        if (blockIdx.x == 0 && tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;
        return false;
    }
    if (tid == 0) *s_flag = 0;
    __syncthreads();
    for (int j = warp; j < 2 * M; j += nwarps) {
        double sum = 0.0;
        for (int b = lane; b < nblocks; b += 32) sum += __ldcg(a.partials + (long long)b * 2 * M + j);
        sum = warp_sum(sum);
        if (lane == 0) {
            const double nrm = sqrt(sum);
            if (j < M) {
                if (nrm > 0.0) *s_flag = 1;               // some replica differs from the average
                if (blockIdx.x == 0 && a.norms_out) a.norms_out[j] = (float)nrm;
            } else {
                s_g[j - M] = (nrm > 0.0) ? (float)((double)a.lambda / nrm) : 0.f;
                if (blockIdx.x == 0 && a.push_norms_out) a.push_norms_out[j - M] = (float)nrm;
            }
        }
    }
    __syncthreads();
    return *s_flag != 0;                                  // identical replicas: nothing moves, x untouched
}

// One cooperative launch: staged distance pass, grid barrier, staged update pass in reverse.
template <int M>
__global__ void __launch_bounds__(GeneralShape<M>::kThreads, 1) general_round_kernel(const GeneralArgs a) {
    constexpr int CH = StagedShape<M>::kChunk;
    constexpr int kStages = StagedShape<M>::kStages;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ unsigned long long full[kStages];
    __shared__ double s_red[GeneralShape<M>::kWarps * 2 * M];
    __shared__ float s_g[M];
    __shared__ int s_flag;
    const int tid = threadIdx.x;
    ChunkRing<M> ring;
    ring.base[0] = a.x;
    ring.init(smem_raw, full, a.ld, a.nvec);

    // ---- distance pass: sum (x_m - x_A)^2 and sum (y_m - P)^2 per worker
    double acc[2 * M];
#pragma unroll
    for (int m = 0; m < 2 * M; ++m) acc[m] = 0.0;
    int failed = ring_pass<StagedShape<M>::kPrefetchA>(ring, a.spin_first, true, 0, [&](float *sb, int k, int) {
        const int cols = ring.cols(k);
        float2 pr[M], pn[M];
#pragma unroll
        for (int m = 0; m < M; ++m) pr[m] = pn[m] = make_float2(0.f, 0.f);
        for (int q = tid * 4; q < cols; q += GeneralShape<M>::kThreads * 4) {
            float4 xv[M];
#pragma unroll
            for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
            general_distances4<M>(xv, a, pr, pn);
        }
#pragma unroll
        for (int m = 0; m < M; ++m) {
            acc[m] += (double)__fadd_rn(pr[m].x, pr[m].y);
            acc[M + m] += (double)__fadd_rn(pn[m].x, pn[m].y);
        }
    });
    if (blockIdx.x == 0 && tid == 0 && !failed) general_tail_distances<M>(a, acc);
    general_write_partials<M, GeneralShape<M>::kWarps>(a, acc, s_red, failed);
    cg::this_grid().sync();
    if (!general_finalise<M>(a, (int)gridDim.x, s_g, &s_flag)) return;

    // ---- update pass, chunks in reverse, newest chunks reused from the ring
    failed = ring_pass<StagedShape<M>::kPrefetchB>(ring, a.spin_later, false, ring.resident(), [&](float *sb, int k, int) {
        const int cols = ring.cols(k);
        float *xg = a.x + ring.col0(k);
        for (int q = tid * 4; q < cols; q += GeneralShape<M>::kThreads * 4) {
            float4 xv[M];
#pragma unroll
            for (int m = 0; m < M; ++m) xv[m] = *reinterpret_cast<const float4 *>(sb + m * CH + q);
            general_update4<M>(xv, a, s_g);
#pragma unroll
            for (int m = 0; m < M; ++m) st_keep(xg + m * a.ld + q, xv[m]);
        }
    });
    if (failed) {
        if (tid == 0) a.hdr->status = DPPF_ERR_TIMEOUT;   // x is partly updated
        return;
    }
    if (blockIdx.x == 0 && tid == 0) general_tail_update<M>(a, s_g);
}

// Two-launch schedule (used when the runtime refuses a cooperative launch, or on request):
// the same two passes with 128-bit loads straight into registers.
template <int M>
__global__ void __launch_bounds__(Tuning<M>::kThreads, Tuning<M>::kBlocksPerSM) general_distance_kernel(const GeneralArgs a) {
    constexpr int T = Tuning<M>::kThreads;
    __shared__ double s_red[Tuning<M>::kWarps * 2 * M];
    float2 pr[M], pn[M];
#pragma unroll
    for (int m = 0; m < M; ++m) pr[m] = pn[m] = make_float2(0.f, 0.f);
    const long long ntiles = (a.nvec + T - 1) / T;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const long long j = t * T + threadIdx.x;
        if (j < a.nvec) {
            float4 xv[M];
#pragma unroll
            for (int m = 0; m < M; ++m) xv[m] = ld_keep(a.x + m * a.ld + j * 4);
            general_distances4<M>(xv, a, pr, pn);
        }
    }
    double acc[2 * M];
#pragma unroll
    for (int m = 0; m < M; ++m) {
        acc[m] = (double)__fadd_rn(pr[m].x, pr[m].y);
        acc[M + m] = (double)__fadd_rn(pn[m].x, pn[m].y);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) general_tail_distances<M>(a, acc);
    general_write_partials<M, Tuning<M>::kWarps>(a, acc, s_red, 0);
}

template <int M>
__global__ void __launch_bounds__(Tuning<M>::kThreads, Tuning<M>::kBlocksPerSM) general_update_kernel(const GeneralArgs a) {
    constexpr int T = Tuning<M>::kThreads;
    __shared__ float s_g[M];
    __shared__ int s_flag;
    if (a.hdr->magic != kMagic || a.hdr->grid != a.grid_a || a.hdr->M != M) {   // not this call's distance launch
        if (blockIdx.x == 0 && threadIdx.x == 0) a.hdr->status = DPPF_ERR_WORKSPACE;
        return;
    }
    if (!general_finalise<M>(a, a.grid_a, s_g, &s_flag)) return;
    const long long ntiles = (a.nvec + T - 1) / T;
    if (ntiles > blockIdx.x) {
        long long t = blockIdx.x + (ntiles - 1 - blockIdx.x) / gridDim.x * gridDim.x;
        for (; t >= 0; t -= gridDim.x) {
            const long long j = t * T + threadIdx.x;
            if (j < a.nvec) {
                float4 xv[M];
#pragma unroll
                for (int m = 0; m < M; ++m) xv[m] = ld_last_use(a.x + m * a.ld + j * 4);
                general_update4<M>(xv, a, s_g);
#pragma unroll
                for (int m = 0; m < M; ++m) st_keep(a.x + m * a.ld + j * 4, xv[m]);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) general_tail_update<M>(a, s_g);
}

}  // namespace
