// General round (arbitrary consensus variable, push from x_A or x_C, two-term push) on the staged pipeline.
#pragma once
#include "round_staged.cuh"

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

}  // namespace
