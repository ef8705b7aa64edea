// Kernels for any worker count (16 < M <= 1024) and the stand-alone SGD-momentum local step.
#pragma once
#include "round_register.cuh"

namespace {

// ---------------------------------------------------------------- generic kernels (16 < M <= 1024)
// Rows are streamed twice per vector (second time from L1/L2); per-worker sums live in
// shared memory, one fp32 slot per (warp, worker), so no thread needs M registers.

template <bool kLocalStep>
__global__ void __launch_bounds__(kThreads) distance_kernel_generic(const RoundArgs a) {
    extern __shared__ __align__(16) unsigned char generic_smem[];
    float *s_acc = reinterpret_cast<float *>(generic_smem);               // [kWarps][M]
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
        a.hdr->schedule = a.schedule;
    }
}

__global__ void __launch_bounds__(kThreads) update_kernel_generic(const RoundArgs a, int nblocks_a) {
    extern __shared__ __align__(16) unsigned char generic_smem[];
    float *s_c = reinterpret_cast<float *>(generic_smem);                 // [M]
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
        hdr->schedule = DPPF_PATH_TWO_KERNEL;
    }
}

}  // namespace
