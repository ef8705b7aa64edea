// Shared pieces of the DPPF kernels: constants, argument structs, cache-hinted accesses and the
// explicitly rounded arithmetic both passes of a round use.
#pragma once
#include "dppf.h"
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <atomic>
#include <climits>
#include <cmath>
#include <cstdint>
namespace cg = cooperative_groups;

namespace {


constexpr int kThreads = 256;            // threads per block: generic and local-step kernels
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTemplateM = 16;        // worker counts with register-resident kernels
constexpr int kMaxBlocksSmallM = 2048;   // partial-sum slots reserved per worker, M <= 16
constexpr int kMaxBlocksLargeM = 512;    // ... and for the generic kernels
constexpr size_t kHeaderBytes = 256;
constexpr unsigned kMagic = 0x44505046u; // "DPPF"

struct WsHeader {
    int status;       // dppf_status seen by the kernels
    unsigned magic;   // written by the distance pass, checked by the update pass
    int grid;         // blocks that wrote partials
    int M;
    int schedule;     // DPPF_PATH_* of the kernels that ran the last call on this workspace
};

struct RoundArgs {
    float *x;
    float *v;         // fused local step only
    const float *g;   // fused local step only
    long long d, ld, nvec;   // nvec = d / 4 full float4 groups per row
    float alpha, lambda, lr, mu, wd;
    float *norms_out; // may be null
    float *norms_stage; // fp32[M] inside the workspace (always written)
    WsHeader *hdr;
    double *partials; // [grid, M]
    int M;            // runtime copy (generic kernels)
    int spin_first, spin_later;   // staged kernel: mbarrier polls before a wait gives up (distance / update pass)
    int schedule;                 // DPPF_PATH_* being launched, recorded in the workspace header
};

// ---------------------------------------------------------------- memory access helpers

__device__ __forceinline__ float4 ld_keep(const float *p) {   // normal L2 priority, skip L1
    return __ldcg(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ float4 ld_last_use(const float *p) {  // evict-first: dead after this read
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void st_keep(float *p, float4 v) {
    __stcg(reinterpret_cast<float4 *>(p), v);
}

// ---------------------------------------------------------------- arithmetic helpers
// Explicitly rounded operations: the compiler may not re-associate or contract them, so
// the distance pass and the update pass see bit-identical deviations.

__device__ __forceinline__ float4 sub4(float4 a, float4 b) {
    return make_float4(__fsub_rn(a.x, b.x), __fsub_rn(a.y, b.y), __fsub_rn(a.z, b.z), __fsub_rn(a.w, b.w));
}
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float4 scale4(float4 a, float s) {
    return make_float4(__fmul_rn(a.x, s), __fmul_rn(a.y, s), __fmul_rn(a.z, s), __fmul_rn(a.w, s));
}
__device__ __forceinline__ float sq_acc(float acc, float4 d) {
    acc = __fmaf_rn(d.x, d.x, acc);
    acc = __fmaf_rn(d.y, d.y, acc);
    acc = __fmaf_rn(d.z, d.z, acc);
    acc = __fmaf_rn(d.w, d.w, acc);
    return acc;
}
// x - c * dev
__device__ __forceinline__ float4 apply4(float4 x, float4 dev, float c) {
    return make_float4(__fmaf_rn(-c, dev.x, x.x), __fmaf_rn(-c, dev.y, x.y),
                       __fmaf_rn(-c, dev.z, x.z), __fmaf_rn(-c, dev.w, x.w));
}
// Local optimiser step on one element: g~ = g + wd x ; v' = mu v + g~ ; x' = x - lr v'.
__device__ __forceinline__ void sgd1(float &x, float &v, float g, float lr, float mu, float wd) {
    float gt = __fmaf_rn(wd, x, g);
    v = __fmaf_rn(mu, v, gt);
    x = __fmaf_rn(-lr, v, x);
}
__device__ __forceinline__ void sgd4(float4 &x, float4 &v, float4 g, float lr, float mu, float wd) {
    sgd1(x.x, v.x, g.x, lr, mu, wd);
    sgd1(x.y, v.y, g.y, lr, mu, wd);
    sgd1(x.z, v.z, g.z, lr, mu, wd);
    sgd1(x.w, v.w, g.w, lr, mu, wd);
}

// Shifted mean of one vector over the M rows: ebar = (sum_{m>=1} (x_m - x_0)) / M, so that
// x_A = x_0 + ebar and the deviation of row m is dev_m = (x_m - x_0) - ebar (dev_0 = -ebar).
template <int M>
__device__ __forceinline__ float4 shifted_mean(const float4 (&xv)[M]) {
    const float inv_m = 1.0f / (float)M;
    float4 esum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int m = 1; m < M; ++m) esum = add4(esum, sub4(xv[m], xv[0]));
    return scale4(esum, inv_m);
}
__device__ __forceinline__ float4 deviation(float4 xm, float4 x0, float4 ebar, int m) {
    if (m == 0) return make_float4(-ebar.x, -ebar.y, -ebar.z, -ebar.w);
    return sub4(sub4(xm, x0), ebar);
}

__device__ __forceinline__ double warp_sum(double a) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    return a;   // butterfly: every lane holds the same bits
}

// Coefficient c_m = alpha - lambda / r_m of the single-line update.  Zero distance: the push
// direction is undefined and the pull acts on a zero vector, so the replica must stay as it
// is, bit for bit (including the sign of zeros).  That case is signalled by a NaN coefficient,
// which the update pass reads as "do not write this row".
__device__ __forceinline__ float coefficient(double S, float alpha, float lambda, float *r_out) {
    double r = sqrt(S);
    *r_out = (float)r;
    if (!(r > 0.0)) return __int_as_float(0x7fc00000);
    return (float)((double)alpha - (double)lambda / r);
}
__device__ __forceinline__ bool row_is_written(float c) { return c == c; }

}  // namespace
