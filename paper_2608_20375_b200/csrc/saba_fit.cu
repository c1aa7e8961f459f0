// Least-squares fit of the SABA gain and cost models to replay logs (Sec. 3.3; the paper fits them on held-out
// prompts by same-prefix budget replay and does not say how: ordinary least squares is the reading taken here).
//
//   gain (Eq. 16):  G = 1 - exp(-B / tau), tau = phi . s + bias, so a logged gain 0 < g_i < 1 at budget B_i gives
//                   tau_i = -B_i / ln(1 - g_i); (phi, bias) = argmin sum_i (tau_i - phi . s_i - bias)^2
//   cost (Eq. 17):  (c0, c1, c2) = argmin sum_i (T_i - c0 - c1 B_i - c2 B_i prefix_i)^2
//
// One pass over the tuples accumulates the normal equations in fp64 (per thread, then per warp by shuffles, per CTA
// in shared memory, per grid by atomics: 36 bytes read per tuple, so the pass is bound by HBM); the CTA that
// finishes last solves the two small systems (columns scaled to unit diagonal first, then Gaussian elimination with
// partial pivoting) and clears the accumulators for the next call.
#include <cuda_runtime.h>
#include <math.h>

#include "common.cuh"
#include "internal.h"

namespace graft {
namespace {

constexpr int kFitThreads = 256;
constexpr int kFitAcc = 25;  // gain: 10 (upper triangle of 4 x 4) + 4 + 1 count; cost: 6 + 3 + 1 count

struct FitParams {
    long long n;
    const float* state;     // [n, 3] conf, degen, hist
    const int32_t* budget;  // [n]
    const float* gain;      // [n]
    const int32_t* prefix;  // [n]
    const float* latency;   // [n]
    double* acc;            // [kFitAcc] zero between calls
    unsigned int* ticket;   // zero between calls
    double* out;            // [10]
};

// x = argmin |A x - r| for the normal equations A (n x n, symmetric, upper triangle given row by row), n <= 4.
// Returns false when a pivot of the scaled system vanishes.
__device__ bool solve_normal(const double* tri, const double* rhs, int n, double* x) {
    double a[4][5], d[4];
    int t = 0;
    for (int i = 0; i < n; ++i)
        for (int j = i; j < n; ++j) {
            a[i][j] = tri[t];
            a[j][i] = tri[t];
            ++t;
        }
    for (int i = 0; i < n; ++i) {
        if (!(a[i][i] > 0.0)) return false;
        d[i] = 1.0 / sqrt(a[i][i]);
    }
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j < n; ++j) a[i][j] *= d[i] * d[j];
        a[i][n] = rhs[i] * d[i];
    }
    for (int c = 0; c < n; ++c) {
        int piv = c;
        for (int i = c + 1; i < n; ++i)
            if (fabs(a[i][c]) > fabs(a[piv][c])) piv = i;
        if (!(fabs(a[piv][c]) > 1e-13)) return false;
        if (piv != c)
            for (int j = c; j <= n; ++j) {
                const double tmp = a[c][j];
                a[c][j] = a[piv][j];
                a[piv][j] = tmp;
            }
        for (int i = c + 1; i < n; ++i) {
            const double f = a[i][c] / a[c][c];
            for (int j = c; j <= n; ++j) a[i][j] -= f * a[c][j];
        }
    }
    for (int i = n - 1; i >= 0; --i) {
        double s = a[i][n];
        for (int j = i + 1; j < n; ++j) s -= a[i][j] * x[j];
        x[i] = s / a[i][i];
    }
    for (int i = 0; i < n; ++i) x[i] *= d[i];
    return true;
}

// one logged round into the running sums
__device__ __forceinline__ void fit_accumulate(double* acc, float s0, float s1, float s2, int budget, float gain,
                                               int prefix, float latency) {
    const double B = (double)budget, g = (double)gain;
    if (g > 0.0 && g < 1.0) {  // a gain of 0 or 1 says nothing about tau
        const double f[4] = {(double)s0, (double)s1, (double)s2, 1.0};
        const double tau = -B / log1p(-g);
        int t = 0;
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = a; b < 4; ++b) acc[t++] += f[a] * f[b];
#pragma unroll
        for (int a = 0; a < 4; ++a) acc[10 + a] += f[a] * tau;
        acc[14] += 1.0;
    }
    const double h[3] = {1.0, B, B * (double)prefix};
    const double T = (double)latency;
    int t = 15;
#pragma unroll
    for (int a = 0; a < 3; ++a)
#pragma unroll
        for (int b = a; b < 3; ++b) acc[t++] += h[a] * h[b];
#pragma unroll
    for (int a = 0; a < 3; ++a) acc[21 + a] += h[a] * T;
    acc[24] += 1.0;
}

// VEC: every array is 16-byte aligned, so a thread takes four consecutive rounds with seven 16-byte loads
template <bool VEC>
__global__ void __launch_bounds__(kFitThreads, 2) saba_fit_kernel(const FitParams p) {
    __shared__ double s_acc[kFitAcc];
    __shared__ bool s_last;
    double acc[kFitAcc];
#pragma unroll
    for (int i = 0; i < kFitAcc; ++i) acc[i] = 0.0;
    if (threadIdx.x < kFitAcc) s_acc[threadIdx.x] = 0.0;
    __syncthreads();
    const long long tid = blockIdx.x * (long long)kFitThreads + threadIdx.x, nth = (long long)gridDim.x * kFitThreads;
    long long done = 0;
    if (VEC) {
        const long long n4 = p.n / 4;
        for (long long q = tid; q < n4; q += nth) {
            const float4 a = __ldg((const float4*)p.state + 3 * q), b = __ldg((const float4*)p.state + 3 * q + 1),
                         c = __ldg((const float4*)p.state + 3 * q + 2);
            const int4 bu = __ldg((const int4*)p.budget + q), pr = __ldg((const int4*)p.prefix + q);
            const float4 ga = __ldg((const float4*)p.gain + q), la = __ldg((const float4*)p.latency + q);
            fit_accumulate(acc, a.x, a.y, a.z, bu.x, ga.x, pr.x, la.x);
            fit_accumulate(acc, a.w, b.x, b.y, bu.y, ga.y, pr.y, la.y);
            fit_accumulate(acc, b.z, b.w, c.x, bu.z, ga.z, pr.z, la.z);
            fit_accumulate(acc, c.y, c.z, c.w, bu.w, ga.w, pr.w, la.w);
        }
        done = n4 * 4;
    }
    for (long long i = done + tid; i < p.n; i += nth)
        fit_accumulate(acc, p.state[3 * i], p.state[3 * i + 1], p.state[3 * i + 2], p.budget[i], p.gain[i], p.prefix[i],
                       p.latency[i]);
#pragma unroll
    for (int i = 0; i < kFitAcc; ++i) {
        double v = acc[i];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
        if ((threadIdx.x & 31) == 0) atomicAdd(&s_acc[i], v);
    }
    __syncthreads();
    if (threadIdx.x < kFitAcc) atomicAdd(p.acc + threadIdx.x, s_acc[threadIdx.x]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(p.ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last || threadIdx.x != 0) return;
    __threadfence();
    double tot[kFitAcc];
    for (int i = 0; i < kFitAcc; ++i) {
        tot[i] = __ldcg(p.acc + i);
        p.acc[i] = 0.0;  // ready for the next call
    }
    *p.ticket = 0u;
    double phi[4] = {0.0, 0.0, 0.0, 0.0}, c[3] = {0.0, 0.0, 0.0};
    int status = 0;
    if (!(tot[14] >= 4.0) || !solve_normal(tot, tot + 10, 4, phi)) status |= 1;
    if (!(tot[24] >= 3.0) || !solve_normal(tot + 15, tot + 21, 3, c)) status |= 2;
    for (int i = 0; i < 4; ++i) p.out[i] = (status & 1) ? 0.0 : phi[i];
    for (int i = 0; i < 3; ++i) p.out[4 + i] = (status & 2) ? 0.0 : c[i];
    p.out[7] = tot[14];
    p.out[8] = tot[24];
    p.out[9] = (double)status;
}

}  // namespace

cudaError_t saba_fit_launch(graft_ctx* ctx, long long n, const float* d_state, const int32_t* d_budget,
                            const float* d_gain, const int32_t* d_prefix, const float* d_latency, double* d_out,
                            cudaStream_t st) {
    FitParams p;
    p.n = n;
    p.state = d_state;
    p.budget = d_budget;
    p.gain = d_gain;
    p.prefix = d_prefix;
    p.latency = d_latency;
    p.acc = ctx->w_fit;
    p.ticket = (unsigned int*)(ctx->w_fit + kFitAcc + 1);
    p.out = d_out;
    const bool vec = (((uintptr_t)d_state | (uintptr_t)d_budget | (uintptr_t)d_gain | (uintptr_t)d_prefix |
                       (uintptr_t)d_latency) & 15) == 0;
    long long grid = ((vec ? n / 4 + 3 : n) + kFitThreads - 1) / kFitThreads;
    const long long cap = (long long)ctx->num_sms * 2;  // what the registers let an SM hold
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    if (vec)
        saba_fit_kernel<true><<<(int)grid, kFitThreads, 0, st>>>(p);
    else
        saba_fit_kernel<false><<<(int)grid, kFitThreads, 0, st>>>(p);
    ctx->launches += 1;
    return cudaGetLastError();
}

}  // namespace graft
