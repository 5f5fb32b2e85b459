// Q0: min-max calibration of the static parameters (Eq. smooth_scale of Sec. 2.4 with the given
// integer weights; per-token-position steps of Sec. 5.1 from the min-max range of Sec. 2.3).
//
//   maxX[k] = max_{b,t} |x[b,t,k]|             maxW[k] = max_n |Wq[n,k]| * dw[n]
//   s[k]    = sqrt( max(maxX[k],1e-5) / max(maxW[k],1e-5) )
//   dx[t]   = max( max_{b,k} |x[b,t,k] / s[k]|, 1e-5 ) / 127
//
// Every arithmetic step is a correctly rounded binary32 operation and max is order independent,
// so the results are unique.  Maxima of non-negative floats are combined with integer atomicMax on
// their bit patterns after a warp-level shuffle reduction.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace ptq {

constexpr float kCalibFloor = 1e-5f;

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// maxX: each warp walks rows with a stride; lanes cover channels k = lane, lane+32, ...
// Per-lane running maxima live in registers (8 channels per lane per pass over K), then one
// atomicMax per (warp, channel).
__global__ void __launch_bounds__(256) ptq_calib_colmax_kernel(const __half *x, long long M, int K,
                                                               unsigned *max_x_bits)
{
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    const long long warp = static_cast<long long>(blockIdx.x) * warps_per_block + (threadIdx.x >> 5);
    const long long nwarps = static_cast<long long>(gridDim.x) * warps_per_block;
    for (int k0 = 0; k0 < K; k0 += 32 * 8) {
        float mx[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) mx[j] = 0.0f;
        for (long long m = warp; m < M; m += nwarps) {
            const __half *row = x + m * K;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int k = k0 + j * 32 + lane;
                if (k < K) mx[j] = fmaxf(mx[j], fabsf(__half2float(row[k])));   // fmaxf drops NaN
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int k = k0 + j * 32 + lane;
            if (k < K && mx[j] > 0.0f) atomicMax(max_x_bits + k, __float_as_uint(mx[j]));
        }
    }
}

// maxW[k] = max_n |Wq[n,k]| * dw[n]: grid (channel blocks, row blocks); a thread scans kCalibRowsPerBlock
// weight rows of its channel (coalesced across the block's channels) and merges with one atomicMax.
constexpr int kCalibRowsPerBlock = 32;

__global__ void __launch_bounds__(128) ptq_calib_wmax_kernel(const int8_t *wq, const float *dw, int N, int K,
                                                             unsigned *max_w_bits)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const int n0 = blockIdx.y * kCalibRowsPerBlock;
    const int n1 = min(N, n0 + kCalibRowsPerBlock);
    float mw = 0.0f;
    for (int n = n0; n < n1; ++n) {
        const float a = __fmul_rn(fabsf(static_cast<float>(wq[static_cast<long long>(n) * K + k])), __ldg(dw + n));
        mw = fmaxf(mw, a);
    }
    if (mw > 0.0f) atomicMax(max_w_bits + k, __float_as_uint(mw));
}

// s[k] from maxX[k] and maxW[k]; one thread per channel.
__global__ void __launch_bounds__(128) ptq_calib_smooth_kernel(const unsigned *max_x_bits, const unsigned *max_w_bits,
                                                               int K, float *s)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const float mx = fmaxf(__uint_as_float(max_x_bits[k]), kCalibFloor);
    const float mw = fmaxf(__uint_as_float(max_w_bits[k]), kCalibFloor);
    s[k] = __fsqrt_rn(__fdiv_rn(mx, mw));
}

// mu[t] = max_{b,k} |x[b,t,k] / s[k]|: one warp per row, shuffle reduction, one atomicMax per row.
__global__ void __launch_bounds__(256) ptq_calib_rowmax_kernel(const __half *x, long long M, int K, int T,
                                                               const float *s, unsigned *mu_bits)
{
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    const long long warp = static_cast<long long>(blockIdx.x) * warps_per_block + (threadIdx.x >> 5);
    const long long nwarps = static_cast<long long>(gridDim.x) * warps_per_block;
    for (long long m = warp; m < M; m += nwarps) {
        const __half *row = x + m * K;
        float mu = 0.0f;
        for (int k = lane; k < K; k += 32)
            mu = fmaxf(mu, fabsf(__fdiv_rn(__half2float(row[k]), __ldg(s + k))));
        mu = warp_max(mu);
        if (lane == 0 && mu > 0.0f) atomicMax(mu_bits + static_cast<int>(m % T), __float_as_uint(mu));
    }
}

__global__ void __launch_bounds__(128) ptq_calib_step_kernel(const unsigned *mu_bits, int T, float *dx, float qmax)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    dx[t] = __fdiv_rn(fmaxf(__uint_as_float(mu_bits[t]), kCalibFloor), qmax);      // 127 levels, or 7 for 4-bit codes
}

// Per-tensor static comparator: ONE step for every token position, from the largest smoothed magnitude
// of the whole calibration batch, dx[t] = max(max_t mu[t], 1e-5) / 127 for all t.  One block.
__global__ void __launch_bounds__(256) ptq_calib_step_tensor_kernel(const unsigned *mu_bits, int T, float *dx,
                                                                    float qmax)
{
    __shared__ unsigned warp_best[8];
    unsigned best = 0u;                                   // bit patterns of non-negative floats order like the floats
    for (int t = threadIdx.x; t < T; t += blockDim.x) best = max(best, mu_bits[t]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
    if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
    __syncthreads();
    best = warp_best[0];
    for (int w = 1; w < static_cast<int>(blockDim.x >> 5); ++w) best = max(best, warp_best[w]);
    const float step = __fdiv_rn(fmaxf(__uint_as_float(best), kCalibFloor), qmax);
    for (int t = threadIdx.x; t < T; t += blockDim.x) dx[t] = step;
}

// --- asymmetric variant: per-token-position range [lo, hi] of x/s, always containing zero ----------
//   hi[t] = max(0, max x/s),  nlo[t] = max(0, max -(x/s))   (both non-negative: atomicMax on the bits)
//   dx[t] = max(hi + nlo, 1e-5) / 255,   z[t] = clip(rne(nlo / dx[t]), 0, 255)
__global__ void __launch_bounds__(256) ptq_calib_rowrange_kernel(const __half *x, long long M, int K, int T,
                                                                 const float *s, unsigned *hi_bits,
                                                                 unsigned *nlo_bits)
{
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    const long long warp = static_cast<long long>(blockIdx.x) * warps_per_block + (threadIdx.x >> 5);
    const long long nwarps = static_cast<long long>(gridDim.x) * warps_per_block;
    for (long long m = warp; m < M; m += nwarps) {
        const __half *row = x + m * K;
        float hi = 0.0f, nlo = 0.0f;
        for (int k = lane; k < K; k += 32) {
            const float u = __fdiv_rn(__half2float(row[k]), __ldg(s + k));
            hi = fmaxf(hi, u);          // fmaxf drops NaN
            nlo = fmaxf(nlo, -u);
        }
        hi = warp_max(hi);
        nlo = warp_max(nlo);
        if (lane == 0) {
            const int t = static_cast<int>(m % T);
            if (hi > 0.0f) atomicMax(hi_bits + t, __float_as_uint(hi));
            if (nlo > 0.0f) atomicMax(nlo_bits + t, __float_as_uint(nlo));
        }
    }
}

__global__ void __launch_bounds__(128) ptq_calib_step_asym_kernel(const unsigned *hi_bits, const unsigned *nlo_bits,
                                                                  int T, float *dx, int *z)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const float hi = __uint_as_float(hi_bits[t]), nlo = __uint_as_float(nlo_bits[t]);
    const float range = fmaxf(__fadd_rn(hi, nlo), kCalibFloor);      // hi - lo with lo = -nlo
    const float d = __fdiv_rn(range, 255.0f);
    const float zr = rintf(__fdiv_rn(nlo, d));                        // -lo / d, ties to even
    dx[t] = d;
    z[t] = static_cast<int>(fminf(fmaxf(zr, 0.0f), 255.0f));
}

// --- step-size search (Sec. 5.2, second stage; "+Truncation" in the ablation) ----------------------
// Per token position t and candidate j (j_lo <= j <= n_grid):
//   Delta = RN(base[t] * RN(j / n_grid)),  u = RN(x / s[k]),  q = clip(rne(RN(u / Delta)), -128, 127)
//   e = RN(u - Delta * q)  (one fused multiply-add),  loss[t,j] = sum_{b,k} e^2 in binary64,
// non-finite u skipped.  One block per (position, group of kSearchCandPerBlock candidates); threads
// stride over the Bc*K elements of the position, keep one binary64 partial sum per candidate, and the
// block reduces them in a fixed order (shuffles, then warp by warp), so a launch is reproducible.
constexpr int kSearchCandPerBlock = 8;
constexpr int kSearchThreads = 256;

struct SearchParams {
    const __half *x;     // [Bc,T,K]
    const float *s;      // [K]
    const float *base;   // [T]
    double *loss;        // [T, n_grid - j_lo + 1]
    int Bc, T, K;
    int n_grid, j_lo;
};

__device__ __forceinline__ float search_candidate_step(float base, int j, int n_grid)
{
    return __fmul_rn(base, __fdiv_rn(static_cast<float>(j), static_cast<float>(n_grid)));
}

__global__ void __launch_bounds__(kSearchThreads) ptq_search_loss_kernel(SearchParams p)
{
    constexpr int C = kSearchCandPerBlock;
    __shared__ double partial[kSearchThreads / 32][C];
    const int t = blockIdx.x;
    const int j0 = p.j_lo + static_cast<int>(blockIdx.y) * C;
    const int ncand = min(C, p.n_grid - j0 + 1);
    const float base = __ldg(p.base + t);
    float delta[C];
    double acc[C];
#pragma unroll
    for (int c = 0; c < C; ++c) {
        delta[c] = search_candidate_step(base, min(j0 + c, p.n_grid), p.n_grid);
        acc[c] = 0.0;
    }
    const int per_pos = p.Bc * p.K;
    for (int i = threadIdx.x; i < per_pos; i += kSearchThreads) {
        const int b = i / p.K;
        const int k = i - b * p.K;
        const float xf = __half2float(p.x[(static_cast<long long>(b) * p.T + t) * p.K + k]);
        const float u = __fdiv_rn(xf, __ldg(p.s + k));
        if (!(fabsf(u) <= 3.402823466e38f)) continue;          // inf and NaN do not enter the loss
#pragma unroll
        for (int c = 0; c < C; ++c) {
            float r = rintf(__fdiv_rn(u, delta[c]));
            r = fminf(fmaxf(r, -128.0f), 127.0f);
            const double e = static_cast<double>(__fmaf_rn(-delta[c], r, u));
            acc[c] = fma(e, e, acc[c]);
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int c = 0; c < C; ++c) {
        double v = acc[c];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) partial[warp][c] = v;
    }
    __syncthreads();
    if (threadIdx.x < ncand) {
        double v = 0.0;
        for (int w = 0; w < kSearchThreads / 32; ++w) v += partial[w][threadIdx.x];
        p.loss[static_cast<long long>(t) * (p.n_grid - p.j_lo + 1) + (j0 - p.j_lo) + threadIdx.x] = v;
    }
}

// The candidate of least loss per position, the largest j among equals (scan from n_grid down, strict <).
__global__ void __launch_bounds__(128) ptq_search_pick_kernel(const double *loss, const float *base, int T, int n_grid,
                                                              int j_lo, int *best, float *dx)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const double *row = loss + static_cast<long long>(t) * (n_grid - j_lo + 1);
    int bj = n_grid;
    double bl = row[n_grid - j_lo];
    for (int j = n_grid - 1; j >= j_lo; --j) {
        const double l = row[j - j_lo];
        if (l < bl) { bl = l; bj = j; }
    }
    best[t] = bj;
    dx[t] = search_candidate_step(__ldg(base + t), bj, n_grid);
}

}  // namespace ptq
