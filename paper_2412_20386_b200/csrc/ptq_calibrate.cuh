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

// s[k] from maxX[k] and the weights; one thread per channel.
__global__ void __launch_bounds__(128) ptq_calib_smooth_kernel(const unsigned *max_x_bits, const int8_t *wq,
                                                               const float *dw, int N, int K, float *s)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    float mw = 0.0f;
    for (int n = 0; n < N; ++n) {
        const float a = __fmul_rn(fabsf(static_cast<float>(wq[static_cast<long long>(n) * K + k])), dw[n]);
        mw = fmaxf(mw, a);
    }
    float mx = __uint_as_float(max_x_bits[k]);
    mx = fmaxf(mx, kCalibFloor);
    mw = fmaxf(mw, kCalibFloor);
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

__global__ void __launch_bounds__(128) ptq_calib_step_kernel(const unsigned *mu_bits, int T, float *dx)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    dx[t] = __fdiv_rn(fmaxf(__uint_as_float(mu_bits[t]), kCalibFloor), 127.0f);
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

}  // namespace ptq
