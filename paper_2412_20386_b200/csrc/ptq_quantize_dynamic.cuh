// Comparator of Sec. 4.1 / the latency table: per-token DYNAMIC quantization.  The step of a token row
// is not a stored parameter but is measured on that row at run time,
//
//     u[m,k]    = x[m,k] / s[k]
//     dx_row[m] = max( max_k |u[m,k]|, 1e-5 ) / 127
//     q[m,k]    = clamp( rne( u[m,k] / dx_row[m] ), -128, 127 )
//
// which costs a reduction over the row before the first code can be written: every row is read
// twice (the second time from L1/L2) and the reciprocals that the static scheme keeps in registers
// for a whole launch have to be rebuilt per row.  The arithmetic (binary32, two correctly rounded
// divisions, ties to even, NaN -> 0) is that of the static quantizer, and the same screened
// reciprocal route is used for the second pass.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "ptq_calibrate.cuh"
#include "ptq_quantize.cuh"

namespace ptq {

struct DynQuantParams {
    const __half *x;     // [M,K]
    int8_t *q;           // [M, q_pitch]
    float *dx_row;       // [M]
    const float *s;      // [K]
    const float *rs;     // [K]  RN(1/s)
    long long M;
    int K;
    int q_pitch;
};

#ifndef PTQ_DYN_ROWS_PER_WARP
#define PTQ_DYN_ROWS_PER_WARP 2
#endif
#ifndef PTQ_DYN_CTAS_PER_SM
#define PTQ_DYN_CTAS_PER_SM 4
#endif
constexpr int kDynRowsPerWarp = PTQ_DYN_ROWS_PER_WARP;
constexpr float kDynScaleLo = 9.313225746154785e-10f;   // 2^-30
constexpr float kDynScaleHi = 1073741824.0f;            // 2^30

__device__ __forceinline__ uint32_t warp_max_u16x2(uint32_t v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __vmaxu2(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// max_k |x[k] / s[k]| over the 8 channels of one chunk; kRecip: Markstein route (finite x only).
template <bool kRecip>
__device__ __forceinline__ float chunk_absmax(const uint4 &v, const float4 &s0, const float4 &s1, const float4 &r0,
                                              const float4 &r1)
{
    const uint32_t xw[4] = {v.x, v.y, v.z, v.w};
    const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const float rv[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
    float mu = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&xw[i]));
        const float u0 = kRecip ? div_rn_by_reciprocal(f.x, sv[2 * i], rv[2 * i]) : __fdiv_rn(f.x, sv[2 * i]);
        const float u1 = kRecip ? div_rn_by_reciprocal(f.y, sv[2 * i + 1], rv[2 * i + 1]) : __fdiv_rn(f.y, sv[2 * i + 1]);
        mu = fmaxf(mu, fmaxf(fabsf(u0), fabsf(u1)));     // fmaxf drops NaN
    }
    return mu;
}

// Vector path: K % 8 == 0, x 16-byte aligned, q 8-byte aligned, q_pitch % 8 == 0.
// A warp takes kDynRowsPerWarp consecutive rows at a time so that one load of s / RN(1/s) serves
// several rows; lanes take consecutive 8-channel chunks (512-byte loads, 256-byte stores per warp).
template <bool kFast>
__global__ void __launch_bounds__(256, PTQ_DYN_CTAS_PER_SM) ptq_quantize_dynamic_vec8_kernel(DynQuantParams p)
{
    constexpr int R = kDynRowsPerWarp;
    const int lane = threadIdx.x & 31;
    const long long warp = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nwarps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const int cpr = p.K >> 3;
    const float4 *s4 = reinterpret_cast<const float4 *>(p.s);
    const float4 *r4 = reinterpret_cast<const float4 *>(p.rs);
    griddep_wait();
    griddep_launch_dependents();

    for (long long m0 = warp * R; m0 < p.M; m0 += nwarps * R) {
        const int rows = static_cast<int>(p.M - m0 < R ? p.M - m0 : R);
        const uint4 *xrow[R];
#pragma unroll
        for (int j = 0; j < R; ++j)
            xrow[j] = reinterpret_cast<const uint4 *>(p.x + (m0 + (j < rows ? j : 0)) * p.K);

        // ---- pass 1: row maxima of |x / s| ------------------------------------------------------
        float mu[R];
        uint32_t mag[R];     // packed maxima of the fp16 magnitude bits: 0x7c00 or more means inf / NaN in the row
#pragma unroll
        for (int j = 0; j < R; ++j) { mu[j] = 0.0f; mag[j] = 0u; }
        for (int c = lane; c < cpr; c += 32) {
            const float4 s0 = __ldg(s4 + 2 * c), s1 = __ldg(s4 + 2 * c + 1);
            float4 r0 = s0, r1 = s1;
            if (kFast) { r0 = __ldg(r4 + 2 * c); r1 = __ldg(r4 + 2 * c + 1); }
#pragma unroll
            for (int j = 0; j < R; ++j) {
                if (j < rows) {
                    const uint4 v = xrow[j][c];
                    const uint32_t a = __vmaxu2(v.x & 0x7fff7fffu, v.y & 0x7fff7fffu);
                    const uint32_t b = __vmaxu2(v.z & 0x7fff7fffu, v.w & 0x7fff7fffu);
                    mag[j] = __vmaxu2(mag[j], __vmaxu2(a, b));
                    mu[j] = fmaxf(mu[j], chunk_absmax<kFast>(v, s0, s1, r0, r1));
                }
            }
        }
        float dxr[R], rdx[R];
        bool fast_row[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            mu[j] = warp_max(mu[j]);
            const uint32_t mg = warp_max_u16x2(mag[j]);
            const bool nonfinite = ((mg & 0xffffu) >= 0x7c00u) || ((mg >> 16) >= 0x7c00u);
            if (kFast && nonfinite && j < rows) {
                // an infinite input defeats the reciprocal route (inf * 0 residuals): redo this row with IEEE division
                float m2 = 0.0f;
                for (int c = lane; c < cpr; c += 32) {
                    const float4 s0 = __ldg(s4 + 2 * c), s1 = __ldg(s4 + 2 * c + 1);
                    m2 = fmaxf(m2, chunk_absmax<false>(xrow[j][c], s0, s1, s0, s1));
                }
                mu[j] = warp_max(m2);
            }
            dxr[j] = __fdiv_rn(fmaxf(mu[j], kCalibFloor), 127.0f);
            rdx[j] = __fdiv_rn(1.0f, dxr[j]);
            fast_row[j] = kFast && dxr[j] >= kDynScaleLo && dxr[j] <= kDynScaleHi;
            if (lane == 0 && j < rows) p.dx_row[m0 + j] = dxr[j];
        }

        // ---- pass 2: codes -----------------------------------------------------------------------
        for (int c = lane; c < cpr; c += 32) {
            float4 r0 = make_float4(0, 0, 0, 0), r1 = r0;
            if (kFast) { r0 = __ldg(r4 + 2 * c); r1 = __ldg(r4 + 2 * c + 1); }
#pragma unroll
            for (int j = 0; j < R; ++j) {
                if (j < rows) {
                    const uint4 v = xrow[j][c];
                    uint2 out;
                    if (fast_row[j]) {
                        const float c8[8] = {__fmul_rn(r0.x, rdx[j]), __fmul_rn(r0.y, rdx[j]), __fmul_rn(r0.z, rdx[j]),
                                             __fmul_rn(r0.w, rdx[j]), __fmul_rn(r1.x, rdx[j]), __fmul_rn(r1.y, rdx[j]),
                                             __fmul_rn(r1.z, rdx[j]), __fmul_rn(r1.w, rdx[j])};
                        out = quantize8<true, false>(v, c8, p.s + c * 8, p.rs + c * 8, dxr[j], rdx[j], 0);
                    } else {
                        const float none[8] = {};
                        out = quantize8<false, false>(v, none, p.s + c * 8, p.rs + c * 8, dxr[j], rdx[j], 0);
                    }
                    *reinterpret_cast<uint2 *>(p.q + (m0 + j) * p.q_pitch + c * 8) = out;
                }
            }
        }
    }
}

// Generic path: any K and alignment; one warp per row, one element per lane and step, IEEE divisions.
__global__ void __launch_bounds__(256) ptq_quantize_dynamic_scalar_kernel(DynQuantParams p)
{
    griddep_wait();
    griddep_launch_dependents();
    const int lane = threadIdx.x & 31;
    const long long warp = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nwarps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long m = warp; m < p.M; m += nwarps) {
        const __half *row = p.x + m * p.K;
        float mu = 0.0f;
        for (int k = lane; k < p.K; k += 32) mu = fmaxf(mu, fabsf(__fdiv_rn(__half2float(row[k]), __ldg(p.s + k))));
        mu = warp_max(mu);
        const float dxr = __fdiv_rn(fmaxf(mu, kCalibFloor), 127.0f);
        if (lane == 0) p.dx_row[m] = dxr;
        int8_t *qrow = p.q + m * p.q_pitch;
        for (int k = lane; k < p.K; k += 32)
            qrow[k] = static_cast<int8_t>(quantize_ieee<false>(__half2float(row[k]), __ldg(p.s + k), dxr));
    }
}

}  // namespace ptq
