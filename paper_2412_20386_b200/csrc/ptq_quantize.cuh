// Q1: activation smoothing + Per-Token-Static quantization (Sec. 5.1; Appendix B.1 parts 1-2)
//
//     q[m,k] = clamp( rne( (x[m,k] / s[k]) / dx[m mod T] ), -128, 127 )
//
// One pass over x: fp16 in (2 B/element), int8 out (1 B/element); the kernel is HBM-bound, so
// the work is in keeping 16-byte accesses coalesced and the per-element instruction count low
// while producing exactly the bits of two IEEE binary32 divisions.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace ptq {

// a / d, correctly rounded (binary32, round-to-nearest-even), given r = RN(1/d).
// q0 = RN(a r) is within 2 ulp of a/d; one residual correction makes it faithful; a second one
// rounds correctly (Markstein's theorem: y = RN(1/d), q faithful, exact residual via FMA).
// Requirements, guaranteed by the caller: a finite; d, r normal; no intermediate under/overflow
// (|a| in {0} U [2^-84, 2^76] and d in [2^-30, 2^30] keep every residual representable).
__device__ __forceinline__ float div_rn_by_reciprocal(float a, float d, float r)
{
    float q = __fmul_rn(a, r);
    float e = __fmaf_rn(-q, d, a);
    q = __fmaf_rn(e, r, q);
    e = __fmaf_rn(-q, d, a);
    return __fmaf_rn(e, r, q);
}

// cvt.rni.sat.s8.f32: round to nearest even, saturate to [-128,127], NaN -> 0 -- the clip(round()) of
// the definition in one instruction.  The result is the sign-extended code.
__device__ __forceinline__ int f32_to_code(float v)
{
    int r;
    asm("cvt.rni.sat.s8.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}

// One element, IEEE divisions (any positive finite s, dx; also the path for inf/NaN inputs).
__device__ __forceinline__ int quantize_ieee(float xf, float s, float dx)
{
    return f32_to_code(__fdiv_rn(__fdiv_rn(xf, s), dx));
}

// One element through the reciprocal route (finite xf, scales inside the safe range).
__device__ __forceinline__ int quantize_fast(float xf, float s, float rs, float dx, float rdx)
{
    const float u = div_rn_by_reciprocal(xf, s, rs);
    return f32_to_code(div_rn_by_reciprocal(u, dx, rdx));
}

// True if either binary16 half of w has all exponent bits set (inf or NaN).
__device__ __forceinline__ bool half2_has_nonfinite(uint32_t w)
{
    const uint32_t t = (w & 0x7c007c00u) + 0x04000400u;   // 0x7c00 + 0x0400 carries into bit 15
    return (t & 0x80008000u) != 0u;
}

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d)
{
    return (static_cast<uint32_t>(a) & 0xffu) | ((static_cast<uint32_t>(b) & 0xffu) << 8) |
           ((static_cast<uint32_t>(c) & 0xffu) << 16) | (static_cast<uint32_t>(d) << 24);
}

// Quantize 8 consecutive channels held as 4 packed half2 words into 2 words of codes.
// s8 / rs8 point at the 8 channels' s and RN(1/s).
template <bool kFast>
__device__ __forceinline__ void quantize8(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3, const float *s8,
                                          const float *rs8, float dx, float rdx, uint32_t &lo, uint32_t &hi)
{
    const uint32_t xw[4] = {x0, x1, x2, x3};
    int c[8];
    bool slow = !kFast;
    if (kFast)
        slow = half2_has_nonfinite(x0) || half2_has_nonfinite(x1) || half2_has_nonfinite(x2) ||
               half2_has_nonfinite(x3);
    if (slow) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half2 h = *reinterpret_cast<const __half2 *>(&xw[i]);
            const float2 f = __half22float2(h);
            c[2 * i] = quantize_ieee(f.x, s8[2 * i], dx);
            c[2 * i + 1] = quantize_ieee(f.y, s8[2 * i + 1], dx);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half2 h = *reinterpret_cast<const __half2 *>(&xw[i]);
            const float2 f = __half22float2(h);
            c[2 * i] = quantize_fast(f.x, s8[2 * i], rs8[2 * i], dx, rdx);
            c[2 * i + 1] = quantize_fast(f.y, s8[2 * i + 1], rs8[2 * i + 1], dx, rdx);
        }
    }
    lo = pack4(c[0], c[1], c[2], c[3]);
    hi = pack4(c[4], c[5], c[6], c[7]);
}

struct QuantParams {
    const __half *x;     // [M,K]
    int8_t *q;           // [M, q_pitch]
    const float *s;      // [K]
    const float *rs;     // [K]  RN(1/s)
    const float *dx;     // [T]
    const float *rdx;    // [T]  RN(1/dx)
    long long M;
    int K;
    int T;
    int q_pitch;         // bytes between rows of q
    int rows_per_iter;   // vector kernel: rows advanced per grid-stride step (grid threads / chunks per row)
};

// Vector path: K % 16 == 0, x and q 16-byte aligned, q_pitch % 16 == 0.
// A "chunk" is 16 consecutive channels of one row: 2 x 16-byte loads, 1 x 16-byte store.
// The grid's thread count is a multiple of the chunks per row, so each thread keeps the same 16
// channels for the whole launch and holds their s and 1/s in registers.
template <bool kFast>
__global__ void __launch_bounds__(256) ptq_quantize_vec16_kernel(QuantParams p)
{
    const int cpr = p.K >> 4;                                        // chunks per row
    const long long gtid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int kc = static_cast<int>(gtid % cpr);
    long long row = gtid / cpr;
    int t = static_cast<int>(row % p.T);
    const int t_step = p.rows_per_iter % p.T;

    float s16[16], rs16[16];
    {
        const float4 *sp = reinterpret_cast<const float4 *>(p.s + kc * 16);
        const float4 *rp = reinterpret_cast<const float4 *>(p.rs + kc * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 a = __ldg(sp + i), b = __ldg(rp + i);
            s16[4 * i] = a.x; s16[4 * i + 1] = a.y; s16[4 * i + 2] = a.z; s16[4 * i + 3] = a.w;
            rs16[4 * i] = b.x; rs16[4 * i + 1] = b.y; rs16[4 * i + 2] = b.z; rs16[4 * i + 3] = b.w;
        }
    }

    const __half *xcol = p.x + kc * 16;
    int8_t *qcol = p.q + kc * 16;

    // Two rows per trip so that four 16-byte loads are in flight per thread.
    while (row < p.M) {
        const long long row2 = row + p.rows_per_iter;
        int t2 = t + t_step;
        if (t2 >= p.T) t2 -= p.T;
        const bool has2 = row2 < p.M;

        const uint4 *src = reinterpret_cast<const uint4 *>(xcol + row * p.K);
        const uint4 a0 = __ldcs(src), a1 = __ldcs(src + 1);
        uint4 b0 = make_uint4(0, 0, 0, 0), b1 = b0;
        if (has2) {
            const uint4 *src2 = reinterpret_cast<const uint4 *>(xcol + row2 * p.K);
            b0 = __ldcs(src2);
            b1 = __ldcs(src2 + 1);
        }
        const float dxa = __ldg(p.dx + t), rdxa = __ldg(p.rdx + t);
        const float dxb = __ldg(p.dx + t2), rdxb = __ldg(p.rdx + t2);

        uint4 out;
        quantize8<kFast>(a0.x, a0.y, a0.z, a0.w, s16, rs16, dxa, rdxa, out.x, out.y);
        quantize8<kFast>(a1.x, a1.y, a1.z, a1.w, s16 + 8, rs16 + 8, dxa, rdxa, out.z, out.w);
        *reinterpret_cast<uint4 *>(qcol + row * p.q_pitch) = out;
        if (has2) {
            quantize8<kFast>(b0.x, b0.y, b0.z, b0.w, s16, rs16, dxb, rdxb, out.x, out.y);
            quantize8<kFast>(b1.x, b1.y, b1.z, b1.w, s16 + 8, rs16 + 8, dxb, rdxb, out.z, out.w);
            *reinterpret_cast<uint4 *>(qcol + row2 * p.q_pitch) = out;
        }
        row = row2 + p.rows_per_iter;
        t = t2 + t_step;
        if (t >= p.T) t -= p.T;
    }
}

// Generic path: any K, any alignment; one element per thread per step.
template <bool kFast>
__global__ void __launch_bounds__(256) ptq_quantize_scalar_kernel(QuantParams p)
{
    const long long total = p.M * p.K;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const long long m = i / p.K;
        const int k = static_cast<int>(i - m * p.K);
        const int t = static_cast<int>(m % p.T);
        const __half h = p.x[i];
        const float xf = __half2float(h);
        const unsigned short bits = __half_as_ushort(h);
        int c;
        if (kFast && (bits & 0x7c00u) != 0x7c00u)
            c = quantize_fast(xf, __ldg(p.s + k), __ldg(p.rs + k), __ldg(p.dx + t), __ldg(p.rdx + t));
        else
            c = quantize_ieee(xf, __ldg(p.s + k), __ldg(p.dx + t));
        p.q[m * p.q_pitch + k] = static_cast<int8_t>(c);
    }
}

}  // namespace ptq
