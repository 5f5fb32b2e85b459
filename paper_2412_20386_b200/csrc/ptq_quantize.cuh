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

#include "ptx_sm100.cuh"

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

// Asymmetric code (zero offset z in [0,255] per token position): clip(rne(v) + z, 0, 255).
// The offset is added to the rounded INTEGER (adding it in binary32 before rounding would erase ties);
// cvt.rni.sat.s16.f32 keeps the intermediate inside +-32768 so the addition cannot overflow, and maps
// NaN to 0, i.e. to the code z.
__device__ __forceinline__ int f32_to_code_asym(float v, int z)
{
    short r;
    asm("cvt.rni.sat.s16.f32 %0, %1;" : "=h"(r) : "f"(v));
    return min(max(static_cast<int>(r) + z, 0), 255);
}

// Code formats: signed 8-bit (the path of Sec. 5.1), unsigned 8-bit with a zero offset, signed 4-bit
// held one per byte (W4A4 of the latency table: clip to [-8, 7]).
constexpr int kCodeS8 = 0, kCodeU8 = 1, kCodeS4 = 2;

template <int kMode>
__device__ __forceinline__ int code_of(float v, int z)
{
    if (kMode == kCodeU8) return f32_to_code_asym(v, z);
    const int r = f32_to_code(v);
    return kMode == kCodeS4 ? min(max(r, -8), 7) : r;
}

// One element, IEEE divisions (any positive finite s, dx; also the path for inf/NaN inputs).
template <int kMode = kCodeS8>
__device__ __forceinline__ int quantize_ieee(float xf, float s, float dx, int z = 0)
{
    return code_of<kMode>(__fdiv_rn(__fdiv_rn(xf, s), dx), z);
}

// One element through the reciprocal route (finite xf, scales inside the safe range).
template <int kMode = kCodeS8>
__device__ __forceinline__ int quantize_fast(float xf, float s, float rs, float dx, float rdx, int z = 0)
{
    const float u = div_rn_by_reciprocal(xf, s, rs);
    return code_of<kMode>(div_rn_by_reciprocal(u, dx, rdx), z);
}

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d)
{
    // low bytes of four registers -> one word (a lowest)
    const uint32_t ab = __byte_perm(static_cast<uint32_t>(a), static_cast<uint32_t>(b), 0x0040);
    const uint32_t cd = __byte_perm(static_cast<uint32_t>(c), static_cast<uint32_t>(d), 0x0040);
    return __byte_perm(ab, cd, 0x5410);
}

// Screening threshold of the fast route below.  v' = x * (RN(1/s) * RN(1/dx)) differs from the
// defined value v = RN(RN(x/s)/dx) by six roundings: |v' - v| <= 6 * 2^-24 * (1 + tiny) * |v|, which is
// below 4.6e-5 for |v| <= 127.5, the largest magnitude at which a rounding tie still changes the
// clamped code.  If v' is farther than 6e-5 from every half-integer, rint(v') = rint(v).
constexpr float kScreenThreshold = 0.49994f;
// Asymmetric codes: rint(v) ranges over [-255, 255] before the offset, so ties matter up to |v| = 255.5,
// where six roundings amount to 9.2e-5; the band is widened to 1.2e-4 accordingly.
constexpr float kScreenThresholdAsym = 0.49988f;
constexpr float kRoundMagic = 12582912.0f;   // 1.5 * 2^23: (v + magic) - magic = rint(v) for |v| < 2^22

// |v - rint(v)| for |v| < 2^22; NaN for NaN and infinite v; meaningless (but finite or NaN) beyond.
__device__ __forceinline__ float dist_to_integer(float v)
{
    const float r = __fadd_rn(__fadd_rn(v, kRoundMagic), -kRoundMagic);
    return fabsf(__fadd_rn(v, -r));
}

// Fast route for 8 consecutive channels held as 4 packed half2 words: one multiply by the combined
// reciprocal c = RN(RN(1/s) * RN(1/dx)), the saturating round-to-nearest-even conversion, and a
// distance-to-tie test.  Returns true when one of the 8 values sits within the error bound of a
// rounding tie, in which case the caller recomputes the 8 codes with the two exact divisions.
// Values beyond +-127.5 clamp to the same code whichever way a tie falls, NaN converts to 0 and
// infinities saturate on both routes, so whether such values pass the test or not only costs time:
// the final codes are always those of the definition.
// Valid only when every scale lies in [2^-30, 2^30] (no under/overflow in c or x * c).
// Unsigned codes: clip(rint(v') + z, 0, 255); ties of v' are still the only place where v' and v
// can disagree, with the wider band of kScreenThresholdAsym.
template <int kMode = kCodeS8>
__device__ __forceinline__ bool quantize8_screen(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3,
                                                 const float (&c8)[8], uint32_t &lo, uint32_t &hi, int z = 0)
{
    const uint32_t xw[4] = {x0, x1, x2, x3};
    int c[8];
    float worst = 0.0f;   // largest distance to an integer; fmaxf drops the NaN that NaN / inf inputs produce,
                          // which is fine: their codes (0, +-saturation) are the same on both routes
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __half2 h = *reinterpret_cast<const __half2 *>(&xw[i]);
        const float2 f = __half22float2(h);
        const float v0 = __fmul_rn(f.x, c8[2 * i]);
        const float v1 = __fmul_rn(f.y, c8[2 * i + 1]);
        c[2 * i] = code_of<kMode>(v0, z);
        c[2 * i + 1] = code_of<kMode>(v1, z);
        worst = fmaxf(worst, fmaxf(dist_to_integer(v0), dist_to_integer(v1)));
    }
    lo = pack4(c[0], c[1], c[2], c[3]);
    hi = pack4(c[4], c[5], c[6], c[7]);
    return worst > (kMode == kCodeU8 ? kScreenThresholdAsym : kScreenThreshold);
}

// max(a, |b|, |c|) in one instruction (three-input max of sm_100); NaN operands are dropped like fmaxf does.
__device__ __forceinline__ float max3_abs(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(fabsf(b)), "f"(fabsf(c)));
    return r;
}

// The same, but a NaN operand makes the result NaN (and keeps it NaN through a chain of these).
__device__ __forceinline__ float max3_abs_nan(float a, float b, float c)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(fabsf(b)), "f"(fabsf(c)));
    return r;
}

// First-level route for signed codes, without any float-to-integer conversion instruction (those run
// at a quarter of the rate of the other arithmetic here).  t = v' + 1.5*2^23 holds rint(v'), ties to
// even, in its low mantissa bits, so for |v'| <= 127.25 the low BYTE of t is the two's-complement code;
// the same t gives the tie distance.  Arithmetic is done two lanes per instruction (packed binary32
// multiply / add / fma of sm_100; each lane is the ordinary correctly rounded operation).  Returns true
// when the chunk has to go to the slower routes: a value within the tie band, a magnitude above
// 127.25 (saturation is not handled here), or a NaN / infinity: the running magnitude maximum
// propagates NaN, and an infinity exceeds the limit, so both fail the one comparison on `big`.
template <int kMode = kCodeS8>
__device__ __forceinline__ bool quantize8_magic(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3,
                                                const float (&c8)[8], uint32_t &lo, uint32_t &hi)
{
    const uint32_t xw[4] = {x0, x1, x2, x3};
    uint32_t tb[8];
    float worst = 0.0f, big = 0.0f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&xw[i]));
        const float2 v = __fmul2_rn(f, make_float2(c8[2 * i], c8[2 * i + 1]));
        const float2 t = __fadd2_rn(v, make_float2(kRoundMagic, kRoundMagic));
        const float2 r = __fadd2_rn(t, make_float2(-kRoundMagic, -kRoundMagic));
        const float2 d = __ffma2_rn(v, make_float2(-1.0f, -1.0f), r);      // rint(v) - v: exact, or NaN
        worst = max3_abs(worst, d.x, d.y);
        big = max3_abs_nan(big, v.x, v.y);
        tb[2 * i] = __float_as_uint(t.x);
        tb[2 * i + 1] = __float_as_uint(t.y);
    }
    lo = pack4(static_cast<int>(tb[0]), static_cast<int>(tb[1]), static_cast<int>(tb[2]), static_cast<int>(tb[3]));
    hi = pack4(static_cast<int>(tb[4]), static_cast<int>(tb[5]), static_cast<int>(tb[6]), static_cast<int>(tb[7]));
    return !(worst <= kScreenThreshold && big <= (kMode == kCodeS4 ? 7.25f : 127.25f));
}

// Exact route for the same 8 channels: two correctly rounded divisions per element.  s8 / rs8 point
// at the channels' s and RN(1/s) in global memory.
template <bool kFast, int kMode = kCodeS8>
__device__ __noinline__ void quantize8_exact(uint32_t x0, uint32_t x1, uint32_t x2, uint32_t x3, const float *s8,
                                             const float *rs8, float dx, float rdx, uint32_t &lo, uint32_t &hi,
                                             int z = 0)
{
    const uint32_t xw[4] = {x0, x1, x2, x3};
    int c[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const __half hv = __ushort_as_half(static_cast<unsigned short>(xw[i >> 1] >> ((i & 1) * 16)));
        const float f = __half2float(hv);
        const float sv = __ldg(s8 + i);
        if (kFast && fabsf(f) <= 65504.0f)
            c[i] = quantize_fast<kMode>(f, sv, __ldg(rs8 + i), dx, rdx, z);
        else
            c[i] = quantize_ieee<kMode>(f, sv, dx, z);
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
    const float2 *dx2;   // [T]  {dx, RN(1/dx)} interleaved (one 8-byte load)
    const int *zp;       // [T]  zero offsets (asymmetric layers), else nullptr
    long long M;
    int K;
    int T;
    int q_pitch;         // bytes between rows of q
    int B;               // images (M = B * T)
    int imgs_per_iter;   // vector kernel: images between consecutive chunks of one thread
    FastDiv fd_cpi, fd_cpr;   // vector kernel: divisors T * K / 8 (chunks per image) and K / 8 (chunks per row)
};

#ifndef PTQ_QUANT_CTAS_PER_SM
#define PTQ_QUANT_CTAS_PER_SM 4
#endif
#ifndef PTQ_QUANT_RING_DEPTH
#define PTQ_QUANT_RING_DEPTH 4
#endif
constexpr int kQuantCtasPerSm = PTQ_QUANT_CTAS_PER_SM;   // resident CTAs per SM the vector kernel is built and launched for
constexpr int kQuantRingDepth = PTQ_QUANT_RING_DEPTH;    // 16-byte loads in flight per thread

// L2 cache policy of the quantize kernel's loads: the activations are read once and never again, so they are
// marked evict-first and do not push the codes (read back by the GEMM kernel launched next) or the next layer's
// parameters out of L2.  Measured: the K = 768 layer of Vim-B 21.3 -> 20.4 us, nothing else changes.  Marking the
// code stores evict-last as well made the GEMM kernels of small-K layers 6 % faster when timed alone, but the
// Vim-B in_proj GEMM 4 % slower and no step faster, so the stores keep the default policy.
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void cp_async_16_hint(void *smem_dst, const void *gmem_src, uint64_t policy)
{
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// The three routes for one chunk of 8 channels, cheapest first; every route that returns codes returns
// the codes of the definition.
template <bool kFast, int kMode>
__device__ __forceinline__ uint2 quantize8(const uint4 &v, const float (&c8)[8], const float *s8, const float *rs8,
                                           float dx, float rdx, int z)
{
    uint2 out;
    bool exact = true;
    if (kFast) {
        bool slow = true;
        if (kMode != kCodeU8) slow = quantize8_magic<kMode>(v.x, v.y, v.z, v.w, c8, out.x, out.y);
        exact = slow && quantize8_screen<kMode>(v.x, v.y, v.z, v.w, c8, out.x, out.y, z);
    }
    if (exact) quantize8_exact<kFast, kMode>(v.x, v.y, v.z, v.w, s8, rs8, dx, rdx, out.x, out.y, z);
    return out;
}

// Vector path: K % 8 == 0, x 16-byte aligned, q 8-byte aligned, q_pitch % 8 == 0.
// A "chunk" is 8 consecutive channels of one token row: one 16-byte load, one 8-byte store.
// Thread g of the grid owns chunk (g mod chunks-per-image) of images b0, b0+S, b0+2S, ... with
// b0 = g / chunks-per-image; the grid's thread count is S * chunks-per-image.  A thread therefore
// sees ONE token position and ONE group of 8 channels for the whole launch -- that is what "static"
// per-token steps buy: the 8 combined reciprocals RN(1/s[k]) * RN(1/dx[t]) are formed once and kept
// in registers, and the per-element work is convert, multiply, round, tie test.  Consecutive lanes
// take consecutive chunks, so warp-wide accesses are contiguous 512-byte loads and 256-byte stores.
// The loads are asynchronous copies (cp.async, L2 only) into a per-thread ring of shared-memory
// slots, kQuantRingDepth images ahead.  A thread reads back only the slots it filled itself, so no
// barrier is involved: cp.async.wait_group orders the thread's own copies.  Loads in flight hold no
// registers, and their number does not depend on how far the arithmetic of the current chunk has got.
template <bool kFast, int kMode = kCodeS8>
__global__ void __launch_bounds__(256, kQuantCtasPerSm) ptq_quantize_vec8_kernel(QuantParams p)
{
    constexpr int D = kQuantRingDepth;
    __shared__ uint4 ring[D][256];
    const int cpr = p.K >> 3;                                        // chunks per row
    const int cpi = p.T * cpr;                                       // chunks per image
    // the grid is at most four resident waves, so the global thread index fits 32 bits; no runtime divisions
    // in front of the parameter loads below (a CTA that starts late runs this prologue on the critical path)
    const unsigned gtid = blockIdx.x * blockDim.x + threadIdx.x;
    int b = static_cast<int>(fd_div(gtid, p.fd_cpi));
    const int c = static_cast<int>(gtid) - b * cpi;
    const int t = static_cast<int>(fd_div(static_cast<unsigned>(c), p.fd_cpr));
    const int kc = c - t * cpr;
    const int S = p.imgs_per_iter;

    const float2 d = __ldg(p.dx2 + t);
    const int z = kMode == kCodeU8 ? __ldg(p.zp + t) : 0;
    const float *s8 = p.s + kc * 8;          // read only on the exact route
    const float *rs8 = p.rs + kc * 8;
    // The parameter loads are issued here, in front of the dependency wait, but their values are first used after
    // the ring has been filled: a CTA that starts late (its wait is already satisfied) then has the parameter
    // loads and its first activation loads in flight together instead of one memory latency after the other.
    float4 r0 = make_float4(0.0f, 0.0f, 0.0f, 0.0f), r1 = r0;
    if (kFast) {
        r0 = __ldg(reinterpret_cast<const float4 *>(rs8));
        r1 = __ldg(reinterpret_cast<const float4 *>(rs8) + 1);
    }

    const long long x_img = static_cast<long long>(p.T) * p.K;          // elements per image of x
    const long long q_img = static_cast<long long>(p.T) * p.q_pitch;    // bytes per image of q
    const __half *xp = p.x + b * x_img + static_cast<long long>(t) * p.K + kc * 8;
    int8_t *qp = p.q + b * q_img + static_cast<long long>(t) * p.q_pitch + kc * 8;
    const long long x_step = S * x_img, q_step = S * q_img;

    // Everything above read only the layer's own parameters; x may come from the kernel before this one.
    griddep_wait();
    griddep_launch_dependents();

    const uint64_t pol_x = l2_policy_evict_first();
    // fill the ring: slot i holds image b + i*S (one commit group per slot, empty past the last image)
#pragma unroll
    for (int i = 0; i < D; ++i) {
        if (b + i * S < p.B) cp_async_16_hint(&ring[i][threadIdx.x], xp + i * x_step, pol_x);
        cp_async_commit();
    }
    float c8[8];
    if (kFast) {
        c8[0] = __fmul_rn(r0.x, d.y); c8[1] = __fmul_rn(r0.y, d.y); c8[2] = __fmul_rn(r0.z, d.y); c8[3] = __fmul_rn(r0.w, d.y);
        c8[4] = __fmul_rn(r1.x, d.y); c8[5] = __fmul_rn(r1.y, d.y); c8[6] = __fmul_rn(r1.z, d.y); c8[7] = __fmul_rn(r1.w, d.y);
    }
    int slot = 0;
    while (b < p.B) {
        cp_async_wait<D - 1>();                                   // the oldest group, i.e. this slot, has landed
        const uint4 v = ring[slot][threadIdx.x];
        *reinterpret_cast<uint2 *>(qp) = quantize8<kFast, kMode>(v, c8, s8, rs8, d.x, d.y, z);
        // refill the slot just consumed (its value has been used above) with the image D*S further on
        if (b + D * S < p.B) cp_async_16_hint(&ring[slot][threadIdx.x], xp + D * x_step, pol_x);
        cp_async_commit();
        slot = (slot + 1 == D) ? 0 : slot + 1;
        b += S;
        xp += x_step;
        qp += q_step;
    }
    cp_async_wait<0>();
}

// Generic path: any K, any alignment; one element per thread per step.
template <bool kFast, int kMode = kCodeS8>
__global__ void __launch_bounds__(256) ptq_quantize_scalar_kernel(QuantParams p)
{
    griddep_wait();
    griddep_launch_dependents();
    const long long total = p.M * p.K;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const long long m = i / p.K;
        const int k = static_cast<int>(i - m * p.K);
        const int t = static_cast<int>(m % p.T);
        const __half h = p.x[i];
        const float xf = __half2float(h);
        const unsigned short bits = __half_as_ushort(h);
        const int z = kMode == kCodeU8 ? __ldg(p.zp + t) : 0;
        int c;
        if (kFast && (bits & 0x7c00u) != 0x7c00u)
            c = quantize_fast<kMode>(xf, __ldg(p.s + k), __ldg(p.rs + k), __ldg(p.dx + t), __ldg(p.rdx + t), z);
        else
            c = quantize_ieee<kMode>(xf, __ldg(p.s + k), __ldg(p.dx + t), z);
        p.q[m * p.q_pitch + k] = static_cast<int8_t>(c);
    }
}

// Two adjacent 4-bit codes (held one per byte, row pitch `pitch`) into one byte, low nibble = even
// channel (the packing step of Appendix B.1): out[m, i] = (q[m, 2i+1] << 4) | (q[m, 2i] & 15); an odd K
// ends the row with a zero high nibble.
__global__ void __launch_bounds__(256) ptq_pack_int4_kernel(const int8_t *q, long long M, int K, int pitch,
                                                            uint8_t *out)
{
    const int pb = (K + 1) >> 1;
    const long long total = M * pb;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
        const long long m = i / pb;
        const int j = static_cast<int>(i - m * pb);
        const int8_t *row = q + m * pitch;
        const int lo = row[2 * j];
        const int hi = (2 * j + 1 < K) ? row[2 * j + 1] : 0;
        out[i] = static_cast<uint8_t>(((hi << 4) | (lo & 15)) & 0xff);
    }
}

}  // namespace ptq
