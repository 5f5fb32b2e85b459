// G1 + E1: integer GEMM on the 5th-generation tensor cores with the dequantization fused into
// the epilogue (Sec. 5.1:  Y = diag(Delta_W) (W-bar X-bar) diag(Delta_X);  Appendix B.1 parts 3-4).
//
//   acc[m,n] = sum_k q[m,k] * Wq[n,k]                       tcgen05.mma kind::i8, s32 in TMEM
//   y[m,n]   = fp16( float(acc) * dx[m mod T] * dw[n] + bias[n] )
//
// The rank-1 scaling is applied to the accumulator as it leaves TMEM, so neither the int32
// product nor an [M,N] step-size tensor ever reaches HBM.
//
// One persistent CTA per SM, 10 warps:
//   warp 0      TMA producer: A tile 128 x 128 B of codes and B tile BN x 128 B of weights per
//               stage, both written with the 128-byte swizzle, completion on a "full" mbarrier
//   warp 1      owns TMEM (512 columns = two 128 x 256 accumulators) and issues the MMAs; a
//               tcgen05.commit frees each shared-memory stage and publishes each accumulator
//   warps 2..9  epilogue: tcgen05.ld (lane quarter = warp % 4; the two warps of a quarter take
//               alternate 64-column steps), scale, convert, stage each step as one 32 x 64 fp16 box in
//               swizzled shared memory (128-byte rows) and write it with one TMA store
// While the epilogue drains accumulator i the MMA warp already fills accumulator i^1.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

namespace ptq {

constexpr int kBM = 128;                                  // rows per tile = TMEM lanes
constexpr int kBK = 128;                                  // bytes of K per stage row (one swizzle row)
constexpr int kMaxBN = 256;                               // columns per accumulator
constexpr int kStages = 4;
constexpr int kATileBytes = kBM * kBK;                    // 16 KB
constexpr int kBTileBytes = kMaxBN * kBK;                 // 32 KB
constexpr int kStageBytes = kATileBytes + kBTileBytes;
constexpr int kNumEpiWarps = 8;                           // two per TMEM lane quarter
constexpr int kEpiStepCols = 64;                          // accumulator columns a warp drains per step
constexpr int kStoreBoxCols = 32;                         // fp16 columns per TMA store box (64-byte rows)
constexpr int kStoreBoxBytes = 32 * kStoreBoxCols * 2;    // 32 rows x 64 B = 2 KB
constexpr int kStagingBytesPerWarp = 2 * kStoreBoxBytes;  // two boxes: one being filled while the other is stored
constexpr int kGemmThreads = 32 * (2 + kNumEpiWarps);
constexpr int kTmemCols = 512;
constexpr int kNumBarriers = 2 * kStages + 4;
// The streaming and CTA-pair kernels stage one 32-row x 64-column box per warp (128-byte rows, 128-byte
// swizzle) and store a whole 64-column step with one TMA store; the fused kernel uses the two 32-column
// boxes above.
#ifndef PTQ_STORE_BOX64
#define PTQ_STORE_BOX64 1
#endif
constexpr bool kStreamBox64 = PTQ_STORE_BOX64 != 0;
constexpr int kStreamBoxCols = kStreamBox64 ? 64 : kStoreBoxCols;
constexpr int kStreamStagingPerWarp = kStreamBox64 ? 32 * 128 : kStagingBytesPerWarp;
// Streaming kernel: per-tile copies of the weight steps (and of the bias, for layers that have one) in
// shared memory, double buffered by tile parity, so that the conversion loop reads them with broadcast
// shared-memory loads instead of global loads.  Layers with a bias run three stages to make room.
constexpr int kScaleBufBytes = kMaxBN * 4;                // one vector of one tile
constexpr int kGemmNumBarriers = kNumBarriers + 1;        // + the barrier that publishes the scale copies
// Two shapes of the shared memory: four stages and one staging box per epilogue warp, or three stages
// and two boxes per warp (a step then never waits for the store before it; chosen where the main loop
// of a tile is short, so that the epilogue is what must keep up).
__host__ __device__ constexpr int gemm_smem_bytes(int stages, int boxes, int has_bias)
{
    // no slack for alignment: the dynamic shared memory array is declared 1024-byte aligned (checked at run time)
    return stages * kStageBytes + boxes * kNumEpiWarps * kStreamStagingPerWarp + (has_bias ? 4 : 2) * kScaleBufBytes +
           kGemmNumBarriers * 8 + 16;
}
constexpr int kGemmSmemBytes = gemm_smem_bytes(kStages, 1, 0);
static_assert(kGemmSmemBytes <= 232448 && gemm_smem_bytes(kStages - 1, 2, 1) <= kGemmSmemBytes,
              "streaming GEMM kernel exceeds the shared memory of one CTA");

struct GemmParams {
    long long M;
    int N, K, T;
    int BN;            // columns per tile: multiple of 16; multiple of 64 when n_tiles > 1
    int n_tiles, m_tiles;
    int k_blocks;      // ceil(K / 128)
    int last_mmas;     // MMAs (K = 32 each) in the last k-block: ceil((K - 128 (k_blocks-1)) / 32)
    const float *dx;   // [T]
    const float *dw;   // [>= n_tiles*BN + 64], zero padded
    const float *bias; // same length, zeros when the layer has no bias
    int has_bias;      // 0: bias is all zeros and need not be read
    int stages;        // streaming kernel: shared-memory stages (3 or 4) ...
    int boxes;         // ... and staging boxes per epilogue warp (2 with three stages, 1 with four)
    __half *y;         // [M,N]
    int32_t *acc_out;  // [M,N] or nullptr (parity tap)
    unsigned *status;  // device status word
    int use_tma_store; // y is written by TMA (needs N % 8 == 0 and a 16-byte aligned y)
    int y_vec2;        // plain-store path may use 4-byte stores (N even, y 4-byte aligned)
    int y_vec8;        // plain-store path may use 16-byte stores (N % 8 == 0, y 16-byte aligned)
    // Asymmetric layers (zero offset per token position): the codes are unsigned, the tensor core
    // accumulates sum_k c * Wq, and the epilogue subtracts z[t] * sum_k Wq[n,k] to obtain the offset-free
    // accumulator sum_k (c - z[t]) * Wq[n,k] exactly (all int32).  nullptr for symmetric layers.
    const int *zp;     // [T]
    const int *wsum;   // [>= n_tiles*BN + 64] row sums of Wq, zero padded
    // Panel kernel only: a work unit is one 128-row panel of codes times `group` adjacent N tiles; `groups`
    // units cover a panel; the weight ring has `b_stages` slots of `b_stage_bytes` (= BN * 128) each.
    int group, groups;
    int b_stages, b_stage_bytes;
    FastDiv fd_T, fd_n_tiles, fd_groups;   // divisors T, n_tiles, groups (the GEMM kernels' loops)
};

// --- epilogue helpers -------------------------------------------------------------------------

// y = float(acc) * dx * dw + bias with one rounding per operation (mul, then fma).
__device__ __forceinline__ float dequant_one(uint32_t acc, float dxr, float dwn, float bn)
{
    return __fmaf_rn(__fmul_rn(__int2float_rn(static_cast<int>(acc)), dxr), dwn, bn);
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b)
{
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

// No "memory" clobber on purpose: the store stays ordered with the other volatile statements (the
// fence.proxy.async and the TMA store that follow it), while ordinary loads of the scale vectors may be
// scheduled across it, which is what keeps their latency off the conversion loop.
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
}

// Convert 32 accumulator columns of this thread's row and write them as the four 16-byte chunks of the
// row's 64-byte line in a staging box (chunk index XOR ((row >> 1) & 3): the 64-byte swizzle the store's
// tensor map expects, which also spreads the 32 rows over all banks).
__device__ __forceinline__ void convert_stage32(const uint32_t (&v)[32], float dxr, const float *dw,
                                                const float *bias, uint32_t row_addr, int lane)
{
    const uint32_t sw = static_cast<uint32_t>((lane >> 1) & 3);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
        const float4 w0 = __ldg(reinterpret_cast<const float4 *>(dw + 8 * jj));
        const float4 w1 = __ldg(reinterpret_cast<const float4 *>(dw + 8 * jj + 4));
        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(bias + 8 * jj));
        const float4 b1 = __ldg(reinterpret_cast<const float4 *>(bias + 8 * jj + 4));
        uint4 o;
        o.x = pack_half2(dequant_one(v[8 * jj + 0], dxr, w0.x, b0.x), dequant_one(v[8 * jj + 1], dxr, w0.y, b0.y));
        o.y = pack_half2(dequant_one(v[8 * jj + 2], dxr, w0.z, b0.z), dequant_one(v[8 * jj + 3], dxr, w0.w, b0.w));
        o.z = pack_half2(dequant_one(v[8 * jj + 4], dxr, w1.x, b1.x), dequant_one(v[8 * jj + 5], dxr, w1.y, b1.y));
        o.w = pack_half2(dequant_one(v[8 * jj + 6], dxr, w1.z, b1.z), dequant_one(v[8 * jj + 7], dxr, w1.w, b1.w));
        st_shared_v4(row_addr + ((static_cast<uint32_t>(jj) ^ sw) << 4), o);
    }
}

// Same for one half (32 columns) of a 128-byte row of a 64-column box: chunks 4*half .. 4*half+3, chunk
// index XOR (row & 7): the 128-byte swizzle.
__device__ __forceinline__ void convert_stage32_sw128(const uint32_t (&v)[32], float dxr, const float *dw,
                                                      const float *bias, uint32_t row_addr, int lane, int half)
{
    const uint32_t sw = static_cast<uint32_t>(lane & 7);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
        const float4 w0 = __ldg(reinterpret_cast<const float4 *>(dw + 8 * jj));
        const float4 w1 = __ldg(reinterpret_cast<const float4 *>(dw + 8 * jj + 4));
        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(bias + 8 * jj));
        const float4 b1 = __ldg(reinterpret_cast<const float4 *>(bias + 8 * jj + 4));
        uint4 o;
        o.x = pack_half2(dequant_one(v[8 * jj + 0], dxr, w0.x, b0.x), dequant_one(v[8 * jj + 1], dxr, w0.y, b0.y));
        o.y = pack_half2(dequant_one(v[8 * jj + 2], dxr, w0.z, b0.z), dequant_one(v[8 * jj + 3], dxr, w0.w, b0.w));
        o.z = pack_half2(dequant_one(v[8 * jj + 4], dxr, w1.x, b1.x), dequant_one(v[8 * jj + 5], dxr, w1.y, b1.y));
        o.w = pack_half2(dequant_one(v[8 * jj + 6], dxr, w1.z, b1.z), dequant_one(v[8 * jj + 7], dxr, w1.w, b1.w));
        st_shared_v4(row_addr + ((static_cast<uint32_t>(4 * half + jj) ^ sw) << 4), o);
    }
}

// Plain masked stores of 32 columns of this thread's row (any N, any alignment of y).
__device__ __forceinline__ void convert_store32_plain(const uint32_t (&v)[32], float dxr, const float *dw,
                                                      const float *bias, __half *yrow, int n_first, int N,
                                                      bool vec2)
{
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const int n = n_first + i;
        if (n >= N) break;
        const float a = dequant_one(v[i], dxr, __ldg(dw + i), __ldg(bias + i));
        const float b = dequant_one(v[i + 1], dxr, __ldg(dw + i + 1), __ldg(bias + i + 1));
        if (vec2 && n + 1 < N) {
            *reinterpret_cast<__half2 *>(yrow + n) = __floats2half2_rn(a, b);
        } else {
            yrow[n] = __float2half_rn(a);
            if (n + 1 < N) yrow[n + 1] = __float2half_rn(b);
        }
    }
}

// 16-byte stores of 32 columns of this thread's row straight from registers (N % 8 == 0 and a
// 16-byte aligned y): the thread's 64 contiguous bytes go out as four stores that L2 merges.
__device__ __forceinline__ void convert_store32_vec8(const uint32_t (&v)[32], float dxr, const float *dw,
                                                     const float *bias, __half *yrow, int n_first, int N)
{
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
        const int n = n_first + 8 * jj;
        if (n >= N) break;
        const float4 w0 = __ldg(reinterpret_cast<const float4 *>(dw + 8 * jj));
        const float4 w1 = __ldg(reinterpret_cast<const float4 *>(dw + 8 * jj + 4));
        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(bias + 8 * jj));
        const float4 b1 = __ldg(reinterpret_cast<const float4 *>(bias + 8 * jj + 4));
        uint4 o;
        o.x = pack_half2(dequant_one(v[8 * jj + 0], dxr, w0.x, b0.x), dequant_one(v[8 * jj + 1], dxr, w0.y, b0.y));
        o.y = pack_half2(dequant_one(v[8 * jj + 2], dxr, w0.z, b0.z), dequant_one(v[8 * jj + 3], dxr, w0.w, b0.w));
        o.z = pack_half2(dequant_one(v[8 * jj + 4], dxr, w1.x, b1.x), dequant_one(v[8 * jj + 5], dxr, w1.y, b1.y));
        o.w = pack_half2(dequant_one(v[8 * jj + 6], dxr, w1.z, b1.z), dequant_one(v[8 * jj + 7], dxr, w1.w, b1.w));
        *reinterpret_cast<uint4 *>(yrow + n) = o;
    }
}

__device__ __forceinline__ void store_acc32(const uint32_t (&v)[32], int32_t *arow, int n_first, int N)
{
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (n_first + i < N) arow[n_first + i] = static_cast<int32_t>(v[i]);
}

// Epilogue of one 128 x BN accumulator for one warp (its 32-lane quarter).  `tmem_row` addresses the
// warp's lanes and the accumulator's first column.  The warp takes every second 64-column step
// (`col_half` selects which) and writes each step as two 32-column boxes; with two staging boxes per
// warp a TMA store is still reading one box while the next is being filled, so the latency of a store
// is not on the warp's critical path.  Returns the updated count of staged boxes.
// kLowReg = false keeps both TMEM loads of a step in flight (64 accumulator registers);
// kLowReg = true loads 32 columns at a time (for kernels whose thread count caps the registers).
template <bool kDebugAcc, bool kLowReg = false, bool kBox64 = false>
__device__ __forceinline__ uint32_t epilogue_tile(const GemmParams &p, const CUtensorMap *tmY, uint32_t tmem_row,
                                                  long long m_row0, int n0, float dxr, uint32_t staging,
                                                  uint32_t nboxes, int lane, int col_half, int zr = 0)
{
    const long long m = m_row0 + lane;
    const bool row_ok = m < p.M;
    for (int c0 = col_half * kEpiStepCols; c0 < p.BN; c0 += 2 * kEpiStepCols) {
        const int n_first = n0 + c0;
        uint32_t v0[32], v1[32];
        tmem_ld_32x32(tmem_row + c0, v0);
        if (!kLowReg) tmem_ld_32x32(tmem_row + c0 + 32, v1);
        tmem_ld_wait();
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t (&v)[32] = (half == 0 || kLowReg) ? v0 : v1;
            if (kLowReg && half == 1) {
                tmem_ld_32x32(tmem_row + c0 + 32, v0);
                tmem_ld_wait();
            }
            const int n_half = n_first + 32 * half;
            if (p.zp != nullptr) {
                // offset-free accumulator: acc - z[t] * sum_k Wq[n,k]
#pragma unroll
                for (int i4 = 0; i4 < 8; ++i4) {
                    const int4 ws = __ldg(reinterpret_cast<const int4 *>(p.wsum + n_half) + i4);
                    v[4 * i4 + 0] -= static_cast<uint32_t>(zr * ws.x);
                    v[4 * i4 + 1] -= static_cast<uint32_t>(zr * ws.y);
                    v[4 * i4 + 2] -= static_cast<uint32_t>(zr * ws.z);
                    v[4 * i4 + 3] -= static_cast<uint32_t>(zr * ws.w);
                }
            }
            if (kDebugAcc) {
                if (p.acc_out != nullptr && row_ok) store_acc32(v, p.acc_out + m * p.N, n_half, p.N);
            }
            if (kBox64 && p.use_tma_store) {
                // one 64-column box per step: wait until the previous step's store has read the box, fill
                // its two halves, store once
                if (half == 0) {
                    if (nboxes >= 1u && lane == 0) bulk_wait_group_read<0>();
                    __syncwarp();
                }
                convert_stage32_sw128(v, dxr, p.dw + n_half, p.bias + n_half, staging + static_cast<uint32_t>(lane) * 128u,
                                      lane, half);
                if (half == 1) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        if (n_first < p.N && m_row0 < p.M)
                            tma_store_2d(tmY, n_first, static_cast<int>(m_row0), staging);   // clipped at N and M
                        bulk_commit_group();
                    }
                    ++nboxes;
                }
            } else if (p.use_tma_store) {
                const uint32_t box = staging + (nboxes & 1u) * kStoreBoxBytes;
                if (nboxes >= 2u && lane == 0) bulk_wait_group_read<1>();   // the store that last used this box has read it
                __syncwarp();
                convert_stage32(v, dxr, p.dw + n_half, p.bias + n_half, box + static_cast<uint32_t>(lane) * 64u, lane);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (n_half < p.N && m_row0 < p.M)
                        tma_store_2d(tmY, n_half, static_cast<int>(m_row0), box);   // clipped at N and M
                    bulk_commit_group();
                }
                ++nboxes;
            } else if (row_ok && p.y_vec8) {
                convert_store32_vec8(v, dxr, p.dw + n_half, p.bias + n_half, p.y + m * p.N, n_half, p.N);
            } else if (row_ok) {
                convert_store32_plain(v, dxr, p.dw + n_half, p.bias + n_half, p.y + m * p.N, n_half, p.N,
                                      p.y_vec2 != 0);
            }
        }
    }
    return nboxes;
}

// Epilogue of one 128 x BN accumulator for one warp of the streaming kernel (TMA-store path); the warp
// takes the 64-column steps c_begin, c_begin + c_stride, ...  As
// epilogue_tile with one 64-column box per step, except that the weight steps (and the bias) of the tile
// are read from their copy in shared memory (`dw_s`, `bias_s`: this tile's BN floats, indexed by the
// column inside the tile) with broadcast loads: no global-memory latency sits in the conversion loop.
// With two staging boxes per warp (`two_boxes`) a step never waits for the store of the step before it.
__device__ __forceinline__ uint32_t pack_half2(float2 r) { return pack_half2(r.x, r.y); }

// Two accumulators at a time with the packed binary32 instructions of sm_100 (each lane of a packed
// operation is the ordinary correctly rounded one): (float(acc) * dx) * dw + bias, then one conversion
// of the pair to binary16.  All 64 columns are converted before the first store, which leaves the
// instruction scheduler free to interleave the eight independent groups.
__device__ __forceinline__ void convert_stage64_sw128(const uint32_t (&v0)[32], const uint32_t (&v1)[32], float dxr,
                                                      const float4 *dw_s, const float4 *bias_s, uint32_t row_addr,
                                                      int lane)
{
    const uint32_t sw = static_cast<uint32_t>(lane & 7);
    const float2 dx2 = make_float2(dxr, dxr);
    uint4 o[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
        const uint32_t (&v)[32] = jj < 4 ? v0 : v1;
        const int j8 = 8 * (jj & 3);
        const float4 w0 = dw_s[2 * jj], w1 = dw_s[2 * jj + 1];
        float4 b0 = make_float4(0.0f, 0.0f, 0.0f, 0.0f), b1 = b0;
        if (bias_s != nullptr) {
            b0 = bias_s[2 * jj];
            b1 = bias_s[2 * jj + 1];
        }
        auto f = [](uint32_t a) { return __int2float_rn(static_cast<int>(a)); };
        const float2 a0 = __fmul2_rn(make_float2(f(v[j8 + 0]), f(v[j8 + 1])), dx2);
        const float2 a1 = __fmul2_rn(make_float2(f(v[j8 + 2]), f(v[j8 + 3])), dx2);
        const float2 a2 = __fmul2_rn(make_float2(f(v[j8 + 4]), f(v[j8 + 5])), dx2);
        const float2 a3 = __fmul2_rn(make_float2(f(v[j8 + 6]), f(v[j8 + 7])), dx2);
        o[jj].x = pack_half2(__ffma2_rn(a0, make_float2(w0.x, w0.y), make_float2(b0.x, b0.y)));
        o[jj].y = pack_half2(__ffma2_rn(a1, make_float2(w0.z, w0.w), make_float2(b0.z, b0.w)));
        o[jj].z = pack_half2(__ffma2_rn(a2, make_float2(w1.x, w1.y), make_float2(b1.x, b1.y)));
        o[jj].w = pack_half2(__ffma2_rn(a3, make_float2(w1.z, w1.w), make_float2(b1.z, b1.w)));
    }
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) st_shared_v4(row_addr + ((static_cast<uint32_t>(jj) ^ sw) << 4), o[jj]);
}

template <bool kDebugAcc>
__device__ __forceinline__ uint32_t epilogue_tile_stream(const GemmParams &p, const CUtensorMap *tmY, uint32_t tmem_row,
                                                         long long m_row0, int n0, float dxr, uint32_t staging,
                                                         const float *dw_s, const float *bias_s, uint32_t nboxes,
                                                         int lane, int c_begin, int c_stride, int zr, bool two_boxes)
{
    const long long m = m_row0 + lane;
    const bool row_ok = m < p.M;
    for (int c0 = c_begin; c0 < p.BN; c0 += c_stride) {
        const int n_first = n0 + c0;
        uint32_t v0[32], v1[32];
        tmem_ld_32x32(tmem_row + c0, v0);
        tmem_ld_32x32(tmem_row + c0 + 32, v1);
        tmem_ld_wait();
        if (p.zp != nullptr) {
            // offset-free accumulator: acc - z[t] * sum_k Wq[n,k]
#pragma unroll
            for (int i4 = 0; i4 < 8; ++i4) {
                const int4 wa = __ldg(reinterpret_cast<const int4 *>(p.wsum + n_first) + i4);
                const int4 wb = __ldg(reinterpret_cast<const int4 *>(p.wsum + n_first + 32) + i4);
                v0[4 * i4 + 0] -= static_cast<uint32_t>(zr * wa.x);
                v0[4 * i4 + 1] -= static_cast<uint32_t>(zr * wa.y);
                v0[4 * i4 + 2] -= static_cast<uint32_t>(zr * wa.z);
                v0[4 * i4 + 3] -= static_cast<uint32_t>(zr * wa.w);
                v1[4 * i4 + 0] -= static_cast<uint32_t>(zr * wb.x);
                v1[4 * i4 + 1] -= static_cast<uint32_t>(zr * wb.y);
                v1[4 * i4 + 2] -= static_cast<uint32_t>(zr * wb.z);
                v1[4 * i4 + 3] -= static_cast<uint32_t>(zr * wb.w);
            }
        }
        if (kDebugAcc) {
            if (p.acc_out != nullptr && row_ok) {
                store_acc32(v0, p.acc_out + m * p.N, n_first, p.N);
                store_acc32(v1, p.acc_out + m * p.N, n_first + 32, p.N);
            }
        }
        // the store that last used this box must have read it before it is refilled
        const uint32_t box = staging + ((two_boxes && (nboxes & 1u)) ? static_cast<uint32_t>(kStreamStagingPerWarp) : 0u);
        if (lane == 0) {
            if (two_boxes) {
                if (nboxes >= 2u) bulk_wait_group_read<1>();
            } else if (nboxes >= 1u) {
                bulk_wait_group_read<0>();
            }
        }
        __syncwarp();
        convert_stage64_sw128(v0, v1, dxr, reinterpret_cast<const float4 *>(dw_s + c0),
                              bias_s != nullptr ? reinterpret_cast<const float4 *>(bias_s + c0) : nullptr,
                              box + static_cast<uint32_t>(lane) * 128u, lane);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            if (n_first < p.N && m_row0 < p.M)
                tma_store_2d(tmY, n_first, static_cast<int>(m_row0), box);   // clipped at N and M
            bulk_commit_group();
        }
        ++nboxes;
    }
    return nboxes;
}

// The activation step (and, on asymmetric layers, the zero offset) of this thread's row of row tile `m_tile`.
// The epilogue loops request it one tile ahead, so that neither the load's latency nor the modulo sits between
// two tiles.  B*T < 2^31 (checked at the boundary), so the row index fits 32 bits.
struct RowStep {
    float dx;
    int z;
};
__device__ __forceinline__ RowStep load_row_step(const GemmParams &p, int m_tile, int quarter, int lane)
{
    // Unconditional loads from clamped indices: a load under a condition is followed by a select that waits for
    // it, which would put the load's latency back into the loop.  Rows beyond M are never stored, so what they
    // get does not matter.
    RowStep r = {0.0f, 0};
    long long m = static_cast<long long>(m_tile) * kBM + quarter * 32 + lane;
    if (m >= p.M) m = p.M - 1;
    const unsigned mu = static_cast<unsigned>(m);
    const unsigned t = mu - fd_div(mu, p.fd_T) * p.fd_T.d;
    r.dx = __ldg(p.dx + t);
    if (p.zp != nullptr) r.z = __ldg(p.zp + t);
    return r;
}

// --- epilogue in two teams -----------------------------------------------------------------------
//
// The arithmetic of a 64-column step (int32 -> binary32, two multiplies, conversion to binary16) keeps a
// scheduler's issue port busy for about 400 cycles per warp, and around it sit waits that nothing else
// of the same warp can fill (TMEM data arriving, the fence, the store issue, the previous store reading
// its box).  With all eight warps on one tile, two warps per scheduler run those steps side by side and
// the tile's epilogue lasts as long as the main loop of a K = 768 tile; the MMA thread then waits for
// the accumulator.  In team mode the eight warps form two teams of four (one warp per TMEM lane quarter
// and per scheduler); team b drains accumulator b, i.e. every second tile of the CTA, all 64-column
// steps of it.  A tile's epilogue takes longer, but it has two main loops' time to finish, and one
// team's waits are filled by the other team's arithmetic.  Used when a CTA has several tiles and the
// main loop of a tile is short (K <= 384), i.e. where the epilogue sets the pace: 7-8 % on such layers
// with many rows; layers with a long main loop are bounded elsewhere and gain nothing.
//
// The team's copy of the tile's weight steps (and bias) lives in scale buffer b; a named barrier over
// the team's 128 threads publishes it (together with the vote on the bounded waits, so that the four
// warps leave the loop together or not at all) and a second one, at the end of the tile, keeps the
// next tile's values from overwriting it while a slower warp still reads.
__device__ __forceinline__ bool team_all(bool pred, int team)
{
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, %2, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(pred)), "r"(1 + team)
        : "memory");
    return r != 0u;
}
__device__ __forceinline__ void team_sync(int team) { asm volatile("bar.sync %0, 128;" ::"r"(1 + team) : "memory"); }

// The CTA's tiles in the order the MMA thread produces them.
struct StreamCursor {
    int tile, total, step, n_tiles;
    FastDiv fd;
    __device__ bool valid() const { return tile < total; }
    __device__ void advance() { tile += step; }
    __device__ int m_tile() const { return static_cast<int>(fd_div(static_cast<unsigned>(tile), fd)); }
    __device__ int n_tile() const { return tile - m_tile() * n_tiles; }
};

template <bool kDebugAcc, class Cursor>
__device__ __forceinline__ void epilogue_team_loop(const GemmParams &p, const CUtensorMap *tmY, Cursor cur, uint32_t tmem_base,
                                                   uint32_t tfull_bar0, uint32_t tempty_bar0, float *scale_s,
                                                   uint32_t staging, bool two_boxes, volatile uint32_t *abort_flag,
                                                   int warp, int lane)
{
    const int quarter = warp & 3;                       // TMEM lanes [32*quarter, 32*quarter+32)
    const int team = (warp - 2) >> 2;                   // = the accumulator buffer this team drains
    const int tt = static_cast<int>(threadIdx.x) - 64 - team * 128;   // 0 .. 127 inside the team
    float *dw_buf = scale_s + team * kMaxBN;
    float *bias_buf = scale_s + (2 + team) * kMaxBN;
    const uint32_t tfull = tfull_bar0 + 8u * team, tempty = tempty_bar0 + 8u * team;
    if (team == 1 && cur.valid()) cur.advance();        // team 1 starts at the CTA's second tile
    float dw_next[2] = {0.0f, 0.0f}, bias_next[2] = {0.0f, 0.0f};
    auto fetch_scales = [&](const Cursor &c) {
        // unconditional loads from clamped indices (see load_row_step); past the last tile the values are not used
        const int n0 = c.valid() ? c.n_tile() * p.BN : 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int col = min(tt + 128 * h, p.BN - 1);
            dw_next[h] = __ldg(p.dw + n0 + col);
            if (p.has_bias) bias_next[h] = __ldg(p.bias + n0 + col);
        }
    };
    fetch_scales(cur);
    RowStep rs_next = {0.0f, 0};
    if (cur.valid()) rs_next = load_row_step(p, cur.m_tile(), quarter, lane);
    uint32_t tphase = 0, nboxes = 0;
    while (cur.valid()) {                               // the same for every thread of the team
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int col = tt + 128 * h;
            if (col < p.BN) {
                dw_buf[col] = dw_next[h];
                if (p.has_bias) bias_buf[col] = bias_next[h];
            }
        }
        const int m_tile = cur.m_tile(), n_tile = cur.n_tile();
        cur.advance();
        if (cur.valid()) cur.advance();                 // the team's next tile: its scales stay in flight during this one
        fetch_scales(cur);
        const long long m_row0 = static_cast<long long>(m_tile) * kBM + quarter * 32;
        const float dxr = rs_next.dx;
        const int zr = rs_next.z;
        if (cur.valid()) rs_next = load_row_step(p, cur.m_tile(), quarter, lane);
        bool got = mbar_wait(tfull, tphase, abort_flag, p.status);
        got = team_all(got, team);                      // also: the team's scale copies are complete and visible
        if (!got) break;
        tc_fence_after_sync();
        const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(team) * kMaxBN;
        nboxes = epilogue_tile_stream<kDebugAcc>(p, tmY, tmem_row, m_row0, n_tile * p.BN, dxr, staging, dw_buf,
                                                 p.has_bias ? bias_buf : nullptr, nboxes, lane, 0, kEpiStepCols, zr, two_boxes);
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty);
        tphase ^= 1u;
        team_sync(team);                                // every warp of the team is done reading the scale copies
    }
    if (lane == 0) bulk_wait_group<0>();                // all of this thread's stores have completed
}

// --- the kernel ---------------------------------------------------------------------------------

template <bool kDebugAcc, bool kTeams = false>
__global__ void __launch_bounds__(kGemmThreads, 1)
ptq_gemm_dequant_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                        const __grid_constant__ CUtensorMap tmY, const GemmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);                        // swizzled tiles need 1024-byte alignment
    if ((base & 1023u) != 0u) {
        // never expected (the array is declared 1024-byte aligned); the layout below has no slack for it
        if (threadIdx.x == 0) atomicOr(p.status, PTQ_DEV_SMEM_ALIGN);
        return;
    }
    const uint32_t nstages = static_cast<uint32_t>(p.stages);
    const bool two_boxes = p.boxes == 2;
    const uint32_t staging_off = nstages * kStageBytes;
    const uint32_t scale_off = staging_off + static_cast<uint32_t>(p.boxes) * kNumEpiWarps * kStreamStagingPerWarp;
    const uint32_t bar_off = scale_off + (p.has_bias ? 4 : 2) * kScaleBufBytes;
    const uint32_t staging_base = base + staging_off;
    const uint32_t bar_base = base + bar_off;
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (kStages + s); };
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kStages + b); };
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kStages + 2 + b); };
    const uint32_t scale_bar = bar_base + 8u * kNumBarriers;
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(smem_raw + bar_off + kGemmNumBarriers * 8);
    volatile uint32_t *abort_flag = tmem_holder + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < nstages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), kTeams ? kNumEpiWarps / 2 : kNumEpiWarps);   // in team mode one team drains a buffer
        }
        mbar_init(scale_bar, kNumEpiWarps);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmW);
        if (p.use_tma_store) prefetch_tensormap(&tmY);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_holder)), kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    // The set-up above touched nothing another kernel writes.  From here on the codes (and, for the
    // dynamic comparator, the row steps) of the quantize kernel launched just before are read.
    griddep_wait();
    griddep_launch_dependents();

    const int total_tiles = p.m_tiles * p.n_tiles;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int m_tile = static_cast<int>(fd_div(static_cast<unsigned>(tile), p.fd_n_tiles));
                const int n_tile = tile - m_tile * p.n_tiles;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a_dst = base + stage * kStageBytes;
                    mbar_arrive_expect_tx(full_bar(stage), static_cast<uint32_t>(kATileBytes + p.BN * kBK));
                    tma_load_2d(a_dst, &tmA, kb * kBK, m_tile * kBM, full_bar(stage));
                    tma_load_2d(a_dst + kATileBytes, &tmW, kb * kBK, n_tile * p.BN, full_bar(stage));
                    ++issued;
                    if (++stage == nstages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok) {
                // Error path only: let this thread's own loads land before the CTA gives up its
                // shared memory (bounded; each stage's last load is at most microseconds away).
                for (uint32_t s = 0; s < nstages; ++s) {
                    const uint32_t uses = (issued + nstages - 1u - s) / nstages;
                    if (uses == 0u) continue;
                    for (int i = 0; i < 200000 && !mbar_try_wait(full_bar(s), (uses - 1u) & 1u); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_s8(kBM, p.BN, p.zp != nullptr);   // unsigned codes on asymmetric layers
            uint32_t stage = 0, phase = 0, buf = 0, bphase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(tempty_bar(buf), bphase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * kMaxBN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t a_addr = base + stage * kStageBytes;
                    const uint64_t a_desc = make_smem_desc_sw128(a_addr);
                    const uint64_t b_desc = make_smem_desc_sw128(a_addr + kATileBytes);
                    const int nmma = (kb == p.k_blocks - 1) ? p.last_mmas : (kBK / 32);
                    mma_i8_ss_kblock(d_tmem, a_desc, b_desc, idesc, kb != 0 ? 1u : 0u, nmma);
                    mma_commit(empty_bar(stage));    // the stage is free once these MMAs have read it
                    if (++stage == nstages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                mma_commit(tfull_bar(buf));          // accumulator complete
                buf ^= 1u;
                if (buf == 0u) bphase ^= 1u;
            }
        }
    } else if (kTeams) {
        // ------------------------------------------------------------------ epilogue warps, two teams (TMA stores only)
        const StreamCursor cur{static_cast<int>(blockIdx.x), total_tiles, static_cast<int>(gridDim.x), p.n_tiles, p.fd_n_tiles};
        epilogue_team_loop<kDebugAcc>(p, &tmY, cur, tmem_base, tfull_bar(0), tempty_bar(0),
                                      reinterpret_cast<float *>(smem_raw + scale_off),
                                      staging_base + static_cast<uint32_t>(warp - 2) * static_cast<uint32_t>(p.boxes) * kStreamStagingPerWarp,
                                      two_boxes, abort_flag, warp, lane);
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;                // TMEM lanes [32*quarter, 32*quarter+32)
        const int col_half = (warp - 2) >> 2;        // which of the alternating 64-column boxes
        const int et = static_cast<int>(threadIdx.x) - 64;                 // 0 .. 255 among the epilogue threads
        const uint32_t staging = staging_base + static_cast<uint32_t>(warp - 2) * static_cast<uint32_t>(p.boxes) * kStreamStagingPerWarp;
        float *scale_s = reinterpret_cast<float *>(smem_raw + scale_off);   // [2][BN] steps, then [2][BN] bias
        // The weight step (and bias) of one column of tile `tile`: fetched into registers one tile ahead ...
        float dw_next = 0.0f, bias_next = 0.0f;
        auto fetch_scales = [&](int tile) {
            // unconditional loads from clamped indices (see load_row_step); past the last tile the values are not used
            const unsigned tl = tile < total_tiles ? static_cast<unsigned>(tile) : 0u;
            const int n = static_cast<int>(tl - fd_div(tl, p.fd_n_tiles) * p.fd_n_tiles.d) * p.BN + min(et, p.BN - 1);
            dw_next = __ldg(p.dw + n);
            if (p.has_bias) bias_next = __ldg(p.bias + n);
        };
        // ... and published in buffer `b` once every warp is done with the tile that used that buffer last
        auto publish_scales = [&](uint32_t b) {
            if (et < p.BN) {
                scale_s[b * kMaxBN + et] = dw_next;
                if (p.has_bias) scale_s[(2 + b) * kMaxBN + et] = bias_next;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(scale_bar);
        };
        uint32_t buf = 0, bphase = 0, nboxes = 0, it = 0;
        if (p.use_tma_store) {
            fetch_scales(blockIdx.x);
            publish_scales(0u);
        }
        RowStep rs_next = load_row_step(p, static_cast<int>(fd_div(blockIdx.x, p.fd_n_tiles)), quarter, lane);
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++it) {
            const int tile_next = tile + static_cast<int>(gridDim.x);
            if (p.use_tma_store) fetch_scales(tile_next);                            // in flight during this tile
            const int m_tile = static_cast<int>(fd_div(static_cast<unsigned>(tile), p.fd_n_tiles));
            const int n_tile = tile - m_tile * p.n_tiles;
            const long long m_row0 = static_cast<long long>(m_tile) * kBM + quarter * 32;
            const float dxr = rs_next.dx;
            const int zr = rs_next.z;
            if (tile_next < total_tiles)
                rs_next = load_row_step(p, static_cast<int>(fd_div(static_cast<unsigned>(tile_next), p.fd_n_tiles)), quarter, lane);
            bool got = true;
            // every epilogue warp has written its share of this tile's scale copies (arrival `it` of the barrier)
            if (p.use_tma_store) got = mbar_wait(scale_bar, it & 1u, abort_flag, p.status);
            got = got && mbar_wait(tfull_bar(buf), bphase, abort_flag, p.status);
            got = __all_sync(0xffffffffu, got);
            if (!got) break;
            tc_fence_after_sync();
            const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * kMaxBN;
            if (p.use_tma_store) {
                const float *dw_s = scale_s + (it & 1u) * kMaxBN;
                const float *bias_s = p.has_bias ? scale_s + (2u + (it & 1u)) * kMaxBN : nullptr;
                nboxes = epilogue_tile_stream<kDebugAcc>(p, &tmY, tmem_row, m_row0, n_tile * p.BN, dxr, staging, dw_s,
                                                         bias_s, nboxes, lane, col_half * kEpiStepCols, 2 * kEpiStepCols, zr, two_boxes);
            } else {
                nboxes = epilogue_tile<kDebugAcc, false, kStreamBox64>(p, &tmY, tmem_row, m_row0, n_tile * p.BN, dxr,
                                                                       staging, nboxes, lane, col_half, zr);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            buf ^= 1u;
            if (buf == 0u) bphase ^= 1u;
            // the next tile's scales go to the other buffer: every warp is past its reads of that buffer,
            // because it has passed this tile's wait on scale_bar, which needed every warp's arrival
            if (p.use_tma_store) publish_scales((it + 1u) & 1u);
        }
        if (lane == 0) bulk_wait_group<0>();         // all of this thread's stores have completed
    }

    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// --- panel variant: the codes of a row panel stay in shared memory ------------------------------
//
// Same computation as the streaming kernel for layers with several N tiles and K <= 768.  A work unit
// is one 128-row panel of codes (all its k-blocks, k_blocks x 16 KB, loaded once) times `group`
// adjacent N tiles; only the weight tiles stream through a ring of stages.  Per output tile a CTA then
// fetches BN x K bytes instead of (128 + BN) x K: a third less operand traffic between L2 and the SMs,
// which is what the streaming kernel's MMA thread waits on (and what costs energy under the power
// cap).  `group` is chosen by the host so that the units divide evenly over the CTAs; the units of one
// panel go to neighbouring CTAs, which read the panel from L2 at about the same time.
//
// Barriers: afull/aempty per panel k-block (one phase per unit: the MMA thread frees k-block kb with a
// commit after the unit's LAST tile has read it, so the next unit's panel arrives k-block by k-block
// while that tile still runs), bfull/bempty per weight stage, tfull/tempty per accumulator, one for
// the scale copies.  The producer interleaves the panel loads with the first tile's weight loads so
// that a wait for a late panel slot never holds back weights whose stage is free.
constexpr int kPanelMaxKBlocks = 6;                       // panel of at most 96 KB (K <= 768)
constexpr int kPanelMaxBStages = 6;
constexpr int kPanelNumBarriers = 2 * kPanelMaxKBlocks + 2 * kPanelMaxBStages + 4 + 1;
constexpr int kPanelSmemLimit = 232448;                   // 227 KB opt-in maximum per CTA
__host__ __device__ constexpr int panel_smem_bytes(int k_blocks, int b_stages, int b_stage_bytes, int boxes, int has_bias)
{
    return k_blocks * kATileBytes + b_stages * b_stage_bytes + boxes * kNumEpiWarps * kStreamStagingPerWarp +
           (has_bias ? 4 : 2) * kScaleBufBytes + kPanelNumBarriers * 8 + 16;
}

template <bool kDebugAcc>
__global__ void __launch_bounds__(kGemmThreads, 1)
ptq_gemm_dequant_panel_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                              const __grid_constant__ CUtensorMap tmY, const GemmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if ((base & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicOr(p.status, PTQ_DEV_SMEM_ALIGN);
        return;
    }
    const uint32_t nb = static_cast<uint32_t>(p.b_stages);
    const uint32_t b_bytes = static_cast<uint32_t>(p.b_stage_bytes);
    const bool two_boxes = p.boxes == 2;
    const uint32_t b_off = static_cast<uint32_t>(p.k_blocks) * kATileBytes;
    const uint32_t staging_off = b_off + nb * b_bytes;
    const uint32_t scale_off = staging_off + static_cast<uint32_t>(p.boxes) * kNumEpiWarps * kStreamStagingPerWarp;
    const uint32_t bar_off = scale_off + (p.has_bias ? 4 : 2) * kScaleBufBytes;
    const uint32_t bar_base = base + bar_off;
    auto afull_bar = [&](uint32_t kb) { return bar_base + 8u * kb; };
    auto aempty_bar = [&](uint32_t kb) { return bar_base + 8u * (kPanelMaxKBlocks + kb); };
    auto bfull_bar = [&](uint32_t s) { return bar_base + 8u * (2 * kPanelMaxKBlocks + s); };
    auto bempty_bar = [&](uint32_t s) { return bar_base + 8u * (2 * kPanelMaxKBlocks + kPanelMaxBStages + s); };
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kPanelMaxKBlocks + 2 * kPanelMaxBStages + b); };
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kPanelMaxKBlocks + 2 * kPanelMaxBStages + 2 + b); };
    const uint32_t scale_bar = bar_base + 8u * (kPanelNumBarriers - 1);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(smem_raw + bar_off + kPanelNumBarriers * 8);
    volatile uint32_t *abort_flag = tmem_holder + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (uint32_t kb = 0; kb < static_cast<uint32_t>(p.k_blocks); ++kb) {
            mbar_init(afull_bar(kb), 1);
            mbar_init(aempty_bar(kb), 1);
        }
        for (uint32_t s = 0; s < nb; ++s) {
            mbar_init(bfull_bar(s), 1);
            mbar_init(bempty_bar(s), 1);
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), kNumEpiWarps);
        }
        mbar_init(scale_bar, kNumEpiWarps);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmW);
        prefetch_tensormap(&tmY);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_holder)), kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    // From here on the codes (and, for the dynamic comparator, the row steps) of the kernel before are read.
    griddep_wait();
    griddep_launch_dependents();

    const int units = p.m_tiles * p.groups;
    // unit u -> panel u / groups, N tiles [first, first + count)
    auto unit_panel = [&](int u) { return static_cast<int>(fd_div(static_cast<unsigned>(u), p.fd_groups)); };
    auto unit_first = [&](int u) { return (u - unit_panel(u) * p.groups) * p.group; };
    auto unit_count = [&](int u) {
        const int left = p.n_tiles - unit_first(u);
        return left < p.group ? left : p.group;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, sphase = 0, uph = 0, b_issued = 0, a_units = 0;
            int a_kb_issued = 0;                 // panel k-blocks issued for the unit in progress
            bool ok = true;
            for (int unit = blockIdx.x; unit < units && ok; unit += gridDim.x, uph ^= 1u) {
                const int m_tile = unit_panel(unit);
                const int n_first = unit_first(unit), n_count = unit_count(unit);
                a_kb_issued = 0;
                for (int j = 0; j < n_count && ok; ++j) {
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (j == 0) {
                            // slot kb of the panel: free once the previous unit's last tile has read it
                            if (!mbar_wait(aempty_bar(kb), uph ^ 1u, abort_flag, p.status)) {
                                ok = false;
                                break;
                            }
                            mbar_arrive_expect_tx(afull_bar(kb), static_cast<uint32_t>(kATileBytes));
                            tma_load_2d(base + static_cast<uint32_t>(kb) * kATileBytes, &tmA, kb * kBK, m_tile * kBM,
                                        afull_bar(kb));
                            ++a_kb_issued;
                        }
                        if (!mbar_wait(bempty_bar(stage), sphase ^ 1u, abort_flag, p.status)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(bfull_bar(stage), b_bytes);
                        tma_load_2d(base + b_off + stage * b_bytes, &tmW, kb * kBK, (n_first + j) * p.BN, bfull_bar(stage));
                        ++b_issued;
                        if (++stage == nb) {
                            stage = 0;
                            sphase ^= 1u;
                        }
                    }
                }
                if (ok) ++a_units;
            }
            if (!ok) {
                // Error path only: let this thread's own loads land before the CTA gives up its shared memory (bounded).
                for (uint32_t s = 0; s < nb; ++s) {
                    const uint32_t uses = (b_issued + nb - 1u - s) / nb;
                    if (uses == 0u) continue;
                    for (int i = 0; i < 200000 && !mbar_try_wait(bfull_bar(s), (uses - 1u) & 1u); ++i) {
                    }
                }
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    const uint32_t uses = a_units + (kb < a_kb_issued ? 1u : 0u);
                    if (uses == 0u) continue;
                    for (int i = 0; i < 200000 && !mbar_try_wait(afull_bar(kb), (uses - 1u) & 1u); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_s8(kBM, p.BN, p.zp != nullptr);
            uint32_t stage = 0, sphase = 0, uph = 0, buf = 0, bphase = 0;
            bool ok = true;
            for (int unit = blockIdx.x; unit < units && ok; unit += gridDim.x, uph ^= 1u) {
                const int n_count = unit_count(unit);
                for (int j = 0; j < n_count && ok; ++j) {
                    if (!mbar_wait(tempty_bar(buf), bphase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + buf * kMaxBN;
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (j == 0 && !mbar_wait(afull_bar(kb), uph, abort_flag, p.status)) {
                            ok = false;
                            break;
                        }
                        if (!mbar_wait(bfull_bar(stage), sphase, abort_flag, p.status)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint64_t a_desc = make_smem_desc_sw128(base + static_cast<uint32_t>(kb) * kATileBytes);
                        const uint64_t b_desc = make_smem_desc_sw128(base + b_off + stage * b_bytes);
                        const int nmma = (kb == p.k_blocks - 1) ? p.last_mmas : (kBK / 32);
                        mma_i8_ss_kblock(d_tmem, a_desc, b_desc, idesc, kb != 0 ? 1u : 0u, nmma);
                        mma_commit(bempty_bar(stage));                       // the weight stage is free once these MMAs have read it
                        if (j == n_count - 1) mma_commit(aempty_bar(kb));    // and, after the unit's last tile, so is the panel slot
                        if (++stage == nb) {
                            stage = 0;
                            sphase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    mma_commit(tfull_bar(buf));          // accumulator complete
                    buf ^= 1u;
                    if (buf == 0u) bphase ^= 1u;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;
        const int et = static_cast<int>(threadIdx.x) - 64;
        const uint32_t staging = base + staging_off + static_cast<uint32_t>(warp - 2) * static_cast<uint32_t>(p.boxes) * kStreamStagingPerWarp;
        float *scale_s = reinterpret_cast<float *>(smem_raw + scale_off);   // [2][BN] steps, then [2][BN] bias
        float dw_next = 0.0f, bias_next = 0.0f;
        auto fetch_scales = [&](int n_tile) {
            const int n = n_tile * p.BN + min(et, p.BN - 1);      // unconditional, clamped (see load_row_step)
            dw_next = __ldg(p.dw + n);
            if (p.has_bias) bias_next = __ldg(p.bias + n);
        };
        auto publish_scales = [&](uint32_t b) {
            if (et < p.BN) {
                scale_s[b * kMaxBN + et] = dw_next;
                if (p.has_bias) scale_s[(2 + b) * kMaxBN + et] = bias_next;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(scale_bar);
        };
        uint32_t buf = 0, bphase = 0, nboxes = 0, it = 0;
        int unit = blockIdx.x, j = 0;
        fetch_scales(unit < units ? unit_first(unit) : 0);
        publish_scales(0u);
        RowStep rs_next = load_row_step(p, unit < units ? unit_panel(unit) : 0, quarter, lane);
        while (unit < units) {
            // the tile after this one: its scales are fetched now and stay in flight during this tile
            int next_unit = unit, next_j = j + 1;
            if (next_j == unit_count(unit)) {
                next_unit = unit + static_cast<int>(gridDim.x);
                next_j = 0;
            }
            fetch_scales(next_unit < units ? unit_first(next_unit) + next_j : 0);
            const int m_tile = unit_panel(unit);
            const int n_tile = unit_first(unit) + j;
            const long long m_row0 = static_cast<long long>(m_tile) * kBM + quarter * 32;
            const float dxr = rs_next.dx;
            const int zr = rs_next.z;
            if (next_unit != unit && next_unit < units) rs_next = load_row_step(p, unit_panel(next_unit), quarter, lane);
            bool got = mbar_wait(scale_bar, it & 1u, abort_flag, p.status);
            got = got && mbar_wait(tfull_bar(buf), bphase, abort_flag, p.status);
            got = __all_sync(0xffffffffu, got);
            if (!got) break;
            tc_fence_after_sync();
            const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * kMaxBN;
            const float *dw_s = scale_s + (it & 1u) * kMaxBN;
            const float *bias_s = p.has_bias ? scale_s + (2u + (it & 1u)) * kMaxBN : nullptr;
            nboxes = epilogue_tile_stream<kDebugAcc>(p, &tmY, tmem_row, m_row0, n_tile * p.BN, dxr, staging, dw_s, bias_s,
                                                     nboxes, lane, col_half * kEpiStepCols, 2 * kEpiStepCols, zr, two_boxes);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            buf ^= 1u;
            if (buf == 0u) bphase ^= 1u;
            publish_scales((it + 1u) & 1u);
            unit = next_unit;
            j = next_j;
            ++it;
        }
        if (lane == 0) bulk_wait_group<0>();         // all of this thread's stores have completed
    }

    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// --- CTA-pair variant --------------------------------------------------------------------------
//
// Same computation with tcgen05 cta_group::2: two CTAs (a cluster of 2 on neighbouring SMs) share one
// 256 x BN output tile.  Each CTA loads its own 128 rows of codes and only HALF of the weight tile
// (BN/2 rows); the leader CTA issues one MMA that reads both CTAs' shared memory and writes 128
// accumulator rows into each CTA's TMEM.  Per CTA and k-block that is 16 KB + 8..16 KB from L2 instead
// of 16 KB + 16..32 KB, which is what the 128 x 256 single-CTA tile is short of: its main loop waits
// on L2, not on the tensor core.  No load is multicast: every CTA fetches only what it stores.
//
// Barrier protocol (all barriers live at the same offsets in both CTAs):
//   full[s]    leader's copy only: one arrive.expect_tx by the leader's producer for the bytes of BOTH
//              CTAs; every TMA load of either CTA credits the leader's barrier
//   empty[s]   both copies, signalled together by the leader's multicast tcgen05.commit
//   tfull[b]   both copies, multicast commit; each CTA's epilogue drains its own TMEM
//   tempty[b]  leader's copy only, count = epilogue warps of both CTAs (remote arrive from the peer)
constexpr int kPairStages = 6;
constexpr int kPairBHalfBytes = (kMaxBN / 2) * kBK;                   // 16 KB
constexpr int kPairStageBytes = kATileBytes + kPairBHalfBytes;         // 32 KB
constexpr int kPairNumBarriers = 2 * kPairStages + 4 + 1;              // + the barrier of the scale copies
__host__ __device__ constexpr int pair_smem_bytes(int has_bias)
{
    return kPairStages * kPairStageBytes + kNumEpiWarps * kStreamStagingPerWarp + (has_bias ? 4 : 2) * kScaleBufBytes +
           kPairNumBarriers * 8 + 16;
}
// layers with a bias need two more scale buffers than fit beside six stages: they take the single-CTA kernel
constexpr int kPairSmemBytes = pair_smem_bytes(0);
static_assert(kPairSmemBytes <= 232448, "CTA-pair GEMM kernel exceeds the shared memory of one CTA");

template <bool kDebugAcc>
__global__ void __launch_bounds__(kGemmThreads, 1)
ptq_gemm_dequant_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmWh,
                             const __grid_constant__ CUtensorMap tmY, const GemmParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    const bool misaligned = (base & 1023u) != 0u;        // same in both CTAs of the pair (same kernel, same layout)
    if (misaligned) {
        if (threadIdx.x == 0) atomicOr(p.status, PTQ_DEV_SMEM_ALIGN);
        return;
    }
    const uint32_t staging_off = kPairStages * kPairStageBytes;
    const uint32_t scale_off = staging_off + kNumEpiWarps * kStreamStagingPerWarp;
    const uint32_t bar_off = scale_off + 2 * kScaleBufBytes;
    const uint32_t staging_base = base + staging_off;
    const uint32_t bar_base = base + bar_off;
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (kPairStages + s); };
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kPairStages + b); };
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kPairStages + 2 + b); };
    const uint32_t scale_bar = bar_base + 8u * (kPairNumBarriers - 1);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(smem_raw + bar_off + kPairNumBarriers * 8);
    volatile uint32_t *abort_flag = tmem_holder + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();          // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int npairs = gridDim.x >> 1;
    const int half_bn = p.BN >> 1;                       // weight rows per CTA

    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < kPairStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 2 * kNumEpiWarps);
        }
        mbar_init(scale_bar, kNumEpiWarps);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmWh);
        if (p.use_tma_store) prefetch_tensormap(&tmY);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(const_cast<uint32_t *>(tmem_holder)), kTmemCols);
        tmem_relinquish_alloc_permit_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                  // both CTAs' barriers exist before anyone signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    const int pair_m_tiles = (p.m_tiles + 1) >> 1;       // 256-row tiles
    const int total_tiles = pair_m_tiles * p.n_tiles;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            const uint32_t stage_tx = 2u * static_cast<uint32_t>(kATileBytes + half_bn * kBK);
            for (int tile = pair; tile < total_tiles && ok; tile += npairs) {
                const int m_tile = tile / p.n_tiles;
                const int n_tile = tile - m_tile * p.n_tiles;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    const uint32_t a_dst = base + stage * kPairStageBytes;
                    if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), stage_tx);
                    tma_load_2d_pair(a_dst, &tmA, kb * kBK, m_tile * (2 * kBM) + static_cast<int>(rank) * kBM,
                                     full_bar(stage));
                    tma_load_2d_pair(a_dst + kATileBytes, &tmWh, kb * kBK,
                                     n_tile * p.BN + static_cast<int>(rank) * half_bn, full_bar(stage));
                    ++issued;
                    if (++stage == kPairStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
            if (!ok && rank == 0) {
                // Error path only: let the loads already issued land (bounded).
                for (uint32_t s = 0; s < kPairStages; ++s) {
                    const uint32_t uses = (issued + kPairStages - 1u - s) / kPairStages;
                    if (uses == 0u) continue;
                    for (int i = 0; i < 200000 && !mbar_try_wait(full_bar(s), (uses - 1u) & 1u); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = make_idesc_s8(2 * kBM, p.BN);
            uint32_t stage = 0, phase = 0, buf = 0, bphase = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += npairs) {
                if (!mbar_wait(tempty_bar(buf), bphase ^ 1u, abort_flag, p.status)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * kMaxBN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t a_addr = base + stage * kPairStageBytes;
                    const uint64_t a_desc = make_smem_desc_sw128(a_addr);
                    const uint64_t b_desc = make_smem_desc_sw128(a_addr + kATileBytes);
                    const int nmma = (kb == p.k_blocks - 1) ? p.last_mmas : (kBK / 32);
                    mma_i8_ss_pair_kblock(d_tmem, a_desc, b_desc, idesc, kb != 0 ? 1u : 0u, nmma);
                    mma_commit_pair(empty_bar(stage));
                    if (++stage == kPairStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                mma_commit_pair(tfull_bar(buf));
                buf ^= 1u;
                if (buf == 0u) bphase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (both CTAs)
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;
        const int et = static_cast<int>(threadIdx.x) - 64;
        const uint32_t staging = staging_base + static_cast<uint32_t>(warp - 2) * kStreamStagingPerWarp;
        float *scale_s = reinterpret_cast<float *>(smem_raw + scale_off);   // [2][BN] weight steps, per CTA
        float dw_next = 0.0f;
        auto fetch_scales = [&](int tile) {
            if (tile < total_tiles && et < p.BN) dw_next = __ldg(p.dw + (tile % p.n_tiles) * p.BN + et);
        };
        auto publish_scales = [&](uint32_t b) {
            if (et < p.BN) scale_s[b * kMaxBN + et] = dw_next;
            __syncwarp();
            if (lane == 0) mbar_arrive(scale_bar);
        };
        uint32_t buf = 0, bphase = 0, nboxes = 0, it = 0;
        if (p.use_tma_store) {
            fetch_scales(pair);
            publish_scales(0u);
        }
        for (int tile = pair; tile < total_tiles; tile += npairs, ++it) {
            if (p.use_tma_store) fetch_scales(tile + npairs);
            const int m_tile = tile / p.n_tiles;
            const int n_tile = tile - m_tile * p.n_tiles;
            const long long m_row0 =
                static_cast<long long>(m_tile) * (2 * kBM) + static_cast<long long>(rank) * kBM + quarter * 32;
            const long long m = m_row0 + lane;
            const float dxr = (m < p.M) ? __ldg(p.dx + static_cast<int>(m % p.T)) : 0.0f;
            bool got = true;
            if (p.use_tma_store) got = mbar_wait(scale_bar, it & 1u, abort_flag, p.status);
            got = got && mbar_wait(tfull_bar(buf), bphase, abort_flag, p.status);
            got = __all_sync(0xffffffffu, got);
            if (!got) break;
            tc_fence_after_sync();
            const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * kMaxBN;
            if (p.use_tma_store)
                nboxes = epilogue_tile_stream<kDebugAcc>(p, &tmY, tmem_row, m_row0, n_tile * p.BN, dxr, staging,
                                                         scale_s + (it & 1u) * kMaxBN, nullptr, nboxes, lane,
                                                         col_half * kEpiStepCols, 2 * kEpiStepCols, 0, false);
            else
                nboxes = epilogue_tile<kDebugAcc, false, kStreamBox64>(p, &tmY, tmem_row, m_row0, n_tile * p.BN, dxr, staging,
                                                                       nboxes, lane, col_half);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(tempty_bar(buf), 0u);     // the leader's MMA thread waits on it
            buf ^= 1u;
            if (buf == 0u) bphase ^= 1u;
            if (p.use_tma_store) publish_scales((it + 1u) & 1u);
        }
        if (lane == 0) bulk_wait_group<0>();
    }

    __syncthreads();
    cluster_sync_all();          // the peer may still signal this CTA's barriers or be read by the leader's MMAs
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

}  // namespace ptq
