// F1 / A-stationary kernel: the whole path Q1 -> G1 -> E1 (Sec. 5.1; Appendix B.1 parts 1-4) in one
// launch, with no int8 round trip through HBM.  The paper has no such variant; results are the same
// bits as the three-step path.
//
// A CTA owns one 128-row panel of activations at a time and keeps its int8 codes in shared memory
// for ALL output tiles of that panel: the codes are produced once per row (not once per output
// tile), and per output tile only the weight tile is streamed in (from L2).  Four quantizer warps
// load fp16 x (16-byte loads), quantize it in registers and write the codes straight into the
// 128-byte-swizzled K-major layout the MMA reads (fence.proxy.async + mbarrier arrive).
//
// Warps: 0 = TMA producer (weights), 1 = TMEM owner + MMA issuer,
// 2..9 = epilogue (shared with the plain GEMM kernel), 10..13 = quantizers.
// Barriers: pfull/pempty per panel k-block (filled once per panel, freed by the commit after the last
// output tile has read it), wfull/wempty per weight stage, tfull/tempty per TMEM accumulator.
// While the last output tile of panel i still runs, the k-blocks it has finished with are already
// being refilled for panel i+1.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "ptq_gemm.cuh"
#include "ptq_quantize.cuh"
#include "ptx_sm100.cuh"

namespace ptq {

constexpr int kFusedMaxKBlocks = 12;                      // panel of at most 12 x 16 KB = 192 KB (K <= 1536)
constexpr int kFusedMaxWStages = 4;
constexpr int kFusedQuantWarps = 4;
constexpr int kFusedThreadsQuant = 32 * (2 + kNumEpiWarps + kFusedQuantWarps);   // 448
constexpr int kFusedNumBarriers = 2 * kFusedMaxKBlocks + 2 * kFusedMaxWStages + 4;
constexpr int kFusedSmemLimit = 232448;                   // 227 KB opt-in maximum per CTA

struct FusedParams {
    GemmParams g;            // BN / n_tiles here are the fused kernel's own tiling
    const __half *x;         // [M,K] fp16
    const float *s;          // [K]
    const float *rs;         // [K] RN(1/s)
    const float2 *dx2;       // [T] {dx, RN(1/dx)}
    int w_stages;            // weight stages in shared memory
    int w_stage_bytes;       // BN * 128
    int has_staging;         // epilogue staging buffers present (TMA stores possible)
};

__host__ __device__ inline int fused_smem_bytes(int k_blocks, int w_stages, int w_stage_bytes, int has_staging)
{
    return 1024 + k_blocks * kATileBytes + w_stages * w_stage_bytes +
           (has_staging ? kNumEpiWarps * kStagingBytesPerWarp : 0) + kFusedNumBarriers * 8 + 16;
}

template <bool kFast, bool kDebugAcc>
__global__ void __launch_bounds__(kFusedThreadsQuant, 1)
ptq_fused_linear_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmY,
                        const FusedParams fp)
{
    const GemmParams &p = fp.g;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - raw);
    const uint32_t panel_base = base;
    const uint32_t w_base = panel_base + p.k_blocks * kATileBytes;
    const uint32_t staging_base = w_base + fp.w_stages * fp.w_stage_bytes;
    const uint32_t bar_off = p.k_blocks * kATileBytes + fp.w_stages * fp.w_stage_bytes +
                             (fp.has_staging ? kNumEpiWarps * kStagingBytesPerWarp : 0);
    const uint32_t bar_base = base + bar_off;
    auto pfull_bar = [&](uint32_t kb) { return bar_base + 8u * kb; };
    auto pempty_bar = [&](uint32_t kb) { return bar_base + 8u * (kFusedMaxKBlocks + kb); };
    auto wfull_bar = [&](uint32_t s) { return bar_base + 8u * (2 * kFusedMaxKBlocks + s); };
    auto wempty_bar = [&](uint32_t s) { return bar_base + 8u * (2 * kFusedMaxKBlocks + kFusedMaxWStages + s); };
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kFusedMaxKBlocks + 2 * kFusedMaxWStages + b); };
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (2 * kFusedMaxKBlocks + 2 * kFusedMaxWStages + 2 + b); };
    volatile uint32_t *tmem_holder =
        reinterpret_cast<volatile uint32_t *>(base_ptr + bar_off + kFusedNumBarriers * 8);
    volatile uint32_t *abort_flag = tmem_holder + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int kb = 0; kb < p.k_blocks; ++kb) {
            mbar_init(pfull_bar(kb), 32u * kFusedQuantWarps);
            mbar_init(pempty_bar(kb), 1);
        }
        for (int s = 0; s < fp.w_stages; ++s) {
            mbar_init(wfull_bar(s), 1);
            mbar_init(wempty_bar(s), 1);
        }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), kNumEpiWarps);
        }
        *abort_flag = 0u;
        fence_mbar_init();
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

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t w_issued = 0;
            bool ok = true;
            for (int m_tile = blockIdx.x; m_tile < p.m_tiles && ok; m_tile += gridDim.x) {
                for (int n_tile = 0; n_tile < p.n_tiles && ok; ++n_tile) {
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!mbar_wait(wempty_bar(stage), phase ^ 1u, abort_flag, p.status)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(wfull_bar(stage), static_cast<uint32_t>(fp.w_stage_bytes));
                        tma_load_2d(w_base + stage * fp.w_stage_bytes, &tmW, kb * kBK, n_tile * p.BN, wfull_bar(stage));
                        ++w_issued;
                        if (++stage == static_cast<uint32_t>(fp.w_stages)) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                }
            }
            if (!ok) {
                // Error path only: let this thread's own loads land before the CTA gives up its shared memory.
                for (uint32_t s = 0; s < static_cast<uint32_t>(fp.w_stages); ++s) {
                    const uint32_t uses = (w_issued + fp.w_stages - 1u - s) / fp.w_stages;
                    if (uses == 0u) continue;
                    for (int i = 0; i < 200000 && !mbar_try_wait(wfull_bar(s), (uses - 1u) & 1u); ++i) {
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_s8(kBM, p.BN);
            uint32_t stage = 0, phase = 0, buf = 0, bphase = 0, it = 0;
            bool ok = true;
            for (int m_tile = blockIdx.x; m_tile < p.m_tiles && ok; m_tile += gridDim.x, ++it) {
                for (int n_tile = 0; n_tile < p.n_tiles && ok; ++n_tile) {
                    if (!mbar_wait(tempty_bar(buf), bphase ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + buf * kMaxBN;
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (n_tile == 0 && !mbar_wait(pfull_bar(kb), it & 1u, abort_flag, p.status)) {
                            ok = false;
                            break;
                        }
                        if (!mbar_wait(wfull_bar(stage), phase, abort_flag, p.status)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint64_t a_desc = make_smem_desc_sw128(panel_base + kb * kATileBytes);
                        const uint64_t b_desc = make_smem_desc_sw128(w_base + stage * fp.w_stage_bytes);
                        const int nmma = (kb == p.k_blocks - 1) ? p.last_mmas : (kBK / 32);
                        mma_i8_ss_kblock(d_tmem, a_desc, b_desc, idesc, kb != 0 ? 1u : 0u, nmma);
                        mma_commit(wempty_bar(stage));
                        if (n_tile == p.n_tiles - 1) mma_commit(pempty_bar(kb));   // last reader of this panel block
                        if (++stage == static_cast<uint32_t>(fp.w_stages)) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    mma_commit(tfull_bar(buf));
                    buf ^= 1u;
                    if (buf == 0u) bphase ^= 1u;
                }
            }
        }
    } else if (warp < 2 + kNumEpiWarps) {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;
        const uint32_t staging = staging_base + static_cast<uint32_t>(warp - 2) * kStagingBytesPerWarp;
        uint32_t buf = 0, bphase = 0, nboxes = 0;
        bool ok = true;
        for (int m_tile = blockIdx.x; m_tile < p.m_tiles && ok; m_tile += gridDim.x) {
            const long long m_row0 = static_cast<long long>(m_tile) * kBM + quarter * 32;
            const long long m = m_row0 + lane;
            const float dxr = (m < p.M) ? __ldg(p.dx + static_cast<int>(m % p.T)) : 0.0f;
            for (int n_tile = 0; n_tile < p.n_tiles; ++n_tile) {
                bool got = mbar_wait(tfull_bar(buf), bphase, abort_flag, p.status);
                got = __all_sync(0xffffffffu, got);
                if (!got) {
                    ok = false;
                    break;
                }
                tc_fence_after_sync();
                const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * kMaxBN;
                nboxes = epilogue_tile<kDebugAcc>(p, &tmY, tmem_row, m_row0, n_tile * p.BN, dxr, staging, nboxes, lane,
                                                  col_half);
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(buf));
                buf ^= 1u;
                if (buf == 0u) bphase ^= 1u;
            }
        }
        if (lane == 0) bulk_wait_group<0>();
    } else {
        // ------------------------------------------------------------------ quantizer warps
        // Thread (r8, c16) handles rows j*16 + r8 (j = 0..7) and the 16 channels c16*16.. of each k-block.
        const int qt = threadIdx.x - 32 * (2 + kNumEpiWarps);
        const int r8 = qt >> 3, c16 = qt & 7;
        uint32_t it = 0;
        bool ok = true;
        for (int m_tile = blockIdx.x; m_tile < p.m_tiles && ok; m_tile += gridDim.x, ++it) {
            const long long m0 = static_cast<long long>(m_tile) * kBM + r8;
            float2 dj[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const long long m = m0 + 16 * j;
                dj[j] = (m < p.M) ? __ldg(fp.dx2 + static_cast<int>(m % p.T)) : make_float2(1.0f, 1.0f);
            }
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int kcol = kb * kBK + c16 * 16;
                const bool col_ok = kcol < p.K;               // K % 16 == 0: all 16 channels or none
                uint4 u[8][2];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const long long m = m0 + 16 * j;
                    u[j][0] = u[j][1] = make_uint4(0, 0, 0, 0);
                    if (col_ok && m < p.M) {
                        const uint4 *src = reinterpret_cast<const uint4 *>(fp.x + m * p.K + kcol);
                        u[j][0] = __ldcs(src);
                        u[j][1] = __ldcs(src + 1);
                    }
                }
                float rs16[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 r = col_ok ? __ldg(reinterpret_cast<const float4 *>(fp.rs + kcol) + i)
                                            : make_float4(1.0f, 1.0f, 1.0f, 1.0f);
                    rs16[4 * i] = r.x; rs16[4 * i + 1] = r.y; rs16[4 * i + 2] = r.z; rs16[4 * i + 3] = r.w;
                }
                if (!mbar_wait(pempty_bar(kb), (it & 1u) ^ 1u, abort_flag, p.status)) {
                    ok = false;
                    break;
                }
                const uint32_t blk = panel_base + kb * kATileBytes;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int row = 16 * j + r8;
                    const long long m = m0 + 16 * j;
                    uint4 out = make_uint4(0, 0, 0, 0);      // rows beyond M and channels beyond K hold zero codes
                    if (col_ok && m < p.M) {
                        float c8[8] = {};
                        if (kFast) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) c8[i] = __fmul_rn(rs16[i], dj[j].y);
                        }
                        const uint2 o0 = quantize8<kFast, false>(u[j][0], c8, fp.s + kcol, fp.rs + kcol, dj[j].x, dj[j].y, 0);
                        if (kFast) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) c8[i] = __fmul_rn(rs16[8 + i], dj[j].y);
                        }
                        const uint2 o1 = quantize8<kFast, false>(u[j][1], c8, fp.s + kcol + 8, fp.rs + kcol + 8, dj[j].x, dj[j].y, 0);
                        out = make_uint4(o0.x, o0.y, o1.x, o1.y);
                    }
                    // 128-byte swizzle of the K-major operand layout: 16-byte chunk index XOR (row mod 8)
                    st_shared_v4(blk + static_cast<uint32_t>(row) * 128u + (static_cast<uint32_t>(c16 ^ (row & 7)) << 4),
                                 out);
                }
                fence_proxy_async_smem();      // make the generic-proxy writes visible to the tensor core's reads
                mbar_arrive(pfull_bar(kb));
            }
        }
    }

    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace ptq
