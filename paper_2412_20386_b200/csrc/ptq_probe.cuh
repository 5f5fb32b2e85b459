// Measurement aids for the roofline discussion (no counterpart in the paper): what this GPU does, with
// nothing else running, for the three data movements that bound the GEMM + dequantization kernel
// (Sec. 5.1; Appendix B.1 parts 3-4) -- plain 16-byte stores, 2-D TMA stores in the epilogue's pattern,
// and operand stages pulled from L2 by 2-D tiled TMA loads -- and the cost of launching an empty kernel.
// They move bytes only; no arithmetic of the method is in them.  All waits are bounded.
#pragma once

#include <stdint.h>

#include "ptx_sm100.cuh"

namespace ptq {

constexpr int kProbeStore16 = 0, kProbeTmaStore = 1, kProbeOperandPull = 2, kProbeLaunch = 3, kProbeLaunchPdl = 4;
constexpr int kProbeBoxBytes = 32 * 64 * 2;               // one 32-row x 64-column fp16 box, as the epilogue stores
constexpr int kProbeStageBytes = (128 + 256) * 128;       // codes tile + weight tile of one k-block

// Every CTA writes its own contiguous 16 KB pieces with 16-byte stores.
__global__ void __launch_bounds__(256) ptq_probe_store16_kernel(uint4 *dst, unsigned long long n16)
{
    constexpr unsigned kPerCta = 1024;                     // 16-byte words per CTA and pass
    const uint4 v = make_uint4(blockIdx.x, threadIdx.x, 3u, 4u);
    for (unsigned long long base = static_cast<unsigned long long>(blockIdx.x) * kPerCta; base < n16;
         base += static_cast<unsigned long long>(gridDim.x) * kPerCta)
        for (unsigned i = threadIdx.x; i < kPerCta && base + i < n16; i += blockDim.x) dst[base + i] = v;
}

// y [M, N] fp16 written tile by tile (128 x 256, the N tiles of a row panel adjacent) by one CTA per SM: eight
// warps, warp w stores the boxes of lane quarter w % 4 and column half w / 4, one box in flight per warp.
__global__ void __launch_bounds__(256, 1) ptq_probe_tma_store_kernel(const __grid_constant__ CUtensorMap tmY, int m_tiles, int n_tiles)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *box = smem_raw + warp * kProbeBoxBytes;
    for (int i = lane; i < kProbeBoxBytes / 4; i += 32) reinterpret_cast<uint32_t *>(box)[i] = 0x3c003c00u;
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        const int quarter = warp & 3, half = warp >> 2;
        const uint32_t src = smem_u32(box);
        bool first = true;
        for (int tile = blockIdx.x; tile < m_tiles * n_tiles; tile += gridDim.x) {
            const int m_tile = tile / n_tiles, n_tile = tile - m_tile * n_tiles;
            for (int c0 = half * 64; c0 < 256; c0 += 128) {
                if (!first) bulk_wait_group_read<0>();
                first = false;
                tma_store_2d(&tmY, n_tile * 256 + c0, m_tile * 128 + quarter * 32, src);
                bulk_commit_group();
            }
        }
        bulk_wait_group<0>();
    }
}

// The operand stages of the same tiling (codes tile 128 x 128 B, weight tile 256 x 128 B per k-block, 128-byte
// swizzle, four stages) pulled from memory by one thread per CTA and released at once by another: no MMA, no epilogue.
__global__ void __launch_bounds__(64, 1) ptq_probe_operand_pull_kernel(const __grid_constant__ CUtensorMap tmA,
                                                                      const __grid_constant__ CUtensorMap tmW, int m_tiles,
                                                                      int n_tiles, int k_blocks, unsigned *status)
{
    constexpr uint32_t kStagesP = 4;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    const uint32_t bar_base = base + kStagesP * kProbeStageBytes;
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem_raw + kStagesP * kProbeStageBytes + 2 * kStagesP * 8);
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < 2 * kStagesP; ++s) mbar_init(bar_base + 8u * s, 1);
        *abort_flag = 0u;
        fence_mbar_init();
    }
    __syncthreads();
    const int total = m_tiles * n_tiles;
    if (threadIdx.x == 0) {
        uint32_t stage = 0, phase = 0, issued = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
            const int m_tile = tile / n_tiles, n_tile = tile - m_tile * n_tiles;
            for (int kb = 0; kb < k_blocks; ++kb) {
                if (!mbar_wait(bar_base + 8u * (kStagesP + stage), phase ^ 1u, abort_flag, status)) {
                    ok = false;
                    break;
                }
                const uint32_t dst = base + stage * kProbeStageBytes;
                mbar_arrive_expect_tx(bar_base + 8u * stage, kProbeStageBytes);
                tma_load_2d(dst, &tmA, kb * 128, m_tile * 128, bar_base + 8u * stage);
                tma_load_2d(dst + 128 * 128, &tmW, kb * 128, n_tile * 256, bar_base + 8u * stage);
                ++issued;
                if (++stage == kStagesP) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
        if (!ok) {
            // let the loads already issued land before the CTA gives up its shared memory (bounded)
            for (uint32_t s = 0; s < kStagesP; ++s) {
                const uint32_t uses = (issued + kStagesP - 1u - s) / kStagesP;
                if (uses == 0u) continue;
                for (int i = 0; i < 200000 && !mbar_try_wait(bar_base + 8u * s, (uses - 1u) & 1u); ++i) {
                }
            }
        }
    } else if (threadIdx.x == 32) {
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
            for (int kb = 0; kb < k_blocks; ++kb) {
                if (!mbar_wait(bar_base + 8u * stage, phase, abort_flag, status)) {
                    ok = false;
                    break;
                }
                mbar_arrive(bar_base + 8u * (kStagesP + stage));
                if (++stage == kStagesP) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    }
}

__global__ void ptq_probe_empty_kernel(int dependent)
{
    if (dependent) {
        griddep_wait();
        griddep_launch_dependents();
    }
}

}  // namespace ptq
