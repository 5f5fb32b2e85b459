// Thin inline-PTX wrappers for the sm_100a features the kernels use:
// mbarrier, TMA (cp.async.bulk.tensor), tcgen05 (alloc / mma / commit / ld) and the
// shared-memory matrix descriptor.  Every wait is bounded: a wait that does not end
// within the time limit records PTQ_DEV_TIMEOUT in the status word and returns false,
// and callers unwind to the common exit so that TMEM is always released.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ptq {

constexpr unsigned PTQ_DEV_OK = 0u;
constexpr unsigned PTQ_DEV_TIMEOUT = 1u;
constexpr unsigned PTQ_DEV_SMEM_ALIGN = 2u;   // dynamic shared memory did not start on a 1024-byte boundary

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// ---------------------------------------------------------------- integer division by launch constants
// Division of a 32-bit number by a launch constant without a division: with magic = ceil(2^64 / d), the
// high 64 bits of magic * n are floor(n / d) for every 32-bit n.  A runtime integer division is a chain of
// some twenty dependent instructions (far more for 64-bit operands); at the top of an epilogue loop or in a
// kernel's prologue, where the warp has nothing else to issue, several of them cost hundreds of cycles.
struct FastDiv {
    unsigned d;
    unsigned long long magic;
};
__host__ __device__ inline FastDiv make_fastdiv(unsigned d)
{
    FastDiv f;
    f.d = d;
    f.magic = d > 1u ? 0xFFFFFFFFFFFFFFFFull / d + 1ull : 0ull;
    return f;
}
__device__ __forceinline__ unsigned fd_div(unsigned n, const FastDiv &f)
{
    return f.d == 1u ? n : static_cast<unsigned>(__umul64hi(f.magic, static_cast<unsigned long long>(n)));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Programmatic dependent launch (sm_90+).  A kernel launched with the programmatic-stream-serialization
// attribute may start while its predecessor in the stream is still running; griddep_wait() blocks the
// calling thread until every prerequisite grid has completed and its memory operations are visible
// (a no-op when the launch carried no such dependency).  griddep_launch_dependents() lets the NEXT
// kernel's CTAs be scheduled as soon as resources free up instead of at this grid's very end.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Time limit of one bounded wait.  Far above any legitimate wait in these kernels (a whole
// launch lasts well under 10 ms) and short enough that an error shows up in seconds.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// Wait for the phase with the given parity.  `abort_flag` is a CTA-wide shared word: once any
// thread has given up, every other wait in the CTA returns false at its next check.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          unsigned *status, unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                *abort_flag = 1u;
                atomicOr(status, PTQ_DEV_TIMEOUT);
                return false;
            }
        }
    }
}

// Self-test of the bounded wait, for the failure-detection tests: one CTA of 64 threads and one mbarrier
// that nothing ever arrives on (no copy, no MMA and no other thread refers to it, so giving up leaves
// nothing in flight).  Thread 0 waits with the short limit `limit_ns` and must give up: it raises the
// CTA's abort flag and sets PTQ_DEV_TIMEOUT in `status`.  Thread 32 waits on the same barrier with the
// ordinary long limit and must leave through the abort flag.  out[0], out[1]: what the two waits returned
// (0 = gave up); out[2]: nanoseconds thread 32 spent waiting.
__global__ void __launch_bounds__(64) ptq_wait_selftest_kernel(unsigned *status, unsigned long long limit_ns,
                                                               unsigned *out)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t abort_word;
    const uint32_t bar_addr = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(bar_addr, 1);
        abort_word = 0u;
        fence_mbar_init();
    }
    __syncthreads();
    volatile uint32_t *abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        out[0] = mbar_wait(bar_addr, 0u, abort_flag, status, limit_ns) ? 1u : 0u;
    } else if (threadIdx.x == 32) {
        const unsigned long long t0 = global_timer_ns();
        out[1] = mbar_wait(bar_addr, 0u, abort_flag, status) ? 1u : 0u;
        out[2] = static_cast<unsigned>(global_timer_ns() - t0);
    }
    __syncthreads();
}

// ---------------------------------------------------------------- proxies / fences
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *m)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}

// 2-D tiled load global -> shared, completion counted in bytes on `bar`.
// c0 is the innermost (contiguous) coordinate; c0 * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap *m, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// 2-D tiled store shared -> global (bulk async group of the issuing thread); coordinates >= 0.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *m, int c0, int c1, uint32_t smem_src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(c0), "r"(c1), "r"(smem_src)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit_group()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <int N>
__device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

template <int N>
__device__ __forceinline__ void bulk_wait_group()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// ---------------------------------------------------------------- tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
                 : "memory");
}

__device__ __forceinline__ void tmem_relinquish_alloc_permit()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

__device__ __forceinline__ void tc_fence_before_sync()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_after_sync()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]; s8 x s8 -> s32, one CTA.
__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The four MMAs of one full k-block (128 bytes of K: the start-address field advances by 2 per 32 bytes)
// issued back to back from ONE statement.  The tensor pipe does not queue far ahead of the issuing
// thread: every instruction the thread spends between two MMAs (descriptor arithmetic, predicates, loop
// control) shows up as an idle gap of the pipe, so the descriptors of all four are formed first.
// `accumulate_first` = 0 makes the first MMA overwrite the accumulator; the other three accumulate.
__device__ __forceinline__ void mma_i8_ss_x4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.eq.b32 q, 0, 0;\n\t"
        "add.u64 a1, %1, 2;\n\t"
        "add.u64 a2, %1, 4;\n\t"
        "add.u64 a3, %1, 6;\n\t"
        "add.u64 b1, %2, 2;\n\t"
        "add.u64 b2, %2, 4;\n\t"
        "add.u64 b3, %2, 6;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], a1, b1, %3, q;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], a2, b2, %3, q;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], a3, b3, %3, q;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate_first)
        : "memory");
}

// The MMAs of one k-block: `nmma` (1..4) instructions of 32 bytes of K each.
__device__ __forceinline__ void mma_i8_ss_kblock(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate_first, int nmma)
{
    if (nmma == 4) {
        mma_i8_ss_x4(d_tmem, a_desc, b_desc, idesc, accumulate_first);
    } else {
        for (int j = 0; j < nmma; ++j)
            mma_i8_ss(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, j != 0 ? 1u : accumulate_first);
    }
}

// mbarrier arrives once all tcgen05 operations issued so far by this thread have completed.
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 32 lanes x 32 columns of 32-bit: thread i of the warp gets lane (base lane + i), columns c..c+31.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// ---------------------------------------------------------------- CTA pairs (cluster of 2, cta_group::2)
__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Arrive on the mbarrier at the same shared-memory offset in CTA `target_rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t target_rank)
{
    asm volatile(
        "{\n\t"
        ".reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t"
        "}"
        ::"r"(local_bar), "r"(target_rank)
        : "memory");
}

// In the shared::cluster window of a CTA pair, bit 24 of an address selects the odd CTA; clearing it
// makes a barrier address refer to the even (leader) CTA's copy.
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;

// 2-D tiled load issued by either CTA of a pair into its OWN shared memory; the byte count is
// credited to the LEADER CTA's mbarrier (no multicast: each CTA fetches only its own tile).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t smem_dst, const CUtensorMap *m, int c0, int c1,
                                                 uint32_t local_bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(c0), "r"(c1), "r"(local_bar & kPeerBitMask)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols)
                 : "memory");
}

__device__ __forceinline__ void tmem_relinquish_alloc_permit_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// One MMA over both CTAs of the pair: D (256 x N, 128 rows in each CTA's TMEM) (+)= A (128 rows from each
// CTA's shared memory) * B (N/2 rows from each CTA's shared memory).  Issued by the leader CTA only.
__device__ __forceinline__ void mma_i8_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t"
        "}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The four MMAs of one full k-block over both CTAs of the pair, issued back to back (see mma_i8_ss_x4).
__device__ __forceinline__ void mma_i8_ss_pair_kblock(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                      uint32_t accumulate_first, int nmma)
{
    if (nmma == 4) {
        asm volatile(
            "{\n\t"
            ".reg .pred p, q;\n\t"
            ".reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "setp.eq.b32 q, 0, 0;\n\t"
            "add.u64 a1, %1, 2;\n\t"
            "add.u64 a2, %1, 4;\n\t"
            "add.u64 a3, %1, 6;\n\t"
            "add.u64 b1, %2, 2;\n\t"
            "add.u64 b2, %2, 4;\n\t"
            "add.u64 b3, %2, 6;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], a1, b1, %3, q;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], a2, b2, %3, q;\n\t"
            "tcgen05.mma.cta_group::2.kind::i8 [%0], a3, b3, %3, q;\n\t"
            "}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate_first)
            : "memory");
    } else {
        for (int j = 0; j < nmma; ++j)
            mma_i8_ss_pair(d_tmem, a_desc + 2u * j, b_desc + 2u * j, idesc, j != 0 ? 1u : accumulate_first);
    }
}

// The mbarriers at this offset in both CTAs of the pair (mask 0b11) arrive once all tcgen05 operations
// issued so far by this thread have completed.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar)
{
    const uint16_t mask = 3;
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(mask)
        : "memory");
}

// Instruction descriptor of tcgen05.mma kind::i8, dense, signed 8-bit A and B (both K-major),
// signed 32-bit accumulator, tile M x N.  Field positions: D format [4,6) (2 = s32),
// A format [7,10) and B format [10,13) (1 = signed 8-bit, 0 = unsigned 8-bit), A/B major [15],[16] (0 = K-major),
// N>>3 at [17,23), M>>4 at [24,29).
__host__ __device__ constexpr uint32_t make_idesc_s8(int M, int N, bool a_unsigned = false)
{
    return (2u << 4) | ((a_unsigned ? 0u : 1u) << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) |
           (static_cast<uint32_t>(M >> 4) << 24);
}

// Shared-memory matrix descriptor for a K-major operand tile stored as rows of 128 bytes with
// the 128-byte swizzle (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B): groups of
// 8 rows are 1024 bytes apart (stride byte offset), the leading byte offset is unused for
// swizzled K-major tiles.  Fields: start address>>4 at [0,14), LBO>>4 at [16,30),
// SBO>>4 at [32,46), descriptor version 1 at [46,48), swizzle mode at [61,64) (2 = 128 B).
// The tile base must be 1024-byte aligned; stepping along K inside the 128-byte row is done by
// adding the byte offset (>>4) to the start-address field.
__device__ __forceinline__ uint64_t make_smem_desc_sw128(uint32_t smem_addr)
{
    return static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}

}  // namespace ptq
