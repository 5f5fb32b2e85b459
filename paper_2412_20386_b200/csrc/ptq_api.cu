// Host side of the C ABI declared in include/ptq_linear.h: argument validation, parameter
// preparation (padding, reciprocals, tensor maps) and kernel launches.  No compute happens here.
#include "../../include/ptq_linear.h"

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "ptq_calibrate.cuh"
#include "ptq_fused.cuh"
#include "ptq_gemm.cuh"
#include "ptq_probe.cuh"
#include "ptq_quantize.cuh"
#include "ptq_quantize_dynamic.cuh"

namespace {

thread_local char g_err[512] = "";
std::atomic<unsigned long long> g_launches{0};

ptq_status_t fail(ptq_status_t st, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}

#define PTQ_CUDA(call)                                                                         \
    do {                                                                                       \
        cudaError_t e_ = (call);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return fail(e_ == cudaErrorMemoryAllocation ? PTQ_ERR_NOMEM : PTQ_ERR_CUDA,        \
                        "%s failed: %s", #call, cudaGetErrorString(e_));                       \
    } while (0)

// cuTensorMapEncodeTiled is reached through the runtime's driver entry point query, so the
// library has no link-time dependency on libcuda and loads on machines without a driver.
typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_tiled()
{
    static encode_tiled_fn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(p);
    });
    return fn;
}

// 2-D row-major tensor [rows, cols] with `pitch_bytes` between rows; box [box_rows, box_cols];
// the swizzle mode follows the box's row bytes (128 or 64, which box_cols * elem_bytes must equal);
// out-of-range elements read as zero and are skipped on stores.
ptq_status_t make_map_2d(CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *ptr,
                         unsigned long long cols, unsigned long long rows, unsigned long long pitch_bytes,
                         unsigned box_cols, unsigned box_rows)
{
    encode_tiled_fn enc = get_encode_tiled();
    if (!enc) return fail(PTQ_ERR_CUDA, "cuTensorMapEncodeTiled entry point not available");
    const unsigned row_bytes = box_cols * elem_bytes;
    if ((row_bytes != 128 && row_bytes != 64) || box_rows == 0 || box_rows > 256)
        return fail(PTQ_ERR_SHAPE, "internal: bad TMA box %u x %u", box_rows, box_cols);
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        return fail(PTQ_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d (cols %llu rows %llu pitch %llu)",
                    static_cast<int>(r), cols, rows, pitch_bytes);
    return PTQ_OK;
}

#ifndef PTQ_GEMM_SHORT_K_BLOCKS
#define PTQ_GEMM_SHORT_K_BLOCKS 3
#endif

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
inline int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb)
{
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + nb && b0 < a0 + na;
}

}  // namespace

// Tensor maps of the caller's buffers, remembered per handle: encoding one costs the host about as much as a
// kernel launch, and a layer is normally called again and again with the same few buffers and batch sizes.
// Keyed by everything the encoding depends on besides the layer (pointer, rows, box width); four entries
// per kind, replaced in turn.  The lock is per handle and held for a lookup or an insertion only.
struct MapCache {
    struct Entry {
        const void *ptr = nullptr;
        long long rows = -1;
        unsigned box_cols = 0;
        CUtensorMap map;
    };
    Entry e[4];
    unsigned next = 0;
    std::mutex mu;
};

struct ptq_linear {
    int K = 0, N = 0, T = 0;
    int Kpad = 0;              // pitch of the codes workspace and of the padded weight: K rounded up to 16
    int BN = 0, n_tiles = 0;   // GEMM tiling along N
    int k_blocks = 0, last_mmas = 0;
    bool fast_div = false;     // all scales inside the range where the reciprocal route is exact
    int device = -1;
    int num_sms = 0;
    int8_t *d_w = nullptr;     // [n_tiles*BN, Kpad], zero padded
    float *d_dw = nullptr, *d_bias = nullptr;            // [n_tiles*BN rounded up to 64, +64], zero padded
    float *d_s = nullptr, *d_rs = nullptr;               // [round_up(K,16)]
    float *d_dx = nullptr, *d_rdx = nullptr;             // [T]
    float2 *d_dx2 = nullptr;                             // [T] {dx, 1/dx}
    int *d_zp = nullptr;                                 // [T] zero offsets (asymmetric layers only)
    int *d_wsum = nullptr;                               // row sums of Wq, padded like d_dw (asymmetric only)
    bool asym = false;
    bool has_bias = false;     // false: d_bias is all zeros
    int act_bits = 8;          // 8: codes in [-128,127] (or [0,255]); 4: codes in [-8,7], one per byte
    unsigned *d_status = nullptr;
    CUtensorMap tmW;
    CUtensorMap tmWh;          // same weights, box of BN/2 rows: the half tile one CTA of a pair loads
    int max_pairs = 0;         // resident 2-CTA clusters of the pair kernel on this device (0: not available)
    // tiling of the fused (A-stationary) kernel
    bool as_ok = false;
    int as_BN = 0, as_n_tiles = 0, as_w_stages = 0, as_w_stage_bytes = 0, as_staging = 0, as_smem = 0;
    CUtensorMap tmWas;
    mutable MapCache codes_maps, y_maps;   // tensor maps of caller buffers seen so far
};

namespace {

ptq_status_t upload(void **dst, const void *src, size_t bytes, size_t alloc_bytes)
{
    PTQ_CUDA(cudaMalloc(dst, alloc_bytes));
    PTQ_CUDA(cudaMemset(*dst, 0, alloc_bytes));
    if (bytes) PTQ_CUDA(cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice));
    return PTQ_OK;
}

ptq_status_t check_device(const ptq_linear *h)
{
    int dev = -1;
    PTQ_CUDA(cudaGetDevice(&dev));
    if (dev != h->device)
        return fail(PTQ_ERR_CUDA, "handle belongs to device %d but device %d is current", h->device, dev);
    return PTQ_OK;
}

// make_map_2d through a handle's cache.
ptq_status_t cached_map_2d(MapCache &cache, CUtensorMap *map, CUtensorMapDataType dt, int elem_bytes, const void *ptr,
                           unsigned long long cols, unsigned long long rows, unsigned long long pitch_bytes,
                           unsigned box_cols, unsigned box_rows)
{
    std::lock_guard<std::mutex> lock(cache.mu);
    for (const MapCache::Entry &e : cache.e)
        if (e.ptr == ptr && e.rows == static_cast<long long>(rows) && e.box_cols == box_cols) {
            *map = e.map;
            return PTQ_OK;
        }
    const ptq_status_t st = make_map_2d(map, dt, elem_bytes, ptr, cols, rows, pitch_bytes, box_cols, box_rows);
    if (st != PTQ_OK) return st;
    MapCache::Entry &slot = cache.e[cache.next];
    cache.next = (cache.next + 1u) % 4u;
    slot.ptr = ptr;
    slot.rows = static_cast<long long>(rows);
    slot.box_cols = box_cols;
    slot.map = *map;
    return PTQ_OK;
}

// Opt a kernel in to `bytes` of dynamic shared memory, once per kernel and device (the attribute belongs
// to the function on the CURRENT device, which the callers have checked to be `device`).  The kernel is
// a template argument so that every kernel has its own flags.
template <auto kKern>
ptq_status_t ensure_smem(int device, int bytes)
{
    constexpr int kMaxDevices = 64;
    static std::atomic<bool> done[kMaxDevices] = {};
    if (device < 0 || device >= kMaxDevices) return fail(PTQ_ERR_CUDA, "device index %d out of range", device);
    // lock-free once the attribute is set; two threads racing on the first call both set the same value
    if (!done[device].load(std::memory_order_acquire)) {
        PTQ_CUDA(cudaFuncSetAttribute(kKern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
        done[device].store(true, std::memory_order_release);
    }
    return PTQ_OK;
}

// How many 2-CTA clusters of the pair kernel can be resident at once (0 if cluster launch is unavailable).
int query_max_pairs(int device)
{
    constexpr int kMaxDevices = 64;
    static int cache[kMaxDevices];
    static bool known[kMaxDevices] = {};
    static std::mutex mu;
    if (device < 0 || device >= kMaxDevices) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (known[device]) return cache[device];
    known[device] = true;                      // per device: attributes and occupancy belong to the current device
    int &cached = cache[device];
    cached = 0;
    if (cudaFuncSetAttribute(ptq::ptq_gemm_dequant_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ptq::kPairSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(ptq::ptq_gemm_dequant_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ptq::kPairSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return cached;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(ptq::kGemmThreads, 1, 1);
    cfg.dynamicSmemBytes = ptq::kPairSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, ptq::ptq_gemm_dequant_pair_kernel<false>, &cfg) == cudaSuccess && n > 0)
        cached = n;
    else
        (void)cudaGetLastError();
    return cached;
}

// Launch with the programmatic-stream-serialization attribute: the kernel may begin (its set-up, up to
// its griddep_wait()) while the previous kernel in the stream drains.  Every kernel launched this way
// calls griddep_wait() before touching anything another kernel may have written.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(static_cast<unsigned>(block), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// Q1 launch: codes to `q` with `q_pitch` bytes between rows.
ptq_status_t launch_quantize(const ptq_linear *h, const void *x, long long M, void *q, int q_pitch,
                             cudaStream_t stream)
{
    ptq::QuantParams p;
    p.x = static_cast<const __half *>(x);
    p.q = static_cast<int8_t *>(q);
    p.s = h->d_s;
    p.rs = h->d_rs;
    p.dx = h->d_dx;
    p.rdx = h->d_rdx;
    p.dx2 = h->d_dx2;
    p.zp = h->d_zp;
    p.M = M;
    p.K = h->K;
    p.T = h->T;
    p.q_pitch = q_pitch;
    const long long B = M / h->T;
    // Vector kernel: thread count = S * (chunks per image), S images apart between a thread's chunks.
    // S is the multiple of `mult` (which makes the thread count a multiple of 256) that brings the grid
    // closest to one resident wave without exceeding it; shapes for which even the smallest S
    // overshoots the wave by far go to the scalar kernel.
    bool vec = (h->K % 8 == 0) && (reinterpret_cast<uintptr_t>(x) % 16 == 0) &&
               (reinterpret_cast<uintptr_t>(q) % 8 == 0) && (q_pitch % 8 == 0);
    long long cpi = 0, S = 0;
    if (vec) {
        cpi = static_cast<long long>(h->T) * (h->K / 8);
        const long long wave = static_cast<long long>(h->num_sms) * ptq::kQuantCtasPerSm * 256;
        const long long mult = 256 / gcd_int(static_cast<int>(cpi % 256 == 0 ? 256 : cpi % 256), 256);
        S = wave / cpi / mult * mult;
        if (S < mult) S = mult;
        const long long bcap = (B + mult - 1) / mult * mult;      // more than B images apart is idle threads only
        if (S > bcap) S = bcap;
        if (S * cpi > 4 * wave) vec = false;
    }
    p.B = static_cast<int>(B);
    p.imgs_per_iter = static_cast<int>(S);
    p.fd_cpi = ptq::make_fastdiv(static_cast<unsigned>(vec ? cpi : 1));
    p.fd_cpr = ptq::make_fastdiv(static_cast<unsigned>(vec ? h->K / 8 : 1));
    if (vec) {
        const int grid = static_cast<int>(S * cpi / 256);
        if (h->act_bits == 4) {
            if (h->fast_div)
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_vec8_kernel<true, ptq::kCodeS4>, grid, 256, 0, stream, p));
            else
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_vec8_kernel<false, ptq::kCodeS4>, grid, 256, 0, stream, p));
        } else if (h->asym) {
            if (h->fast_div)
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_vec8_kernel<true, ptq::kCodeU8>, grid, 256, 0, stream, p));
            else
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_vec8_kernel<false, ptq::kCodeU8>, grid, 256, 0, stream, p));
        } else if (h->fast_div)
            PTQ_CUDA(launch_pdl(ptq::ptq_quantize_vec8_kernel<true>, grid, 256, 0, stream, p));
        else
            PTQ_CUDA(launch_pdl(ptq::ptq_quantize_vec8_kernel<false>, grid, 256, 0, stream, p));
    } else {
        long long want = (M * h->K + 255) / 256;
        const long long cap = static_cast<long long>(h->num_sms) * 8;
        if (want > cap) want = cap;
        if (want < 1) want = 1;
        const int g = static_cast<int>(want);
        if (h->act_bits == 4) {
            if (h->fast_div)
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_scalar_kernel<true, ptq::kCodeS4>, g, 256, 0, stream, p));
            else
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_scalar_kernel<false, ptq::kCodeS4>, g, 256, 0, stream, p));
        } else if (h->asym) {
            if (h->fast_div)
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_scalar_kernel<true, ptq::kCodeU8>, g, 256, 0, stream, p));
            else
                PTQ_CUDA(launch_pdl(ptq::ptq_quantize_scalar_kernel<false, ptq::kCodeU8>, g, 256, 0, stream, p));
        } else if (h->fast_div)
            PTQ_CUDA(launch_pdl(ptq::ptq_quantize_scalar_kernel<true>, g, 256, 0, stream, p));
        else
            PTQ_CUDA(launch_pdl(ptq::ptq_quantize_scalar_kernel<false>, g, 256, 0, stream, p));
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    PTQ_CUDA(cudaGetLastError());
    return PTQ_OK;
}

// Dynamic comparator: codes to `q` and the per-row steps to `dx_row`.
ptq_status_t launch_quantize_dynamic(const ptq_linear *h, const void *x, long long M, void *q, int q_pitch,
                                     float *dx_row, cudaStream_t stream)
{
    ptq::DynQuantParams p;
    p.x = static_cast<const __half *>(x);
    p.q = static_cast<int8_t *>(q);
    p.dx_row = dx_row;
    p.s = h->d_s;
    p.rs = h->d_rs;
    p.M = M;
    p.K = h->K;
    p.q_pitch = q_pitch;
    const bool vec = (h->K % 8 == 0) && (reinterpret_cast<uintptr_t>(x) % 16 == 0) &&
                     (reinterpret_cast<uintptr_t>(q) % 8 == 0) && (q_pitch % 8 == 0);
    const long long rows_per_cta = vec ? 8 * ptq::kDynRowsPerWarp : 8;
    long long want = (M + rows_per_cta - 1) / rows_per_cta;
    const long long cap = static_cast<long long>(h->num_sms) * 8;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    if (!vec)
        PTQ_CUDA(launch_pdl(ptq::ptq_quantize_dynamic_scalar_kernel, static_cast<int>(want), 256, 0, stream, p));
    else if (h->fast_div)
        PTQ_CUDA(launch_pdl(ptq::ptq_quantize_dynamic_vec8_kernel<true>, static_cast<int>(want), 256, 0, stream, p));
    else
        PTQ_CUDA(launch_pdl(ptq::ptq_quantize_dynamic_vec8_kernel<false>, static_cast<int>(want), 256, 0, stream, p));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    PTQ_CUDA(cudaGetLastError());
    return PTQ_OK;
}

#ifndef PTQ_GEMM_PANEL
#define PTQ_GEMM_PANEL 1
#endif
#ifndef PTQ_GEMM_TEAMS
#define PTQ_GEMM_TEAMS 1
#endif
#ifndef PTQ_GEMM_TEAM_MIN_ROUNDS
#define PTQ_GEMM_TEAM_MIN_ROUNDS 3
#endif

// Whether this launch takes the panel kernel (the codes of a row panel resident in shared memory for a
// group of N tiles), and with which tiling: fills p.group, p.groups, p.b_stages, p.b_stage_bytes.
// It pays on large compute-bound layers only (measured: 2-3 % of the Vim-B step, nothing or a loss on
// layers with K <= 384 or few tiles), so it is taken when the layer has at least four k-blocks and
// eight tiles per SM, and only with a group size G whose work units divide over the CTAs as evenly as
// single tiles do: rounds(G) * G <= rounds(1).  Among those the largest G wins (fewest panel loads).
bool plan_panel(const ptq_linear *h, ptq::GemmParams &p, bool tma_store)
{
    p.group = p.groups = p.b_stages = p.b_stage_bytes = 0;
    const long long tiles = static_cast<long long>(p.m_tiles) * p.n_tiles;
    if (!PTQ_GEMM_PANEL || !tma_store || p.n_tiles < 2 || p.k_blocks < 4 || p.k_blocks > ptq::kPanelMaxKBlocks ||
        tiles < 8ll * h->num_sms)
        return false;
    const int stage_bytes = p.BN * ptq::kBK;
    const int fixed = ptq::panel_smem_bytes(p.k_blocks, 0, 0, p.boxes, p.has_bias);
    int stages = (ptq::kPanelSmemLimit - fixed) / stage_bytes;
    if (stages < 3) return false;
    if (stages > ptq::kPanelMaxBStages) stages = ptq::kPanelMaxBStages;
    const long long rounds1 = (tiles + h->num_sms - 1) / h->num_sms;
    int best_g = 1;
    for (int g = 2; g <= p.n_tiles; ++g) {
        const long long units = static_cast<long long>((p.n_tiles + g - 1) / g) * p.m_tiles;
        const long long grid = units < h->num_sms ? units : h->num_sms;
        const long long rounds = (units + grid - 1) / grid;
        if (rounds * g <= rounds1) best_g = g;
    }
    if (best_g < 2) return false;
    p.group = best_g;
    p.groups = (p.n_tiles + best_g - 1) / best_g;
    p.fd_groups = ptq::make_fastdiv(static_cast<unsigned>(p.groups));
    p.b_stages = stages;
    p.b_stage_bytes = stage_bytes;
    return true;
}

// Whether the streaming kernel runs its epilogue in two teams: short main loop (K <= 384) and several tiles per CTA.
bool gemm_teams(const ptq_linear *h, const ptq::GemmParams &p, bool tma_store, bool short_k)
{
    const long long tiles = static_cast<long long>(p.m_tiles) * p.n_tiles;
    return PTQ_GEMM_TEAMS && tma_store && short_k && tiles >= static_cast<long long>(PTQ_GEMM_TEAM_MIN_ROUNDS) * h->num_sms;
}

// G1+E1 launch on codes [M, Kpad] at `codes`.
// dx_rows != nullptr: the steps are per ROW (dynamic comparator), i.e. dx = dx_rows and T = M.
ptq_status_t launch_gemm(const ptq_linear *h, const void *codes, long long M, void *y, void *acc_out,
                         cudaStream_t stream, bool want_pair = false, const float *dx_rows = nullptr)
{
    CUtensorMap tmA, tmY;
    ptq_status_t st = cached_map_2d(h->codes_maps, &tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes,
                                    static_cast<unsigned long long>(h->K), static_cast<unsigned long long>(M),
                                    static_cast<unsigned long long>(h->Kpad), ptq::kBK, ptq::kBM);
    if (st != PTQ_OK) return st;
    const bool tma_store = (h->N % 8 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    const int m_tiles_ = static_cast<int>((M + ptq::kBM - 1) / ptq::kBM);
#ifdef PTQ_EXP_FORCE_PAIR
    want_pair = true;
#endif
    const bool use_pair = want_pair && h->max_pairs > 0 && !h->has_bias &&
                          static_cast<long long>((m_tiles_ + 1) / 2) * h->n_tiles >= h->max_pairs;
    if (tma_store) {
        st = cached_map_2d(h->y_maps, &tmY, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, static_cast<unsigned long long>(h->N),
                           static_cast<unsigned long long>(M), static_cast<unsigned long long>(h->N) * 2,
                           ptq::kStreamBoxCols, 32);
        if (st != PTQ_OK) return st;
    } else {
        tmY = h->tmW;   // never dereferenced by the kernel in this mode
    }

    ptq::GemmParams p;
    p.M = M;
    p.N = h->N;
    p.K = h->K;
    p.T = dx_rows ? static_cast<int>(M) : h->T;
    p.BN = h->BN;
    p.n_tiles = h->n_tiles;
    p.m_tiles = static_cast<int>((M + ptq::kBM - 1) / ptq::kBM);
    p.k_blocks = h->k_blocks;
    p.last_mmas = h->last_mmas;
    p.dx = dx_rows ? dx_rows : h->d_dx;
    p.dw = h->d_dw;
    p.bias = h->d_bias;
    p.has_bias = h->has_bias ? 1 : 0;
    // Short main loops (up to three k-blocks per tile, K <= 384) leave the epilogue little time: three stages and two
    // staging boxes per warp; longer ones keep four stages.  Layers with a bias hold two more scale copies.
    const bool short_k = h->k_blocks <= PTQ_GEMM_SHORT_K_BLOCKS;
    p.stages = (short_k || h->has_bias) ? ptq::kStages - 1 : ptq::kStages;
    p.boxes = short_k ? 2 : 1;
    const int gemm_smem = ptq::gemm_smem_bytes(p.stages, p.boxes, p.has_bias);
    p.y = static_cast<__half *>(y);
    p.acc_out = static_cast<int32_t *>(acc_out);
    p.status = h->d_status;
    p.use_tma_store = tma_store ? 1 : 0;
    p.y_vec2 = (h->N % 2 == 0 && reinterpret_cast<uintptr_t>(y) % 4 == 0) ? 1 : 0;
    p.y_vec8 = 0;   // this kernel always has a staging buffer; 16-byte alignment means TMA stores
    p.zp = h->d_zp;
    p.wsum = h->d_wsum;
    p.fd_T = ptq::make_fastdiv(static_cast<unsigned>(p.T));
    p.fd_n_tiles = ptq::make_fastdiv(static_cast<unsigned>(p.n_tiles));
    p.fd_groups = ptq::make_fastdiv(1u);

    if (use_pair) {
        // enough 256-row tiles to occupy every CTA pair: cta_group::2 kernel (half the weight bytes per CTA)
        const int npairs = h->max_pairs;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * npairs, 1, 1);
        cfg.blockDim = dim3(ptq::kGemmThreads, 1, 1);
        cfg.dynamicSmemBytes = ptq::kPairSmemBytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (acc_out)
            PTQ_CUDA(cudaLaunchKernelEx(&cfg, ptq::ptq_gemm_dequant_pair_kernel<true>, tmA, h->tmWh, tmY, p));
        else
            PTQ_CUDA(cudaLaunchKernelEx(&cfg, ptq::ptq_gemm_dequant_pair_kernel<false>, tmA, h->tmWh, tmY, p));
        g_launches.fetch_add(1, std::memory_order_relaxed);
        PTQ_CUDA(cudaGetLastError());
        return PTQ_OK;
    }
    const long long tiles = static_cast<long long>(p.m_tiles) * p.n_tiles;
    // Short main loop (K <= 384) and several tiles per CTA: the epilogue sets the pace and runs in two teams of
    // four warps, one per accumulator; otherwise all eight warps share every tile (shorter latency of a tile).
    const bool teams = gemm_teams(h, p, tma_store, short_k);
    const bool dbg = acc_out != nullptr;
    if (plan_panel(h, p, tma_store)) {
        // several N tiles and 512 <= K <= 768: the codes of a row panel stay in shared memory for `group` tiles
        const int psmem = ptq::panel_smem_bytes(p.k_blocks, p.b_stages, p.b_stage_bytes, p.boxes, p.has_bias);
        const long long units = static_cast<long long>(p.m_tiles) * p.groups;
        const int pgrid = static_cast<int>(units < h->num_sms ? units : h->num_sms);
        ptq_status_t ps = dbg ? ensure_smem<ptq::ptq_gemm_dequant_panel_kernel<true>>(h->device, ptq::kPanelSmemLimit)
                              : ensure_smem<ptq::ptq_gemm_dequant_panel_kernel<false>>(h->device, ptq::kPanelSmemLimit);
        if (ps != PTQ_OK) return ps;
        if (dbg)
            PTQ_CUDA(launch_pdl(ptq::ptq_gemm_dequant_panel_kernel<true>, pgrid, ptq::kGemmThreads, psmem, stream, tmA, h->tmW, tmY, p));
        else
            PTQ_CUDA(launch_pdl(ptq::ptq_gemm_dequant_panel_kernel<false>, pgrid, ptq::kGemmThreads, psmem, stream, tmA, h->tmW, tmY, p));
        g_launches.fetch_add(1, std::memory_order_relaxed);
        PTQ_CUDA(cudaGetLastError());
        return PTQ_OK;
    }
    const int grid = static_cast<int>(tiles < h->num_sms ? tiles : h->num_sms);
    auto go = [&](auto kern) -> ptq_status_t {
        PTQ_CUDA(launch_pdl(kern, grid, ptq::kGemmThreads, gemm_smem, stream, tmA, h->tmW, tmY, p));
        return PTQ_OK;
    };
    ptq_status_t gs;
    if (teams) {
        gs = dbg ? ensure_smem<ptq::ptq_gemm_dequant_kernel<true, true>>(h->device, ptq::kGemmSmemBytes)
                 : ensure_smem<ptq::ptq_gemm_dequant_kernel<false, true>>(h->device, ptq::kGemmSmemBytes);
        if (gs == PTQ_OK) gs = dbg ? go(ptq::ptq_gemm_dequant_kernel<true, true>) : go(ptq::ptq_gemm_dequant_kernel<false, true>);
    } else {
        gs = dbg ? ensure_smem<ptq::ptq_gemm_dequant_kernel<true, false>>(h->device, ptq::kGemmSmemBytes)
                 : ensure_smem<ptq::ptq_gemm_dequant_kernel<false, false>>(h->device, ptq::kGemmSmemBytes);
        if (gs == PTQ_OK) gs = dbg ? go(ptq::ptq_gemm_dequant_kernel<true, false>) : go(ptq::ptq_gemm_dequant_kernel<false, false>);
    }
    if (gs != PTQ_OK) return gs;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    PTQ_CUDA(cudaGetLastError());
    return PTQ_OK;
}

// Tiling of the A-stationary kernel for a layer: the code panel (k_blocks x 16 KB) stays resident, the
// rest of shared memory holds weight stages and, if it fits, the epilogue's staging buffers.
void choose_astat(ptq_linear *h)
{
    h->as_ok = false;
    if (h->k_blocks > ptq::kFusedMaxKBlocks) return;
    const int cand_bn[3] = {h->BN, 128, 64};
    for (int staging = 1; staging >= 0 && !h->as_ok; --staging) {
        for (int c = 0; c < 3 && !h->as_ok; ++c) {
            int bn = cand_bn[c];
            if (c > 0 && bn >= h->BN) continue;
            const int n_tiles = (c == 0) ? h->n_tiles : (h->N + bn - 1) / bn;
            const int stage_bytes = bn * ptq::kBK;
            const int fixed = ptq::fused_smem_bytes(h->k_blocks, 0, 0, staging);
            int stages = (ptq::kFusedSmemLimit - fixed) / stage_bytes;
            if (stages < 2) continue;
            if (stages > ptq::kFusedMaxWStages) stages = ptq::kFusedMaxWStages;
            h->as_ok = true;
            h->as_BN = bn;
            h->as_n_tiles = n_tiles;
            h->as_w_stages = stages;
            h->as_w_stage_bytes = stage_bytes;
            h->as_staging = staging;
            h->as_smem = ptq::fused_smem_bytes(h->k_blocks, stages, stage_bytes, staging);
        }
    }
}

template <auto kKern>
ptq_status_t launch_fused_kernel(const ptq_linear *h, const CUtensorMap &tmY, const ptq::FusedParams &fp, int grid,
                                 cudaStream_t stream)
{
    const ptq_status_t attr_status = ensure_smem<kKern>(h->device, ptq::kFusedSmemLimit);
    if (attr_status != PTQ_OK) return attr_status;
    kKern<<<grid, ptq::kFusedThreadsQuant, h->as_smem, stream>>>(h->tmWas, tmY, fp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    PTQ_CUDA(cudaGetLastError());
    return PTQ_OK;
}

// F1 launch: x fp16 [M,K] -> y (Q1 + G1 + E1 in one kernel, the code panel of a row tile resident in shared memory).
ptq_status_t launch_fused(const ptq_linear *h, const void *x, long long M, void *y, void *acc_out, cudaStream_t stream)
{
    CUtensorMap tmY;
    ptq_status_t st;
    const bool aligned = (h->N % 8 == 0) && (reinterpret_cast<uintptr_t>(y) % 16 == 0);
    const bool tma_store = aligned && h->as_staging;
    if (tma_store) {
        st = cached_map_2d(h->y_maps, &tmY, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, y, static_cast<unsigned long long>(h->N),
                           static_cast<unsigned long long>(M), static_cast<unsigned long long>(h->N) * 2,
                           ptq::kStoreBoxCols, 32);
        if (st != PTQ_OK) return st;
    } else {
        tmY = h->tmWas;   // never dereferenced by the kernel in this mode
    }
    ptq::FusedParams fp;
    ptq::GemmParams &p = fp.g;
    p.M = M;
    p.N = h->N;
    p.K = h->K;
    p.T = h->T;
    p.BN = h->as_BN;
    p.n_tiles = h->as_n_tiles;
    p.m_tiles = static_cast<int>((M + ptq::kBM - 1) / ptq::kBM);
    p.k_blocks = h->k_blocks;
    p.last_mmas = h->last_mmas;
    p.dx = h->d_dx;
    p.dw = h->d_dw;
    p.bias = h->d_bias;
    p.has_bias = h->has_bias ? 1 : 0;
    p.y = static_cast<__half *>(y);
    p.acc_out = static_cast<int32_t *>(acc_out);
    p.status = h->d_status;
    p.use_tma_store = tma_store ? 1 : 0;
    p.y_vec2 = (h->N % 2 == 0 && reinterpret_cast<uintptr_t>(y) % 4 == 0) ? 1 : 0;
    p.y_vec8 = (aligned && !tma_store) ? 1 : 0;
    p.zp = nullptr;
    p.wsum = nullptr;
    fp.x = static_cast<const __half *>(x);
    fp.s = h->d_s;
    fp.rs = h->d_rs;
    fp.dx2 = h->d_dx2;
    fp.w_stages = h->as_w_stages;
    fp.w_stage_bytes = h->as_w_stage_bytes;
    fp.has_staging = h->as_staging;
    const int grid = p.m_tiles < h->num_sms ? p.m_tiles : h->num_sms;
    const bool dbg = acc_out != nullptr;
    if (h->fast_div)
        return dbg ? launch_fused_kernel<ptq::ptq_fused_linear_kernel<true, true>>(h, tmY, fp, grid, stream)
                   : launch_fused_kernel<ptq::ptq_fused_linear_kernel<true, false>>(h, tmY, fp, grid, stream);
    return dbg ? launch_fused_kernel<ptq::ptq_fused_linear_kernel<false, true>>(h, tmY, fp, grid, stream)
               : launch_fused_kernel<ptq::ptq_fused_linear_kernel<false, false>>(h, tmY, fp, grid, stream);
}

bool fused_usable(const ptq_linear *h) { return h->as_ok && h->K % 16 == 0; }

// Scratch for ptq_linear_forward_static: lives in the library image on every device that loads it.
// In host code the symbol below is only a stand-in; the kernels must be given the device address
// that cudaGetSymbolAddress returns, looked up once per device with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[PTQ_STATIC_SCRATCH_BYTES];

ptq_status_t static_scratch_address(int device, void **out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void *addr[kMaxDevices] = {};
    if (device < 0 || device >= kMaxDevices) return fail(PTQ_ERR_CUDA, "device index %d out of range", device);
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[device]) {
        void *p = nullptr;
        PTQ_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));   // the current device is `device` (checked by the caller)
        if (!p) return fail(PTQ_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
        addr[device] = p;
    }
    *out = addr[device];
    return PTQ_OK;
}

ptq_status_t validate_forward(const ptq_linear *h, const void *x, int B, const void *y)
{
    if (!h || !x || !y) return fail(PTQ_ERR_NULL, "handle, x and y must not be NULL");
    if (B < 1) return fail(PTQ_ERR_SHAPE, "B must be >= 1 (got %d)", B);
    const long long M = static_cast<long long>(B) * h->T;
    if (M > 0x7fffff00ll) return fail(PTQ_ERR_SHAPE, "B*T = %lld is too large", M);
    if (reinterpret_cast<uintptr_t>(x) % 2 || reinterpret_cast<uintptr_t>(y) % 2)
        return fail(PTQ_ERR_ALIGN, "x and y must be 2-byte aligned");
    if (ranges_overlap(x, static_cast<size_t>(M) * h->K * 2, y, static_cast<size_t>(M) * h->N * 2))
        return fail(PTQ_ERR_VALUE, "x and y overlap");
    return check_device(h);
}

}  // namespace

extern "C" {

const char *ptq_status_string(ptq_status_t st)
{
    switch (st) {
        case PTQ_OK: return "PTQ_OK";
        case PTQ_ERR_NULL: return "PTQ_ERR_NULL";
        case PTQ_ERR_SHAPE: return "PTQ_ERR_SHAPE";
        case PTQ_ERR_VALUE: return "PTQ_ERR_VALUE";
        case PTQ_ERR_ALIGN: return "PTQ_ERR_ALIGN";
        case PTQ_ERR_ARCH: return "PTQ_ERR_ARCH";
        case PTQ_ERR_CUDA: return "PTQ_ERR_CUDA";
        case PTQ_ERR_NOMEM: return "PTQ_ERR_NOMEM";
        case PTQ_ERR_TIMEOUT: return "PTQ_ERR_TIMEOUT";
    }
    return "PTQ_ERR_UNKNOWN";
}

const char *ptq_last_error(void) { return g_err; }

unsigned long long ptq_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void ptq_linear_destroy(ptq_linear_t *h)
{
    if (!h) return;
    cudaFree(h->d_w);
    cudaFree(h->d_dw);
    cudaFree(h->d_bias);
    cudaFree(h->d_s);
    cudaFree(h->d_rs);
    cudaFree(h->d_dx);
    cudaFree(h->d_rdx);
    cudaFree(h->d_dx2);
    cudaFree(h->d_zp);
    cudaFree(h->d_wsum);
    cudaFree(h->d_status);
    delete h;
}

static ptq_status_t create_impl(ptq_linear_t **out, int K, int N, int T, const int8_t *w_q, const float *w_step,
                                const float *smooth, const float *act_step, const int32_t *act_zero,
                                const float *bias, unsigned flags, int act_bits = 8)
{
    if (!out) return fail(PTQ_ERR_NULL, "out must not be NULL");
    *out = nullptr;
    if (!w_q || !w_step || !smooth || !act_step)
        return fail(PTQ_ERR_NULL, "w_q, w_step, smooth and act_step must not be NULL");
    if (K < 1 || K > PTQ_MAX_K || N < 1 || N > PTQ_MAX_N || T < 1 || T > PTQ_MAX_T)
        return fail(PTQ_ERR_SHAPE, "K, N, T out of range (K=%d N=%d T=%d)", K, N, T);
    if (flags != PTQ_FLAG_NONE) return fail(PTQ_ERR_VALUE, "flags must be PTQ_FLAG_NONE at create");

    // Parameter values (host-only checks come first so that they are testable without a device).
    const float lo = std::ldexp(1.0f, -30), hi = std::ldexp(1.0f, 30);
    bool fast = true;
    for (int k = 0; k < K; ++k) {
        if (!(smooth[k] > 0.0f) || !std::isfinite(smooth[k]))
            return fail(PTQ_ERR_VALUE, "smooth[%d] = %g must be finite and > 0", k, smooth[k]);
        if (smooth[k] < lo || smooth[k] > hi) fast = false;
    }
    for (int t = 0; t < T; ++t) {
        if (!(act_step[t] > 0.0f) || !std::isfinite(act_step[t]))
            return fail(PTQ_ERR_VALUE, "act_step[%d] = %g must be finite and > 0", t, act_step[t]);
        if (act_step[t] < lo || act_step[t] > hi) fast = false;
    }
    for (int n = 0; n < N; ++n) {
        if (!(w_step[n] > 0.0f) || !std::isfinite(w_step[n]))
            return fail(PTQ_ERR_VALUE, "w_step[%d] = %g must be finite and > 0", n, w_step[n]);
        if (bias && !std::isfinite(bias[n])) return fail(PTQ_ERR_VALUE, "bias[%d] is not finite", n);
    }
    for (int t = 0; act_zero && t < T; ++t)
        if (act_zero[t] < 0 || act_zero[t] > 255)
            return fail(PTQ_ERR_VALUE, "act_zero[%d] = %d is outside [0,255]", t, act_zero[t]);
    for (long long i = 0; i < static_cast<long long>(N) * K; ++i)
        if (w_q[i] == -128)
            return fail(PTQ_ERR_VALUE, "w_q[%lld] = -128 is outside the symmetric range [-127,127]", i);

    int dev = -1;
    PTQ_CUDA(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    PTQ_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10 || prop.minor != 0)
        return fail(PTQ_ERR_ARCH, "device %d is compute capability %d.%d; this library needs 10.0 (sm_100a)", dev,
                    prop.major, prop.minor);

    ptq_linear *h = new (std::nothrow) ptq_linear();
    if (!h) return fail(PTQ_ERR_NOMEM, "host allocation failed");
    h->K = K;
    h->N = N;
    h->T = T;
    h->Kpad = round_up(K, 16);
    h->device = dev;
    h->num_sms = prop.multiProcessorCount;
    h->fast_div = fast;
    h->n_tiles = (N + ptq::kMaxBN - 1) / ptq::kMaxBN;
    if (h->n_tiles == 1)
        h->BN = round_up(N, 16);
    else
        h->BN = round_up((N + h->n_tiles - 1) / h->n_tiles, 64);
    h->k_blocks = (K + ptq::kBK - 1) / ptq::kBK;
    h->last_mmas = (K - (h->k_blocks - 1) * ptq::kBK + 31) / 32;

    h->asym = act_zero != nullptr;
    h->has_bias = bias != nullptr;
    h->act_bits = act_bits;
    choose_astat(h);
    if (h->asym || act_bits != 8) h->as_ok = false;   // these layers run the quantize kernel + single-CTA GEMM kernel only
    int Npad = h->n_tiles * h->BN;
    if (h->as_ok && h->as_n_tiles * h->as_BN > Npad) Npad = h->as_n_tiles * h->as_BN;
    const int Nvec = round_up(Npad, 64) + 64;
    const int Kvec = round_up(K, 16);
    std::vector<int8_t> wpad(static_cast<size_t>(Npad) * h->Kpad, 0);
    for (int n = 0; n < N; ++n) std::memcpy(&wpad[static_cast<size_t>(n) * h->Kpad], w_q + static_cast<size_t>(n) * K, K);
    std::vector<float> rs(Kvec, 1.0f), sp(Kvec, 1.0f), rdx(T);
    for (int k = 0; k < K; ++k) {
        sp[k] = smooth[k];
        rs[k] = 1.0f / smooth[k];
    }
    std::vector<float> dx2(2 * static_cast<size_t>(T));
    for (int t = 0; t < T; ++t) {
        rdx[t] = 1.0f / act_step[t];
        dx2[2 * t] = act_step[t];
        dx2[2 * t + 1] = rdx[t];
    }

    ptq_status_t st = PTQ_OK;
    do {
        if ((st = upload(reinterpret_cast<void **>(&h->d_w), wpad.data(), wpad.size(), wpad.size())) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_dw), w_step, sizeof(float) * N, sizeof(float) * Nvec)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_bias), bias, bias ? sizeof(float) * N : 0, sizeof(float) * Nvec)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_s), sp.data(), sizeof(float) * Kvec, sizeof(float) * Kvec)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_rs), rs.data(), sizeof(float) * Kvec, sizeof(float) * Kvec)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_dx), act_step, sizeof(float) * T, sizeof(float) * T)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_rdx), rdx.data(), sizeof(float) * T, sizeof(float) * T)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_dx2), dx2.data(), sizeof(float) * 2 * T, sizeof(float) * 2 * T)) != PTQ_OK) break;
        if ((st = upload(reinterpret_cast<void **>(&h->d_status), nullptr, 0, sizeof(unsigned))) != PTQ_OK) break;
        if (h->asym) {
            std::vector<int> wsum(Nvec, 0);
            for (int n = 0; n < N; ++n) {
                int acc = 0;
                for (int k = 0; k < K; ++k) acc += w_q[static_cast<size_t>(n) * K + k];
                wsum[n] = acc;
            }
            if ((st = upload(reinterpret_cast<void **>(&h->d_zp), act_zero, sizeof(int) * T, sizeof(int) * T)) != PTQ_OK) break;
            if ((st = upload(reinterpret_cast<void **>(&h->d_wsum), wsum.data(), sizeof(int) * Nvec, sizeof(int) * Nvec)) != PTQ_OK) break;
        }
        st = make_map_2d(&h->tmW, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, h->d_w, static_cast<unsigned long long>(K),
                         static_cast<unsigned long long>(Npad), static_cast<unsigned long long>(h->Kpad), ptq::kBK,
                         static_cast<unsigned>(h->BN));
        if (st != PTQ_OK) break;
        st = make_map_2d(&h->tmWh, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, h->d_w, static_cast<unsigned long long>(K),
                         static_cast<unsigned long long>(Npad), static_cast<unsigned long long>(h->Kpad), ptq::kBK,
                         static_cast<unsigned>(h->BN / 2));
        if (st != PTQ_OK) break;
        h->max_pairs = h->asym ? 0 : query_max_pairs(dev);
        if (h->as_ok)
            st = make_map_2d(&h->tmWas, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, h->d_w, static_cast<unsigned long long>(K),
                             static_cast<unsigned long long>(Npad), static_cast<unsigned long long>(h->Kpad),
                             ptq::kBK, static_cast<unsigned>(h->as_BN));
        else
            h->tmWas = h->tmW;
    } while (0);
    if (st != PTQ_OK) {
        char keep[sizeof(g_err)];
        std::memcpy(keep, g_err, sizeof(keep));
        ptq_linear_destroy(h);
        std::memcpy(g_err, keep, sizeof(keep));
        return st;
    }
    *out = h;
    return PTQ_OK;
}

ptq_status_t ptq_linear_create(ptq_linear_t **out, int K, int N, int T, const int8_t *w_q, const float *w_step,
                               const float *smooth, const float *act_step, const float *bias, unsigned flags)
{
    return create_impl(out, K, N, T, w_q, w_step, smooth, act_step, nullptr, bias, flags);
}

ptq_status_t ptq_linear_create_asym(ptq_linear_t **out, int K, int N, int T, const int8_t *w_q, const float *w_step,
                                    const float *smooth, const float *act_step, const int32_t *act_zero,
                                    const float *bias, unsigned flags)
{
    if (out) *out = nullptr;
    if (!act_zero) return fail(PTQ_ERR_NULL, "act_zero must not be NULL");
    return create_impl(out, K, N, T, w_q, w_step, smooth, act_step, act_zero, bias, flags);
}

size_t ptq_linear_workspace_bytes(const ptq_linear_t *h, int B, unsigned flags)
{
    if (!h || B < 1) return 0;
    if ((flags & PTQ_FLAG_FUSED_PROLOGUE) && ptq_linear_fused_supported(h)) return 0;
    return static_cast<size_t>(B) * h->T * h->Kpad;
}

int ptq_linear_fused_supported(const ptq_linear_t *h) { return (h && fused_usable(h)) ? 1 : 0; }

ptq_status_t ptq_quantize(const ptq_linear_t *h, const void *x_fp16, int B, void *q_int8, void *stream)
{
    if (!h || !x_fp16 || !q_int8) return fail(PTQ_ERR_NULL, "handle, x and q must not be NULL");
    if (B < 1) return fail(PTQ_ERR_SHAPE, "B must be >= 1 (got %d)", B);
    if (reinterpret_cast<uintptr_t>(x_fp16) % 2) return fail(PTQ_ERR_ALIGN, "x must be 2-byte aligned");
    ptq_status_t st = check_device(h);
    if (st != PTQ_OK) return st;
    const long long M = static_cast<long long>(B) * h->T;
    if (ranges_overlap(x_fp16, static_cast<size_t>(M) * h->K * 2, q_int8, static_cast<size_t>(M) * h->K))
        return fail(PTQ_ERR_VALUE, "x and q overlap");
    return launch_quantize(h, x_fp16, M, q_int8, h->K, static_cast<cudaStream_t>(stream));
}

int ptq_linear_describe(const ptq_linear_t *h, char *buf, int buf_bytes)
{
    if (!h) return 0;
    char tmp[512];
    const int n = snprintf(tmp, sizeof(tmp),
                           "K=%d N=%d T=%d Kpad=%d%s | quantize: %s | gemm: BN=%d n_tiles=%d k_blocks=%d "
                           "pair_clusters=%d | fused: %s BN=%d n_tiles=%d w_stages=%d staging=%d smem=%d",
                           h->K, h->N, h->T, h->Kpad, h->asym ? " asymmetric" : (h->act_bits == 4 ? " w4a4" : ""),
                           h->fast_div ? "screened reciprocal route" : "IEEE division",
                           h->BN, h->n_tiles, h->k_blocks, h->max_pairs,
                           (h->as_ok && h->K % 16 == 0) ? "yes" : "no", h->as_BN, h->as_n_tiles, h->as_w_stages,
                           h->as_staging, h->as_smem);
    if (buf && buf_bytes > 0) {
        strncpy(buf, tmp, static_cast<size_t>(buf_bytes) - 1);
        buf[buf_bytes - 1] = 0;
    }
    return n;
}

int ptq_linear_code_pitch(const ptq_linear_t *h) { return h ? h->Kpad : 0; }

int ptq_linear_gemm_variant(const ptq_linear_t *h, int B)
{
    if (!h || B < 1) return -1;
    const long long M = static_cast<long long>(B) * h->T;
    if (h->N % 8 != 0) return 0;
    ptq::GemmParams p = {};
    p.BN = h->BN;
    p.n_tiles = h->n_tiles;
    p.m_tiles = static_cast<int>((M + ptq::kBM - 1) / ptq::kBM);
    p.k_blocks = h->k_blocks;
    p.has_bias = h->has_bias ? 1 : 0;
    const bool short_k = h->k_blocks <= PTQ_GEMM_SHORT_K_BLOCKS;
    p.boxes = short_k ? 2 : 1;
    if (plan_panel(h, p, true)) return 2;
    return gemm_teams(h, p, true, short_k) ? 1 : 0;
}

ptq_status_t ptq_linear_gemm_dequant(const ptq_linear_t *h, const void *q_int8, int B, void *y_fp16, void *stream)
{
    if (!h || !q_int8 || !y_fp16) return fail(PTQ_ERR_NULL, "handle, q and y must not be NULL");
    if (B < 1) return fail(PTQ_ERR_SHAPE, "B must be >= 1 (got %d)", B);
    if (reinterpret_cast<uintptr_t>(q_int8) % 16) return fail(PTQ_ERR_ALIGN, "q must be 16-byte aligned");
    if (reinterpret_cast<uintptr_t>(y_fp16) % 2) return fail(PTQ_ERR_ALIGN, "y must be 2-byte aligned");
    ptq_status_t st = check_device(h);
    if (st != PTQ_OK) return st;
    const long long M = static_cast<long long>(B) * h->T;
    if (ranges_overlap(q_int8, static_cast<size_t>(M) * h->Kpad, y_fp16, static_cast<size_t>(M) * h->N * 2))
        return fail(PTQ_ERR_VALUE, "q and y overlap");
    return launch_gemm(h, q_int8, M, y_fp16, nullptr, static_cast<cudaStream_t>(stream));
}

ptq_status_t ptq_linear_forward_debug(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                      void *q_int8_out, void *acc_int32_out, void *workspace,
                                      size_t workspace_bytes, unsigned flags, void *stream)
{
    ptq_status_t st = validate_forward(h, x_fp16, B, y_fp16);
    if (st != PTQ_OK) return st;
    if (flags & ~(PTQ_FLAG_FUSED_PROLOGUE | PTQ_FLAG_CTA_PAIR)) return fail(PTQ_ERR_VALUE, "unknown flags 0x%x", flags);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long long M = static_cast<long long>(B) * h->T;
    if ((flags & PTQ_FLAG_FUSED_PROLOGUE) && fused_usable(h) && reinterpret_cast<uintptr_t>(x_fp16) % 16 == 0) {
        // F1: one kernel, no workspace.  The codes never exist in memory; a requested tap is produced by
        // the quantize kernel on its own.
        if ((st = launch_fused(h, x_fp16, M, y_fp16, acc_int32_out, s)) != PTQ_OK) return st;
        if (q_int8_out) return launch_quantize(h, x_fp16, M, q_int8_out, h->K, s);
        return PTQ_OK;
    }
    const size_t need = static_cast<size_t>(M) * h->Kpad;
    if (!workspace) return fail(PTQ_ERR_NULL, "workspace must not be NULL for this layer, alignment and flags");
    if (workspace_bytes < need)
        return fail(PTQ_ERR_SHAPE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return fail(PTQ_ERR_ALIGN, "workspace must be 16-byte aligned");
    if (ranges_overlap(workspace, need, y_fp16, static_cast<size_t>(M) * h->N * 2) ||
        ranges_overlap(workspace, need, x_fp16, static_cast<size_t>(M) * h->K * 2))
        return fail(PTQ_ERR_VALUE, "workspace overlaps x or y");
    if ((st = launch_quantize(h, x_fp16, M, workspace, h->Kpad, s)) != PTQ_OK) return st;
    if ((st = launch_gemm(h, workspace, M, y_fp16, acc_int32_out, s, (flags & PTQ_FLAG_CTA_PAIR) != 0)) != PTQ_OK)
        return st;
    if (q_int8_out)
        PTQ_CUDA(cudaMemcpy2DAsync(q_int8_out, h->K, workspace, h->Kpad, h->K, static_cast<size_t>(M),
                                   cudaMemcpyDeviceToDevice, s));
    return PTQ_OK;
}

ptq_status_t ptq_linear_forward(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16, void *workspace,
                                size_t workspace_bytes, unsigned flags, void *stream)
{
    return ptq_linear_forward_debug(h, x_fp16, B, y_fp16, nullptr, nullptr, workspace, workspace_bytes, flags, stream);
}

ptq_status_t ptq_linear_forward_static(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                       void *stream)
{
    ptq_status_t st = validate_forward(h, x_fp16, B, y_fp16);
    if (st != PTQ_OK) return st;
    const long long M = static_cast<long long>(B) * h->T;
    const unsigned long long need = static_cast<unsigned long long>(M) * h->Kpad;
    if (need > PTQ_STATIC_SCRATCH_BYTES)
        return fail(PTQ_ERR_SHAPE,
                    "B*T*pitch = %llu bytes of codes exceed the built-in scratch of %u bytes; "
                    "split the batch or use ptq_linear_forward with a caller workspace",
                    need, PTQ_STATIC_SCRATCH_BYTES);
    void *scratch = nullptr;
    if ((st = static_scratch_address(h->device, &scratch)) != PTQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = launch_quantize(h, x_fp16, M, scratch, h->Kpad, s)) != PTQ_OK) return st;
    return launch_gemm(h, scratch, M, y_fp16, nullptr, s);
}

ptq_status_t ptq_search_act_step(int K, int T, const void *xcal_fp16, int Bc, const float *smooth,
                                 const float *base_step, int n_grid, int j_lo, float *act_step_out,
                                 int32_t *best_out, double *loss_out, void *stream)
{
    if (!xcal_fp16 || !smooth || !base_step || !act_step_out)
        return fail(PTQ_ERR_NULL, "search: pointers must not be NULL");
    if (K < 1 || K > PTQ_MAX_K || T < 1 || T > PTQ_MAX_T || Bc < 1 ||
        static_cast<long long>(Bc) * K > 0x7fffffffll)
        return fail(PTQ_ERR_SHAPE, "search: dimensions out of range (K=%d T=%d Bc=%d)", K, T, Bc);
    if (n_grid < 1 || n_grid > PTQ_MAX_SEARCH_GRID || j_lo < 1 || j_lo > n_grid)
        return fail(PTQ_ERR_VALUE, "search: need 1 <= j_lo <= n_grid <= %d (got j_lo=%d n_grid=%d)",
                    PTQ_MAX_SEARCH_GRID, j_lo, n_grid);
    if (reinterpret_cast<uintptr_t>(xcal_fp16) % 2) return fail(PTQ_ERR_ALIGN, "xcal must be 2-byte aligned");
    for (int k = 0; k < K; ++k)
        if (!(smooth[k] > 0.0f) || !std::isfinite(smooth[k]))
            return fail(PTQ_ERR_VALUE, "search: smooth[%d] = %g is not positive and finite", k, smooth[k]);
    for (int t = 0; t < T; ++t)
        if (!(base_step[t] >= 1e-30f) || !std::isfinite(base_step[t]))
            return fail(PTQ_ERR_VALUE, "search: base_step[%d] = %g is not in [1e-30, inf)", t, base_step[t]);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int C = n_grid - j_lo + 1;
    float *d_f = nullptr;      // [K] s, [T] base, [T] dx
    int *d_best = nullptr;     // [T]
    double *d_loss = nullptr;  // [T, C]
    auto body = [&]() -> ptq_status_t {
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_f), sizeof(float) * (K + 2 * static_cast<size_t>(T))));
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_best), sizeof(int) * static_cast<size_t>(T)));
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_loss), sizeof(double) * static_cast<size_t>(T) * C));
        PTQ_CUDA(cudaMemcpyAsync(d_f, smooth, sizeof(float) * K, cudaMemcpyHostToDevice, s));
        PTQ_CUDA(cudaMemcpyAsync(d_f + K, base_step, sizeof(float) * T, cudaMemcpyHostToDevice, s));
        ptq::SearchParams p;
        p.x = static_cast<const __half *>(xcal_fp16);
        p.s = d_f;
        p.base = d_f + K;
        p.loss = d_loss;
        p.Bc = Bc;
        p.T = T;
        p.K = K;
        p.n_grid = n_grid;
        p.j_lo = j_lo;
        const dim3 grid(static_cast<unsigned>(T), static_cast<unsigned>((C + ptq::kSearchCandPerBlock - 1) / ptq::kSearchCandPerBlock));
        ptq::ptq_search_loss_kernel<<<grid, ptq::kSearchThreads, 0, s>>>(p);
        ptq::ptq_search_pick_kernel<<<(T + 127) / 128, 128, 0, s>>>(d_loss, d_f + K, T, n_grid, j_lo, d_best, d_f + K + T);
        g_launches.fetch_add(2, std::memory_order_relaxed);
        PTQ_CUDA(cudaGetLastError());
        PTQ_CUDA(cudaMemcpyAsync(act_step_out, d_f + K + T, sizeof(float) * T, cudaMemcpyDeviceToHost, s));
        if (best_out) PTQ_CUDA(cudaMemcpyAsync(best_out, d_best, sizeof(int) * T, cudaMemcpyDeviceToHost, s));
        if (loss_out)
            PTQ_CUDA(cudaMemcpyAsync(loss_out, d_loss, sizeof(double) * static_cast<size_t>(T) * C, cudaMemcpyDeviceToHost, s));
        PTQ_CUDA(cudaStreamSynchronize(s));
        return PTQ_OK;
    };
    const ptq_status_t st = body();
    cudaFree(d_f);
    cudaFree(d_best);
    cudaFree(d_loss);
    return st;
}

static size_t dynamic_codes_bytes(const ptq_linear *h, long long M)
{
    return (static_cast<size_t>(M) * h->Kpad + 255) / 256 * 256;
}

size_t ptq_linear_workspace_bytes_dynamic(const ptq_linear_t *h, int B)
{
    if (!h || B < 1) return 0;
    const long long M = static_cast<long long>(B) * h->T;
    return dynamic_codes_bytes(h, M) + static_cast<size_t>(M) * sizeof(float);
}

ptq_status_t ptq_linear_forward_dynamic_debug(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                              void *q_int8_out, void *acc_int32_out, void *step_fp32_out,
                                              void *workspace, size_t workspace_bytes, void *stream)
{
    ptq_status_t st = validate_forward(h, x_fp16, B, y_fp16);
    if (st != PTQ_OK) return st;
    if (h->asym || h->act_bits != 8)
        return fail(PTQ_ERR_VALUE, "the dynamic comparator is defined for symmetric 8-bit layers only");
    const long long M = static_cast<long long>(B) * h->T;
    const size_t codes = dynamic_codes_bytes(h, M);
    const size_t need = codes + static_cast<size_t>(M) * sizeof(float);
    if (!workspace) return fail(PTQ_ERR_NULL, "workspace must not be NULL");
    if (workspace_bytes < need)
        return fail(PTQ_ERR_SHAPE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return fail(PTQ_ERR_ALIGN, "workspace must be 16-byte aligned");
    if (ranges_overlap(workspace, need, y_fp16, static_cast<size_t>(M) * h->N * 2) ||
        ranges_overlap(workspace, need, x_fp16, static_cast<size_t>(M) * h->K * 2))
        return fail(PTQ_ERR_VALUE, "workspace overlaps x or y");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float *dx_row = reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + codes);
    if ((st = launch_quantize_dynamic(h, x_fp16, M, workspace, h->Kpad, dx_row, s)) != PTQ_OK) return st;
    if ((st = launch_gemm(h, workspace, M, y_fp16, acc_int32_out, s, false, dx_row)) != PTQ_OK) return st;
    if (q_int8_out)
        PTQ_CUDA(cudaMemcpy2DAsync(q_int8_out, h->K, workspace, h->Kpad, h->K, static_cast<size_t>(M),
                                   cudaMemcpyDeviceToDevice, s));
    if (step_fp32_out)
        PTQ_CUDA(cudaMemcpyAsync(step_fp32_out, dx_row, static_cast<size_t>(M) * sizeof(float),
                                 cudaMemcpyDeviceToDevice, s));
    return PTQ_OK;
}

ptq_status_t ptq_linear_forward_dynamic(const ptq_linear_t *h, const void *x_fp16, int B, void *y_fp16,
                                        void *workspace, size_t workspace_bytes, void *stream)
{
    return ptq_linear_forward_dynamic_debug(h, x_fp16, B, y_fp16, nullptr, nullptr, nullptr, workspace,
                                            workspace_bytes, stream);
}

ptq_status_t ptq_linear_device_status(const ptq_linear_t *h)
{
    if (!h) return fail(PTQ_ERR_NULL, "handle must not be NULL");
    ptq_status_t st = check_device(h);
    if (st != PTQ_OK) return st;
    unsigned word = 0;
    PTQ_CUDA(cudaDeviceSynchronize());
    PTQ_CUDA(cudaMemcpy(&word, h->d_status, sizeof(word), cudaMemcpyDeviceToHost));
    if (word & ptq::PTQ_DEV_SMEM_ALIGN) {
        PTQ_CUDA(cudaMemset(h->d_status, 0, sizeof(word)));
        return fail(PTQ_ERR_CUDA, "a kernel found its shared memory misaligned and did not run (status word 0x%x); its output is undefined", word);
    }
    if (word) {
        PTQ_CUDA(cudaMemset(h->d_status, 0, sizeof(word)));
        return fail(PTQ_ERR_TIMEOUT, "a kernel abandoned a bounded wait (status word 0x%x); its output is undefined", word);
    }
    return PTQ_OK;
}

ptq_status_t ptq_linear_selftest_wait_timeout(const ptq_linear_t *h, unsigned limit_us, unsigned *result3, void *stream)
{
    if (!h || !result3) return fail(PTQ_ERR_NULL, "handle and result must not be NULL");
    if (limit_us < 1 || limit_us > 100000) return fail(PTQ_ERR_VALUE, "limit_us must be in [1, 100000] (got %u)", limit_us);
    ptq_status_t st = check_device(h);
    if (st != PTQ_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned *d_out = nullptr;
    PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_out), 3 * sizeof(unsigned)));
    auto body = [&]() -> ptq_status_t {
        PTQ_CUDA(cudaMemsetAsync(d_out, 0xff, 3 * sizeof(unsigned), s));
        ptq::ptq_wait_selftest_kernel<<<1, 64, 0, s>>>(h->d_status, 1000ull * limit_us, d_out);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        PTQ_CUDA(cudaGetLastError());
        PTQ_CUDA(cudaMemcpyAsync(result3, d_out, 3 * sizeof(unsigned), cudaMemcpyDeviceToHost, s));
        PTQ_CUDA(cudaStreamSynchronize(s));
        return PTQ_OK;
    };
    st = body();
    cudaFree(d_out);
    return st;
}

ptq_status_t ptq_probe(int kind, void *buf, size_t bytes, int iters, double *result, void *stream)
{
    if (!result) return fail(PTQ_ERR_NULL, "probe: result must not be NULL");
    *result = 0.0;
    if (kind < ptq::kProbeStore16 || kind > ptq::kProbeLaunchPdl) return fail(PTQ_ERR_VALUE, "probe: unknown kind %d", kind);
    if (iters < 1 || iters > 100000) return fail(PTQ_ERR_VALUE, "probe: iters must be in [1, 100000] (got %d)", iters);
    const bool moves_bytes = kind <= ptq::kProbeOperandPull;
    if (moves_bytes && !buf) return fail(PTQ_ERR_NULL, "probe: buf must not be NULL for this kind");
    if (moves_bytes && reinterpret_cast<uintptr_t>(buf) % 256) return fail(PTQ_ERR_ALIGN, "probe: buf must be 256-byte aligned");
    int dev = -1, sms = 0, major = 0, minor = 0;
    PTQ_CUDA(cudaGetDevice(&dev));
    PTQ_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    PTQ_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    PTQ_CUDA(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
    if (major != 10 || minor != 0)
        return fail(PTQ_ERR_ARCH, "device %d is compute capability %d.%d; this library needs 10.0 (sm_100a)", dev, major, minor);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    constexpr size_t kTail = 256;                      // the last 256 bytes of buf hold the kernels' status word
    constexpr int N = 3072, K = 768;                   // the Vim-B in_proj shape: y [M, 3072] fp16, codes [M, 768], weights [3072, 768]
    unsigned char *base = static_cast<unsigned char *>(buf);
    unsigned *status = moves_bytes ? reinterpret_cast<unsigned *>(base + (bytes >= kTail ? bytes - kTail : 0)) : nullptr;
    double moved = 0.0;                                // bytes per launch
    int grid = sms, m_tiles = 0;
    CUtensorMap tm0, tm1;
    if (kind == ptq::kProbeStore16) {
        if (bytes < kTail + (1u << 20)) return fail(PTQ_ERR_SHAPE, "probe: buf too small (%zu bytes)", bytes);
        moved = static_cast<double>((bytes - kTail) / 16 * 16);
        grid = sms * 32;
    } else if (kind == ptq::kProbeTmaStore) {
        m_tiles = static_cast<int>((bytes - (bytes >= kTail ? kTail : bytes)) / (static_cast<size_t>(N) * 2 * ptq::kBM));
        if (m_tiles < 1) return fail(PTQ_ERR_SHAPE, "probe: buf too small (%zu bytes)", bytes);
        if (m_tiles > 4096) m_tiles = 4096;
        ptq_status_t st = make_map_2d(&tm0, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, N, static_cast<unsigned long long>(m_tiles) * ptq::kBM,
                                      static_cast<unsigned long long>(N) * 2, 64, 32);
        if (st != PTQ_OK) return st;
        moved = static_cast<double>(m_tiles) * ptq::kBM * N * 2;
        PTQ_CUDA(cudaFuncSetAttribute(ptq::ptq_probe_tma_store_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * ptq::kProbeBoxBytes));
    } else if (kind == ptq::kProbeOperandPull) {
        const size_t w_bytes = static_cast<size_t>(N) * K;
        if (bytes < kTail + w_bytes + static_cast<size_t>(ptq::kBM) * K) return fail(PTQ_ERR_SHAPE, "probe: buf too small (%zu bytes)", bytes);
        m_tiles = static_cast<int>((bytes - kTail - w_bytes) / (static_cast<size_t>(ptq::kBM) * K));
        if (m_tiles > 4096) m_tiles = 4096;
        ptq_status_t st = make_map_2d(&tm0, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, base + w_bytes, K, static_cast<unsigned long long>(m_tiles) * ptq::kBM, K, 128, 128);
        if (st == PTQ_OK) st = make_map_2d(&tm1, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, base, K, N, K, 128, 256);
        if (st != PTQ_OK) return st;
        moved = static_cast<double>(m_tiles) * (N / 256) * (K / 128) * ptq::kProbeStageBytes;
        PTQ_CUDA(cudaFuncSetAttribute(ptq::ptq_probe_operand_pull_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      4 * ptq::kProbeStageBytes + 128));
    }
    if (status) PTQ_CUDA(cudaMemsetAsync(status, 0, sizeof(unsigned), s));
    auto launch = [&]() -> cudaError_t {
        switch (kind) {
            case ptq::kProbeStore16:
                ptq::ptq_probe_store16_kernel<<<grid, 256, 0, s>>>(reinterpret_cast<uint4 *>(base), static_cast<unsigned long long>(moved / 16));
                break;
            case ptq::kProbeTmaStore:
                ptq::ptq_probe_tma_store_kernel<<<sms, 256, 8 * ptq::kProbeBoxBytes, s>>>(tm0, m_tiles, N / 256);
                break;
            case ptq::kProbeOperandPull:
                ptq::ptq_probe_operand_pull_kernel<<<sms, 64, 4 * ptq::kProbeStageBytes + 128, s>>>(tm0, tm1, m_tiles, N / 256, K / 128, status);
                break;
            case ptq::kProbeLaunch:
                ptq::ptq_probe_empty_kernel<<<sms, 256, 0, s>>>(0);
                break;
            default:
                return launch_pdl(ptq::ptq_probe_empty_kernel, sms, 256, 0, s, 1);
        }
        return cudaGetLastError();
    };
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    PTQ_CUDA(cudaEventCreate(&e0));
    cudaError_t err = cudaEventCreate(&e1);
    for (int i = 0; i < 3 && err == cudaSuccess; ++i) err = launch();
    if (err == cudaSuccess) err = cudaEventRecord(e0, s);
    for (int i = 0; i < iters && err == cudaSuccess; ++i) err = launch();
    if (err == cudaSuccess) err = cudaEventRecord(e1, s);
    if (err == cudaSuccess) err = cudaEventSynchronize(e1);
    float ms = 0.0f;
    if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
    g_launches.fetch_add(static_cast<unsigned long long>(iters) + 3ull, std::memory_order_relaxed);
    cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (err != cudaSuccess) return fail(PTQ_ERR_CUDA, "probe: %s", cudaGetErrorString(err));
    if (status) {
        unsigned word = 0;
        PTQ_CUDA(cudaMemcpy(&word, status, sizeof(word), cudaMemcpyDeviceToHost));
        if (word) return fail(PTQ_ERR_TIMEOUT, "probe: a bounded wait gave up (status word 0x%x)", word);
    }
    const double per_launch_s = static_cast<double>(ms) * 1e-3 / iters;
    *result = moves_bytes ? moved / per_launch_s / 1e9 : per_launch_s * 1e6;   // GB/s, or microseconds per launch
    return PTQ_OK;
}

static ptq_status_t calibrate_impl(int K, int N, int T, const void *xcal_fp16, int Bc, const int8_t *w_q,
                                   const float *w_step, float *smooth_out, float *act_step_out,
                                   int32_t *act_zero_out, void *stream, float qmax = 127.0f,
                                   bool per_tensor = false)
{
    if (!xcal_fp16 || !w_q || !w_step || !smooth_out || !act_step_out)
        return fail(PTQ_ERR_NULL, "calibrate: pointers must not be NULL");
    if (K < 1 || K > PTQ_MAX_K || N < 1 || N > PTQ_MAX_N || T < 1 || T > PTQ_MAX_T || Bc < 1)
        return fail(PTQ_ERR_SHAPE, "calibrate: dimensions out of range (K=%d N=%d T=%d Bc=%d)", K, N, T, Bc);
    if (reinterpret_cast<uintptr_t>(xcal_fp16) % 2) return fail(PTQ_ERR_ALIGN, "xcal must be 2-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev = -1, sms = 0;
    PTQ_CUDA(cudaGetDevice(&dev));
    PTQ_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long M = static_cast<long long>(Bc) * T;

    unsigned *d_bits = nullptr;   // [K] maxX bits, then [T] mu (or hi) bits, then [T] -lo bits, then [K] maxW bits
    float *d_out = nullptr;       // [K] s, then [T] dx, then [T] z (int)
    float *d_dw = nullptr;
    int8_t *d_w = nullptr;
    ptq_status_t st = PTQ_OK;
    auto body = [&]() -> ptq_status_t {
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_bits), sizeof(unsigned) * (2 * K + 2 * T)));
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_out), sizeof(float) * (K + 2 * T)));
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_dw), sizeof(float) * N));
        PTQ_CUDA(cudaMalloc(reinterpret_cast<void **>(&d_w), static_cast<size_t>(N) * K));
        PTQ_CUDA(cudaMemsetAsync(d_bits, 0, sizeof(unsigned) * (2 * K + 2 * T), s));
        PTQ_CUDA(cudaMemcpyAsync(d_dw, w_step, sizeof(float) * N, cudaMemcpyHostToDevice, s));
        PTQ_CUDA(cudaMemcpyAsync(d_w, w_q, static_cast<size_t>(N) * K, cudaMemcpyHostToDevice, s));
        const __half *x = static_cast<const __half *>(xcal_fp16);
        long long want = (M + 7) / 8;
        if (want > sms * 8ll) want = sms * 8ll;
        const int grid = static_cast<int>(want < 1 ? 1 : want);
        ptq::ptq_calib_colmax_kernel<<<grid, 256, 0, s>>>(x, M, K, d_bits);
        unsigned *d_wbits = d_bits + K + 2 * T;
        const dim3 wgrid(static_cast<unsigned>((K + 127) / 128),
                         static_cast<unsigned>((N + ptq::kCalibRowsPerBlock - 1) / ptq::kCalibRowsPerBlock));
        ptq::ptq_calib_wmax_kernel<<<wgrid, 128, 0, s>>>(d_w, d_dw, N, K, d_wbits);
        ptq::ptq_calib_smooth_kernel<<<(K + 127) / 128, 128, 0, s>>>(d_bits, d_wbits, K, d_out);
        if (act_zero_out) {
            ptq::ptq_calib_rowrange_kernel<<<grid, 256, 0, s>>>(x, M, K, T, d_out, d_bits + K, d_bits + K + T);
            ptq::ptq_calib_step_asym_kernel<<<(T + 127) / 128, 128, 0, s>>>(d_bits + K, d_bits + K + T, T, d_out + K,
                                                                           reinterpret_cast<int *>(d_out + K + T));
        } else {
            ptq::ptq_calib_rowmax_kernel<<<grid, 256, 0, s>>>(x, M, K, T, d_out, d_bits + K);
            if (per_tensor)
                ptq::ptq_calib_step_tensor_kernel<<<1, 256, 0, s>>>(d_bits + K, T, d_out + K, qmax);
            else
                ptq::ptq_calib_step_kernel<<<(T + 127) / 128, 128, 0, s>>>(d_bits + K, T, d_out + K, qmax);
        }
        g_launches.fetch_add(5, std::memory_order_relaxed);
        PTQ_CUDA(cudaGetLastError());
        PTQ_CUDA(cudaMemcpyAsync(smooth_out, d_out, sizeof(float) * K, cudaMemcpyDeviceToHost, s));
        PTQ_CUDA(cudaMemcpyAsync(act_step_out, d_out + K, sizeof(float) * T, cudaMemcpyDeviceToHost, s));
        if (act_zero_out)
            PTQ_CUDA(cudaMemcpyAsync(act_zero_out, d_out + K + T, sizeof(int32_t) * T, cudaMemcpyDeviceToHost, s));
        PTQ_CUDA(cudaStreamSynchronize(s));
        return PTQ_OK;
    };
    st = body();
    cudaFree(d_bits);
    cudaFree(d_out);
    cudaFree(d_dw);
    cudaFree(d_w);
    return st;
}

ptq_status_t ptq_calibrate(int K, int N, int T, const void *xcal_fp16, int Bc, const int8_t *w_q,
                           const float *w_step, float *smooth_out, float *act_step_out, void *stream)
{
    return calibrate_impl(K, N, T, xcal_fp16, Bc, w_q, w_step, smooth_out, act_step_out, nullptr, stream);
}

ptq_status_t ptq_calibrate_per_tensor(int K, int N, int T, const void *xcal_fp16, int Bc, const int8_t *w_q,
                                      const float *w_step, float *smooth_out, float *act_step_out, void *stream)
{
    return calibrate_impl(K, N, T, xcal_fp16, Bc, w_q, w_step, smooth_out, act_step_out, nullptr, stream, 127.0f, true);
}

ptq_status_t ptq_calibrate_asym(int K, int N, int T, const void *xcal_fp16, int Bc, const int8_t *w_q,
                                const float *w_step, float *smooth_out, float *act_step_out,
                                int32_t *act_zero_out, void *stream)
{
    if (!act_zero_out) return fail(PTQ_ERR_NULL, "calibrate: pointers must not be NULL");
    return calibrate_impl(K, N, T, xcal_fp16, Bc, w_q, w_step, smooth_out, act_step_out, act_zero_out, stream);
}

// Sign-extending unpack of rows of 4-bit values, two per byte, low nibble = even column.
static void unpack_int4_host(const uint8_t *packed, int rows, int cols, std::vector<int8_t> &out)
{
    const int pb = (cols + 1) / 2;
    out.resize(static_cast<size_t>(rows) * cols);
    for (int r = 0; r < rows; ++r)
        for (int k = 0; k < cols; ++k) {
            const int nib = (packed[static_cast<size_t>(r) * pb + k / 2] >> ((k & 1) * 4)) & 15;
            out[static_cast<size_t>(r) * cols + k] = static_cast<int8_t>(nib >= 8 ? nib - 16 : nib);
        }
}

ptq_status_t ptq_linear_create_w4a4(ptq_linear_t **out, int K, int N, int T, const uint8_t *w_q_packed,
                                    const float *w_step, const float *smooth, const float *act_step,
                                    const float *bias, unsigned flags)
{
    if (!out) return fail(PTQ_ERR_NULL, "out must not be NULL");
    *out = nullptr;
    if (!w_q_packed) return fail(PTQ_ERR_NULL, "w_q_packed must not be NULL");
    if (K < 1 || K > PTQ_MAX_K || N < 1 || N > PTQ_MAX_N)
        return fail(PTQ_ERR_SHAPE, "K, N out of range (K=%d N=%d)", K, N);
    std::vector<int8_t> w;
    unpack_int4_host(w_q_packed, N, K, w);
    return create_impl(out, K, N, T, w.data(), w_step, smooth, act_step, nullptr, bias, flags, 4);
}

ptq_status_t ptq_calibrate_w4a4(int K, int N, int T, const void *xcal_fp16, int Bc, const uint8_t *w_q_packed,
                                const float *w_step, float *smooth_out, float *act_step_out, void *stream)
{
    if (!w_q_packed) return fail(PTQ_ERR_NULL, "calibrate: pointers must not be NULL");
    if (K < 1 || K > PTQ_MAX_K || N < 1 || N > PTQ_MAX_N)
        return fail(PTQ_ERR_SHAPE, "calibrate: dimensions out of range (K=%d N=%d)", K, N);
    std::vector<int8_t> w;
    unpack_int4_host(w_q_packed, N, K, w);
    return calibrate_impl(K, N, T, xcal_fp16, Bc, w.data(), w_step, smooth_out, act_step_out, nullptr, stream, 7.0f);
}

ptq_status_t ptq_quantize_packed4(const ptq_linear_t *h, const void *x_fp16, int B, void *q_packed, void *workspace,
                                  size_t workspace_bytes, void *stream)
{
    if (!h || !x_fp16 || !q_packed || !workspace) return fail(PTQ_ERR_NULL, "handle, x, q and workspace must not be NULL");
    if (h->act_bits != 4) return fail(PTQ_ERR_VALUE, "packed 4-bit codes need a layer made by ptq_linear_create_w4a4");
    if (B < 1) return fail(PTQ_ERR_SHAPE, "B must be >= 1 (got %d)", B);
    if (reinterpret_cast<uintptr_t>(x_fp16) % 2) return fail(PTQ_ERR_ALIGN, "x must be 2-byte aligned");
    if (reinterpret_cast<uintptr_t>(workspace) % 16) return fail(PTQ_ERR_ALIGN, "workspace must be 16-byte aligned");
    ptq_status_t st = check_device(h);
    if (st != PTQ_OK) return st;
    const long long M = static_cast<long long>(B) * h->T;
    const size_t need = static_cast<size_t>(M) * h->Kpad;
    if (workspace_bytes < need) return fail(PTQ_ERR_SHAPE, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    const size_t out_bytes = static_cast<size_t>(M) * ((h->K + 1) / 2);
    if (ranges_overlap(workspace, need, q_packed, out_bytes) ||
        ranges_overlap(workspace, need, x_fp16, static_cast<size_t>(M) * h->K * 2) ||
        ranges_overlap(q_packed, out_bytes, x_fp16, static_cast<size_t>(M) * h->K * 2))
        return fail(PTQ_ERR_VALUE, "x, q and workspace overlap");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if ((st = launch_quantize(h, x_fp16, M, workspace, h->Kpad, s)) != PTQ_OK) return st;
    long long want = (static_cast<long long>(out_bytes) + 255) / 256;
    const long long cap = static_cast<long long>(h->num_sms) * 16;
    if (want > cap) want = cap;
    ptq::ptq_pack_int4_kernel<<<static_cast<int>(want), 256, 0, s>>>(static_cast<const int8_t *>(workspace), M, h->K,
                                                                    h->Kpad, static_cast<uint8_t *>(q_packed));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    PTQ_CUDA(cudaGetLastError());
    return PTQ_OK;
}

}  // extern "C"
