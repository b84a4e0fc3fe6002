// libgq C-ABI (see include/gq.h): argument validation, tensor maps, launches.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <utility>
#include <vector>

#include "../../include/gq.h"
#include "gq_hessian.cuh"
#include "gq_objective.cuh"
#include "gq_cd.cuh"
#include "gq_codebook.cuh"
#include "gq_exchange.cuh"
#include "gq_wide_gemm.cuh"
#include "gq_gram_dot.cuh"
#include "gq_kernels.cuh"

#define GQ_VERSION_NUMBER 100   /* 0.1.0 */

namespace {

constexpr int kMaxDevices = 64;

thread_local int32_t tl_last_cuda_error = 0;
std::atomic<uint64_t> g_launches{0};

// Optional per-kernel timing (gq_kernel_timing_*): a pair of events around every launch.
std::atomic<int> g_timing_on{0};
std::mutex g_timing_mutex;
std::vector<std::pair<cudaEvent_t, cudaEvent_t>> g_timing_events[GQ_KERNEL_COUNT];

struct LaunchScope {
    int id;
    cudaStream_t st;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    LaunchScope(int id_, cudaStream_t st_) : id(id_), st(st_)
    {
        g_launches.fetch_add(1);
        if (g_timing_on.load(std::memory_order_relaxed)) {
            if (cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess) {
                cudaEventRecord(e0, st);
            } else {
                if (e0) cudaEventDestroy(e0);
                e0 = e1 = nullptr;
            }
        }
    }
    ~LaunchScope()
    {
        if (e0) {
            cudaEventRecord(e1, st);
            std::lock_guard<std::mutex> lock(g_timing_mutex);
            g_timing_events[id].emplace_back(e0, e1);
        }
    }
};

// Per-device status word {status, site, block, unit}; written by kernels, read by gq_check().
__device__ uint32_t g_status_word[4];

struct DeviceInfo {
    bool ready = false;
    int sm_count = 0;
    int max_pairs = 0;          // CTA pairs (clusters of two) of a tensor-core kernel that can be resident at once
    uint32_t *status_ptr = nullptr;
};
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mutex;
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

#define GQ_CUDA(call)                                   \
    do {                                                \
        cudaError_t e_ = (call);                        \
        if (e_ != cudaSuccess) {                        \
            tl_last_cuda_error = static_cast<int32_t>(e_); \
            return GQ_ERR_CUDA;                         \
        }                                               \
    } while (0)

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// True if the byte ranges [a, a + na) and [b, b + nb) share a byte (empty ranges never do).
inline bool overlaps(const void *a, size_t na, const void *b, size_t nb)
{
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + nb && b0 < a0 + na;
}
// Bytes spanned by `rows` rows of `width` elements with leading dimension `ld` (elements of `elem` bytes).
inline size_t span_bytes(int64_t rows, int64_t width, int64_t ld, size_t elem)
{
    if (rows <= 0 || width <= 0) return 0;
    return (static_cast<size_t>(rows - 1) * static_cast<size_t>(ld) + static_cast<size_t>(width)) * elem;
}
// True if two row sets of fp32 elements share an element: `rows` rows of width na at a (leading dimension ld_a)
// and of width nb at b (leading dimension ld_b).  Exact when the leading dimensions are equal (two column
// ranges of one [rows, ld] buffer interleave without touching); otherwise decided by the spans.
inline bool rows_overlap_f32(const float *a, int64_t na, int64_t ld_a, const float *b, int64_t nb, int64_t ld_b, int64_t rows)
{
    if (!overlaps(a, span_bytes(rows, na, ld_a, 4), b, span_bytes(rows, nb, ld_b, 4))) return false;
    const intptr_t diff = reinterpret_cast<intptr_t>(b) - reinterpret_cast<intptr_t>(a);
    if (ld_a != ld_b || diff % 4 != 0) return true;
    const int64_t D = diff / 4, ld = ld_a;
    int64_t r = D % ld, q = D / ld;
    if (r < 0) {
        r += ld;
        q -= 1;
    }
    // element (k, i) of a and (k', j) of b coincide iff (k - k') ld = D + j - i, i.e. r + j - i is 0 or ld
    const bool same_row = r < na && q > -rows && q < rows;                 // r + j - i = 0, k - k' = q
    const bool next_row = r + nb > ld && q + 1 > -rows && q + 1 < rows;    // r + j - i = ld, k - k' = q + 1
    return same_row || next_row;
}

int32_t device_info(DeviceInfo **out)
{
    int dev = 0;
    GQ_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return GQ_ERR_UNSUPPORTED_SHAPE;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceInfo &di = g_dev[dev];
    if (!di.ready) {
        GQ_CUDA(cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev));
        void *sym = nullptr;
        GQ_CUDA(cudaGetSymbolAddress(&sym, g_status_word));
        di.status_ptr = static_cast<uint32_t *>(sym);
        GQ_CUDA(cudaFuncSetAttribute(gq::pair_gemm_kernel<gq::MODE_OBJECTIVE>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, gq::OBJ_SMEM_BYTES));
        GQ_CUDA(cudaFuncSetAttribute(gq::pair_gemm_kernel<gq::MODE_PANEL>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, gq::OBJ_SMEM_BYTES));
        GQ_CUDA(cudaFuncSetAttribute(gq::pair_gemm_kernel<gq::MODE_FULL>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, gq::OBJ_SMEM_BYTES));
        GQ_CUDA(cudaFuncSetAttribute(gq::wide_gemm_kernel<gq::WG_FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, gq::WG_SMEM_BYTES));
        GQ_CUDA(cudaFuncSetAttribute(gq::gram_dot_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, gq::GD_SMEM_BYTES));
        GQ_CUDA(cudaFuncSetAttribute(gq::cd_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     gq::CD_SMEM_BYTES));
        GQ_CUDA(cudaFuncSetAttribute(gq::hessian_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     gq::HS_SMEM_BYTES));
        {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(static_cast<unsigned>(di.sm_count & ~1));
            cfg.blockDim = dim3(gq::HS_THREADS);
            cfg.dynamicSmemBytes = gq::HS_SMEM_BYTES;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = 2;
            attr.val.clusterDim.y = 1;
            attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, gq::hessian_kernel, &cfg) != cudaSuccess ||
                clusters < 1) {
                (void)cudaGetLastError();
                clusters = di.sm_count / 2;
            }
            if (clusters > di.sm_count / 2) clusters = di.sm_count / 2;
            if (clusters < 1) clusters = 1;
            di.max_pairs = clusters;
        }
        if (!g_encode) {
            void *fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            GQ_CUDA(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
            if (qres != cudaDriverEntryPointSuccess || !fn) {
                tl_last_cuda_error = static_cast<int32_t>(cudaErrorNotSupported);
                return GQ_ERR_CUDA;
            }
            g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
        }
        di.ready = true;
    }
    *out = &di;
    return GQ_OK;
}

unsigned long long wait_budget_ns()
{
    static const unsigned long long v = [] {
        const char *e = std::getenv("GQ_WAIT_BUDGET_MS");
        long ms = e ? std::atol(e) : 2000;
        if (ms < 1) ms = 1;
        if (ms > 60000) ms = 60000;
        return static_cast<unsigned long long>(ms) * 1000000ull;
    }();
    return v;
}

// 16-bit tensor [groups][rows][features] (bf16 unless `dtype` says fp16; row stride ld, group stride gstride, in elements) as a TMA map
// with 64-feature x 64-row boxes and the 128-byte swizzle.
int32_t make_map(CUtensorMap *map, const void *base, int64_t features, int64_t rows, int64_t groups, int64_t ld,
                 int64_t gstride, CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16)
{
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(features), static_cast<cuuint64_t>(rows),
                          static_cast<cuuint64_t>(groups)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(ld) * 2, static_cast<cuuint64_t>(gstride) * 2};
    cuuint32_t box[3] = {gq::BOX_FEATURES, gq::TILE_K, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, dtype, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = static_cast<int32_t>(cudaErrorInvalidValue);
        return GQ_ERR_CUDA;
    }
    return GQ_OK;
}

// fp32 tensor [groups][d][d] as a TMA map with 32 x 32 boxes and the 128-byte swizzle (reduce-add target).
int32_t make_map_h(CUtensorMap *map, float *H, int64_t d, int64_t groups)
{
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(groups)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 4, static_cast<cuuint64_t>(d) * static_cast<cuuint64_t>(d) * 4};
    cuuint32_t box[3] = {32, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, H, dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = static_cast<int32_t>(cudaErrorInvalidValue);
        return GQ_ERR_CUDA;
    }
    return GQ_OK;
}

int grid_for(long long work_items, int threads, int sm_count, int blocks_per_sm)
{
    long long blocks = (work_items + threads - 1) / threads;
    const long long cap = static_cast<long long>(sm_count) * blocks_per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return static_cast<int>(blocks);
}

// Number of 256 x 256 tiles that touch the upper triangle of a d x d matrix.
int tiles_for(int64_t d)
{
    const int64_t nj = (d + gq::TILE_N - 1) / gq::TILE_N;
    return static_cast<int>(nj * (nj + 1) / 2);
}

// Edge of the super-blocks of the tile order: the pairs that run at the same time (pairs / units per tile
// of them work on distinct tiles) should cover a roughly square patch of tiles.
int raster_for(int pairs, int units_per_tile)
{
    int tiles_at_once = pairs / units_per_tile;
    if (tiles_at_once < 1) tiles_at_once = 1;
    int r = 1;
    while ((r + 1) * (r + 1) <= tiles_at_once) ++r;
    return r;
}

// Number of (row block, pair of neighbouring column blocks) slots that touch the upper triangle.
int colpair_slots_for(int64_t d)
{
    const int64_t nj = (d + gq::TILE_N - 1) / gq::TILE_N;
    const int64_t q = nj / 2;                     // complete column pairs: pair q' has 2 q' + 2 row blocks
    return static_cast<int>(q * (q + 1) + ((nj & 1) ? nj : 0));
}

int32_t check_layer_shape(int64_t d_in, int64_t d_out, int32_t g, bool need_out)
{
    if (g < 1 || d_in < 1) return GQ_ERR_INVALID_ARG;
    if (d_in % 8 != 0 || d_in < 8 || d_in > 65536 || g > 1024) return GQ_ERR_UNSUPPORTED_SHAPE;
    if (need_out) {
        if (d_out < 1 || d_out % g != 0) return GQ_ERR_INVALID_ARG;
        if ((d_out / g) % 8 != 0 || d_out > (1ll << 24)) return GQ_ERR_UNSUPPORTED_SHAPE;
    }
    return GQ_OK;
}

struct ByteRange {
    const void *p;
    size_t bytes;
};
// No written range may share a byte with a read-only range or with another written range.
template <int NW, int NR>
int32_t check_disjoint(const ByteRange (&written)[NW], const ByteRange (&read_only)[NR])
{
    for (int a = 0; a < NW; ++a) {
        for (int b = 0; b < NR; ++b)
            if (overlaps(written[a].p, written[a].bytes, read_only[b].p, read_only[b].bytes)) return GQ_ERR_INVALID_ARG;
        for (int b = a + 1; b < NW; ++b)
            if (overlaps(written[a].p, written[a].bytes, written[b].p, written[b].bytes)) return GQ_ERR_INVALID_ARG;
    }
    return GQ_OK;
}

// gq_objective / gq_objective_noalloc: the outputs (loss, scratch) must not share memory with W, W_hat, H or each
// other (W and W_hat may be the same buffer: both are only read).
int32_t check_objective_aliasing(const float *W, const float *W_hat, int64_t d_in, int64_t d_out, const float *H, int32_t g,
                                 const double *loss_out, const void *workspace, size_t ws_bytes)
{
    const size_t w_bytes = static_cast<size_t>(d_out) * d_in * 4, h_bytes = static_cast<size_t>(g) * d_in * d_in * 4;
    const size_t l_bytes = static_cast<size_t>(g + 1) * 8;
    const void *outs[2] = {loss_out, workspace};
    const size_t out_bytes[2] = {l_bytes, ws_bytes};
    for (int o = 0; o < 2; ++o)
        if (overlaps(outs[o], out_bytes[o], W, w_bytes) || overlaps(outs[o], out_bytes[o], W_hat, w_bytes) ||
            overlaps(outs[o], out_bytes[o], H, h_bytes))
            return GQ_ERR_INVALID_ARG;
    if (overlaps(loss_out, l_bytes, workspace, ws_bytes)) return GQ_ERR_INVALID_ARG;
    return GQ_OK;
}

// Scratch of gq_hessian_accumulate: the split saliency words, 8 bytes per (pair of groups, token).
size_t hessian_ws_bytes(int64_t n_max, int64_t, int32_t g)
{
    return round_up(static_cast<size_t>((g + 1) / 2) * static_cast<size_t>(n_max) * 8, 1024);
}

struct ObjectiveLayout {
    size_t header_off, half_off, partials_off, total;
};
// Scratch of gq_objective: a 1 KiB header (largest |delta| and the chosen power-of-two scale), delta as one fp16
// matrix, and one fp64 partial sum per (work unit, CTA of the pair, epilogue warp).
ObjectiveLayout objective_layout(int64_t d_in, int64_t d_out, int32_t g)
{
    ObjectiveLayout L;
    L.header_off = 0;
    L.half_off = 1024;
    L.partials_off = L.half_off + round_up(static_cast<size_t>(d_in) * static_cast<size_t>(d_out) * 2, 1024);
    L.total = L.partials_off +
              round_up(static_cast<size_t>(tiles_for(d_in)) * g * gq::GD_PARTIALS_PER_UNIT * sizeof(double), 1024);
    return L;
}

struct CodebookLayout {
    size_t h0, h1, w0, w1, qt, hw, pm, hp, gmat, rvec, total;
    int64_t slab_channels, slab_ld;
};
CodebookLayout codebook_layout(int64_t d_in, int64_t d_out, int32_t g, int32_t m)
{
    CodebookLayout L;
    const int64_t mk = d_out / g;
    L.slab_channels = mk < gq::CB_SLAB_CHANNELS ? mk : gq::CB_SLAB_CHANNELS;
    L.slab_ld = (L.slab_channels * m + 7) / 8 * 8;
    const size_t h2 = round_up(static_cast<size_t>(g) * d_in * d_in * 2, 1024);
    const size_t w2 = round_up(static_cast<size_t>(d_in) * d_out * 2, 1024);
    size_t o = 0;
    L.h0 = o; o += h2;
    L.h1 = o; o += h2;
    L.w0 = o; o += w2;
    L.w1 = o; o += w2;
    L.qt = o; o += round_up(static_cast<size_t>(d_in) * d_out, 1024);
    L.hw = o; o += round_up(static_cast<size_t>(d_in) * d_out * 4, 1024);
    L.pm = o; o += round_up(static_cast<size_t>(d_in) * L.slab_ld * 2, 1024);
    L.hp = o; o += round_up(static_cast<size_t>(d_in) * L.slab_ld * 4, 1024);
    L.gmat = o; o += round_up(static_cast<size_t>(d_out) * gq::CB_MAX_LEVELS * gq::CB_MAX_LEVELS * 8, 1024);
    L.rvec = o; o += round_up(static_cast<size_t>(d_out) * gq::CB_MAX_LEVELS * 8, 1024);
    L.total = o;
    return L;
}

struct CdLayout {
    size_t wt, wht, et, ehi, elo, hhi, hlo, rdiag, p, qt, total;
};
CdLayout cd_layout(int64_t d_in, int64_t d_out, int32_t g)
{
    CdLayout L;
    const size_t mat4 = round_up(static_cast<size_t>(d_in) * d_out * 4, 1024);
    const size_t mat2 = round_up(static_cast<size_t>(d_in) * d_out * 2, 1024);
    const size_t h2 = round_up(static_cast<size_t>(g) * d_in * d_in * 2, 1024);
    size_t o = 0;
    L.wt = o; o += mat4;
    L.wht = o; o += mat4;
    L.et = o; o += mat4;
    L.ehi = o; o += mat2;
    L.elo = o; o += mat2;
    L.hhi = o; o += h2;
    L.hlo = o; o += h2;
    L.rdiag = o; o += round_up(static_cast<size_t>(g) * d_in * 4, 1024);
    L.p = o; o += round_up(static_cast<size_t>(gq::CD_BLOCK) * d_out * 4, 1024);
    L.qt = o; o += round_up(static_cast<size_t>(d_in) * d_out, 1024);
    L.total = o;
    return L;
}

}  // namespace

extern "C" {

int gq_version(void) { return GQ_VERSION_NUMBER; }

const char *gq_status_string(int32_t status)
{
    switch (status) {
    case GQ_OK: return "GQ_OK";
    case GQ_ERR_INVALID_ARG: return "GQ_ERR_INVALID_ARG";
    case GQ_ERR_ALIGNMENT: return "GQ_ERR_ALIGNMENT";
    case GQ_ERR_UNSUPPORTED_SHAPE: return "GQ_ERR_UNSUPPORTED_SHAPE";
    case GQ_ERR_WORKSPACE: return "GQ_ERR_WORKSPACE";
    case GQ_ERR_CUDA: return "GQ_ERR_CUDA";
    case GQ_ERR_TIMEOUT: return "GQ_ERR_TIMEOUT";
    default: return "GQ_ERR_UNKNOWN";
    }
}

int32_t gq_last_cuda_error(void) { return tl_last_cuda_error; }

uint64_t gq_launch_count(void) { return g_launches.load(); }

// Argument checks of the saliency step (gq_saliency, gq_saliency_prepared and the saliency half of
// gq_hessian_accumulate_ahead).  GQ_OK with *empty = true means: nothing to do, pointers were not looked at.
static int32_t check_saliency_args(const void *grad, int64_t n, int64_t d_out, int64_t ld_grad, int32_t g, float grad_scale,
                                   const float *s, int64_t ld_s, bool prepare, const void *hessian_workspace,
                                   size_t workspace_bytes, bool *empty)
{
    *empty = false;
    if (n < 0 || g < 1 || d_out < 1 || d_out % g != 0 || ld_grad < d_out || ld_s < n ||
        !(grad_scale == grad_scale) || grad_scale - grad_scale != 0.0f)
        return GQ_ERR_INVALID_ARG;
    if ((d_out / g) % 8 != 0 || g > 1024 || d_out > (1ll << 24) || n * g >= (1ll << 31)) return GQ_ERR_UNSUPPORTED_SHAPE;
    if (ld_grad % 8 != 0) return GQ_ERR_ALIGNMENT;
    if (n == 0) {                          // nothing to read or write: pointers are not looked at
        *empty = true;
        return GQ_OK;
    }
    if (!grad || !s) return GQ_ERR_INVALID_ARG;
    if (!aligned(grad, 16) || !aligned(s, 4)) return GQ_ERR_ALIGNMENT;
    const size_t g_bytes = span_bytes(n, d_out, ld_grad, 2), s_bytes = span_bytes(g, n, ld_s, 4);
    if (overlaps(grad, g_bytes, s, s_bytes)) return GQ_ERR_INVALID_ARG;
    if (prepare) {
        const size_t ws_bytes = hessian_ws_bytes(n, 8, g);
        if (!hessian_workspace || workspace_bytes < ws_bytes) return GQ_ERR_WORKSPACE;
        if (!aligned(hessian_workspace, 1024)) return GQ_ERR_ALIGNMENT;
        if (overlaps(hessian_workspace, ws_bytes, grad, g_bytes) || overlaps(hessian_workspace, ws_bytes, s, s_bytes))
            return GQ_ERR_INVALID_ARG;
    }
    return GQ_OK;
}

static int32_t saliency_impl(const void *grad, int64_t n, int64_t d_out, int64_t ld_grad, int32_t g, float grad_scale,
                             float *s, int64_t ld_s, bool prepare, void *hessian_workspace, size_t workspace_bytes,
                             void *stream)
{
    bool empty;
    if (int32_t rc = check_saliency_args(grad, n, d_out, ld_grad, g, grad_scale, s, ld_s, prepare, hessian_workspace,
                                         workspace_bytes, &empty))
        return rc;
    if (empty) return GQ_OK;
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    const int m = static_cast<int>(d_out / g);
    const float coef = grad_scale * grad_scale / static_cast<float>(m);
    const unsigned grid = static_cast<unsigned>((n * g + 7) / 8);            // one warp per (token, group) segment
    {
        LaunchScope scope(GQ_KERNEL_SALIENCY, static_cast<cudaStream_t>(stream));
        gq::saliency_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const __nv_bfloat16 *>(grad), static_cast<unsigned>(n), m, ld_grad, g, coef, s, ld_s,
            prepare ? static_cast<uint32_t *>(hessian_workspace) : nullptr);
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

int32_t gq_saliency(const void *grad, int64_t n, int64_t d_out, int64_t ld_grad, int32_t g, float grad_scale,
                    float *s, int64_t ld_s, void *stream)
{
    return saliency_impl(grad, n, d_out, ld_grad, g, grad_scale, s, ld_s, false, nullptr, 0, stream);
}

int32_t gq_saliency_prepared(const void *grad, int64_t n, int64_t d_out, int64_t ld_grad, int32_t g, float grad_scale,
                             float *s, int64_t ld_s, void *hessian_workspace, size_t workspace_bytes, void *stream)
{
    return saliency_impl(grad, n, d_out, ld_grad, g, grad_scale, s, ld_s, true, hessian_workspace, workspace_bytes, stream);
}

int32_t gq_saliency_strided(const void *grad, int32_t dtype, int64_t batch, int64_t seq, int64_t d_out, int64_t stride_b,
                            int64_t stride_t, int32_t g, float grad_scale, float *s, int64_t ld_s, void *stream)
{
    if (batch < 0 || seq < 0 || g < 1 || d_out < 1 || d_out % g != 0 || stride_t < d_out || stride_b < 0 ||
        (dtype != GQ_DTYPE_BF16 && dtype != GQ_DTYPE_FP16 && dtype != GQ_DTYPE_FP32) ||
        !(grad_scale == grad_scale) || grad_scale - grad_scale != 0.0f)
        return GQ_ERR_INVALID_ARG;
    if (batch > (1ll << 31) || seq > (1ll << 31)) return GQ_ERR_UNSUPPORTED_SHAPE;
    const int64_t n = batch * seq;
    if (ld_s < n) return GQ_ERR_INVALID_ARG;
    if (batch > 1 && stride_b < (seq - 1) * stride_t + d_out) return GQ_ERR_INVALID_ARG;      // sequences overlap
    if ((d_out / g) % 8 != 0 || g > 1024 || d_out > (1ll << 24) || n * g >= (1ll << 31)) return GQ_ERR_UNSUPPORTED_SHAPE;
    const int64_t per16 = (dtype == GQ_DTYPE_FP32) ? 4 : 8;                    // elements per 16 bytes
    if (stride_t % per16 != 0 || stride_b % per16 != 0) return GQ_ERR_ALIGNMENT;
    if (n == 0) return GQ_OK;
    if (!grad || !s) return GQ_ERR_INVALID_ARG;
    if (!aligned(grad, 16) || !aligned(s, 4)) return GQ_ERR_ALIGNMENT;
    const size_t elem = (dtype == GQ_DTYPE_FP32) ? 4 : 2;
    const size_t g_bytes = (static_cast<size_t>(batch - 1) * stride_b + static_cast<size_t>(seq - 1) * stride_t + d_out) * elem;
    if (overlaps(grad, g_bytes, s, span_bytes(g, n, ld_s, 4))) return GQ_ERR_INVALID_ARG;
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    const int m = static_cast<int>(d_out / g);
    const float coef = grad_scale * grad_scale / static_cast<float>(m);
    const unsigned grid = static_cast<unsigned>((n * g + 7) / 8);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        LaunchScope scope(GQ_KERNEL_SALIENCY, st);
        if (dtype == GQ_DTYPE_BF16)
            gq::saliency_strided_kernel<gq::SAL_BF16><<<grid, 256, 0, st>>>(grad, static_cast<unsigned>(n), static_cast<unsigned>(seq), m,
                                                                         stride_b, stride_t, g, coef, s, ld_s);
        else if (dtype == GQ_DTYPE_FP16)
            gq::saliency_strided_kernel<gq::SAL_FP16><<<grid, 256, 0, st>>>(grad, static_cast<unsigned>(n), static_cast<unsigned>(seq), m,
                                                                         stride_b, stride_t, g, coef, s, ld_s);
        else
            gq::saliency_strided_kernel<gq::SAL_FP32><<<grid, 256, 0, st>>>(grad, static_cast<unsigned>(n), static_cast<unsigned>(seq), m,
                                                                         stride_b, stride_t, g, coef, s, ld_s);
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

size_t gq_hessian_workspace_bytes(int64_t n_max, int64_t d_in, int32_t g, uint32_t flags)
{
    if ((flags & ~static_cast<uint32_t>(GQ_HESSIAN_DETERMINISTIC | GQ_HESSIAN_S_PREPARED)) != 0 || n_max < 0 ||
        check_layer_shape(d_in, 0, g, false) != GQ_OK)
        return 0;
    return hessian_ws_bytes(n_max, d_in, g);
}

// Rate at which the two spare warps per CTA of a full guided-Hessian launch stream gradients (measured on B200).
#ifndef GQ_AHEAD_BYTES_PER_S
#define GQ_AHEAD_BYTES_PER_S 1.0e12
#endif

static int32_t hessian_accumulate_impl(const void *X, int64_t n, int64_t d_in, int64_t ld_x, const float *s, int64_t ld_s,
                                       int32_t g, float *H, uint32_t flags, void *workspace, size_t workspace_bytes,
                                       const gq::SaliencyAhead *ahead, void *stream)
{
    if (n < 0 || ld_x < d_in || ld_s < n ||
        (flags & ~static_cast<uint32_t>(GQ_HESSIAN_DETERMINISTIC | GQ_HESSIAN_S_PREPARED)) != 0)
        return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, 0, g, false)) return rc;
    if (n > (1ll << 31) - 64) return GQ_ERR_UNSUPPORTED_SHAPE;
    if (ld_x % 8 != 0) return GQ_ERR_ALIGNMENT;
    if (n == 0) return GQ_OK;              // an empty chunk adds nothing: pointers are not looked at
    if (!X || !s || !H) return GQ_ERR_INVALID_ARG;
    if (!aligned(X, 16) || !aligned(H, 128) || !aligned(s, 4)) return GQ_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < hessian_ws_bytes(n, d_in, g)) return GQ_ERR_WORKSPACE;
    if (!aligned(workspace, 1024)) return GQ_ERR_ALIGNMENT;
    {
        // the output and the scratch must not share memory with an input or with each other
        const size_t h_bytes = static_cast<size_t>(g) * d_in * d_in * 4, ws_bytes = hessian_ws_bytes(n, d_in, g);
        const size_t x_bytes = span_bytes(n, d_in, ld_x, 2), s_bytes = span_bytes(g, n, ld_s, 4);
        if (overlaps(H, h_bytes, X, x_bytes) || overlaps(H, h_bytes, s, s_bytes) || overlaps(H, h_bytes, workspace, ws_bytes) ||
            overlaps(workspace, ws_bytes, X, x_bytes) || overlaps(workspace, ws_bytes, s, s_bytes))
            return GQ_ERR_INVALID_ARG;
    }
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CUtensorMap mapX, mapH;
    if (int32_t rc = make_map(&mapX, X, d_in, n, 1, ld_x, n * ld_x)) return rc;
    if (int32_t rc = make_map_h(&mapH, H, d_in, g)) return rc;
    if ((flags & GQ_HESSIAN_S_PREPARED) == 0) {
        const int grid_s = grid_for(static_cast<long long>((g + 1) / 2) * n, 256, di->sm_count, 4);
        {
            LaunchScope scope(GQ_KERNEL_SPLIT_SALIENCY, st);
            gq::split_saliency_kernel<<<grid_s, 256, 0, st>>>(s, ld_s, static_cast<int>(n), g,
                                                             static_cast<uint2 *>(workspace));
        }
        GQ_CUDA(cudaGetLastError());
    }
    gq::HessianParams p{};
    p.X = static_cast<const __nv_bfloat16 *>(X);
    p.ld_x = ld_x;
    p.s2 = static_cast<const uint2 *>(workspace);
    p.n = static_cast<int>(n);
    p.d = static_cast<int>(d_in);
    p.g = g;
    p.nj = static_cast<int>((d_in + gq::TILE_N - 1) / gq::TILE_N);
    p.full_pairs = g / 2;
    p.raster = raster_for(di->max_pairs, p.full_pairs > 0 ? p.full_pairs : 1);
    p.narrow_units = tiles_for(d_in) * p.full_pairs;
    const int units = p.narrow_units + ((g & 1) ? colpair_slots_for(d_in) : 0);
    const int ksteps = static_cast<int>((n + gq::TILE_K - 1) / gq::TILE_K);
    const bool balanced = (flags & GQ_HESSIAN_DETERMINISTIC) == 0;
    int pairs = di->max_pairs;
    if (!balanced && units < pairs) pairs = units;
    p.sched = gq::plan_schedule(units, ksteps, pairs, balanced);
    p.status = di->status_ptr;
    p.wait_budget_ns = wait_budget_ns();
    const int grid = 2 * ((p.sched.full_waves == 0 && p.sched.tail_pairs > 0) ? p.sched.tail_pairs : pairs);
    if (ahead) {
        // Does the saliency step fit behind the Hessian step?  Measured on B200 with all 148 CTAs: the two spare
        // warps per CTA stream the gradient block at about 1.0e12 bytes/s while the tensor cores work through
        // 1.25e15 issued flop/s; both rates shrink with the number of CTAs of a small launch.  If the gradients
        // would take longer than 85 % of the Hessian work (plus 5 us, about what a launch of its own costs), the
        // launch would only get longer: the saliency step then runs as a kernel of its own.  (Leaving part of the
        // block to the spare warps and the rest to a kernel was measured too: no better than the kernel alone.)
        const double share = static_cast<double>(grid) / (2.0 * di->max_pairs);
        const double tiles = 2.0 * units;              // every unit fills (up to) two 256 x 256 accumulators
        const double t_hessian = 2.0 * gq::TILE_M * gq::TILE_N * (static_cast<double>(ksteps) * gq::TILE_K) * tiles / (1.25e15 * share);
        const double t_saliency = static_cast<double>(ahead->n) * ahead->m * g * 2.0 / (GQ_AHEAD_BYTES_PER_S * share);
        if (t_saliency <= 0.85 * t_hessian + 5e-6) {
            p.ahead = *ahead;
        } else {
            const unsigned grid_s = static_cast<unsigned>((static_cast<long long>(ahead->n) * g + 7) / 8);
            {
                LaunchScope scope(GQ_KERNEL_SALIENCY, st);
                gq::saliency_kernel<<<grid_s, 256, 0, st>>>(ahead->grad, ahead->n, ahead->m, ahead->ld_grad, g, ahead->coef,
                                                            ahead->s, ahead->ld_s, ahead->words);
            }
            GQ_CUDA(cudaGetLastError());
        }
    }
    {
        LaunchScope scope(GQ_KERNEL_HESSIAN, st);
        gq::hessian_kernel<<<grid, gq::HS_THREADS, gq::HS_SMEM_BYTES, st>>>(mapX, mapH, p);
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

int32_t gq_hessian_accumulate(const void *X, int64_t n, int64_t d_in, int64_t ld_x, const float *s, int64_t ld_s,
                              int32_t g, float *H, uint32_t flags, void *workspace, size_t workspace_bytes,
                              void *stream)
{
    return hessian_accumulate_impl(X, n, d_in, ld_x, s, ld_s, g, H, flags, workspace, workspace_bytes, nullptr, stream);
}

int32_t gq_hessian_accumulate_ahead(const void *X, int64_t n, int64_t d_in, int64_t ld_x, const float *s, int64_t ld_s,
                                    int32_t g, float *H, uint32_t flags, void *workspace, size_t workspace_bytes,
                                    const void *next_grad, int64_t next_n, int64_t d_out, int64_t ld_grad, float grad_scale,
                                    float *next_s, int64_t next_ld_s, void *next_workspace, size_t next_workspace_bytes,
                                    void *stream)
{
    bool empty;
    if (int32_t rc = check_saliency_args(next_grad, next_n, d_out, ld_grad, g, grad_scale, next_s, next_ld_s, true,
                                         next_workspace, next_workspace_bytes, &empty))
        return rc;
    if (empty)
        return hessian_accumulate_impl(X, n, d_in, ld_x, s, ld_s, g, H, flags, workspace, workspace_bytes, nullptr, stream);
    if (n <= 0) {
        // no Hessian work to hide behind: check the rest of the call as gq_hessian_accumulate would, then run the
        // saliency step as a launch of its own
        if (int32_t rc = hessian_accumulate_impl(X, n, d_in, ld_x, s, ld_s, g, H, flags, workspace, workspace_bytes, nullptr, stream))
            return rc;
        return saliency_impl(next_grad, next_n, d_out, ld_grad, g, grad_scale, next_s, next_ld_s, true, next_workspace,
                             next_workspace_bytes, stream);
    }
    if (!X || !s || !H || !workspace || d_in < 1 || ld_x < d_in || ld_s < n) return GQ_ERR_INVALID_ARG;
    {
        // what the look-ahead writes must not share memory with anything the Hessian step reads or writes, and
        // what it reads must not be written by the Hessian step
        const size_t h_bytes = static_cast<size_t>(g) * d_in * d_in * 4, ws_bytes = hessian_ws_bytes(n, d_in, g);
        const size_t x_bytes = span_bytes(n, d_in, ld_x, 2), s_bytes = span_bytes(g, n, ld_s, 4);
        const size_t ng_bytes = span_bytes(next_n, d_out, ld_grad, 2), ns_bytes = span_bytes(g, next_n, next_ld_s, 4);
        const size_t nws_bytes = hessian_ws_bytes(next_n, 8, g);
        const void *outs[2] = {next_s, next_workspace};
        const size_t out_bytes[2] = {ns_bytes, nws_bytes};
        for (int o = 0; o < 2; ++o)
            if (overlaps(outs[o], out_bytes[o], H, h_bytes) || overlaps(outs[o], out_bytes[o], X, x_bytes) ||
                overlaps(outs[o], out_bytes[o], workspace, ws_bytes))
                return GQ_ERR_INVALID_ARG;
        // s and next_s may be two column ranges of one [g, ld] buffer that holds the saliency of all chunks
        if (rows_overlap_f32(s, n, ld_s, next_s, next_n, next_ld_s, g) || overlaps(next_workspace, nws_bytes, s, s_bytes))
            return GQ_ERR_INVALID_ARG;
        if (overlaps(next_grad, ng_bytes, H, h_bytes) || overlaps(next_grad, ng_bytes, workspace, ws_bytes))
            return GQ_ERR_INVALID_ARG;
    }
    gq::SaliencyAhead a{};
    a.grad = static_cast<const __nv_bfloat16 *>(next_grad);
    a.n = static_cast<unsigned>(next_n);
    a.m = static_cast<int>(d_out / g);
    a.ld_grad = ld_grad;
    a.coef = grad_scale * grad_scale / static_cast<float>(a.m);
    a.s = next_s;
    a.ld_s = next_ld_s;
    a.words = static_cast<uint32_t *>(next_workspace);
    return hessian_accumulate_impl(X, n, d_in, ld_x, s, ld_s, g, H, flags, workspace, workspace_bytes, &a, stream);
}

int32_t gq_hessian_finalize(float *H, int64_t d_in, int32_t g, void *stream)
{
    if (!H) return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, 0, g, false)) return rc;
    if (!aligned(H, 128)) return GQ_ERR_ALIGNMENT;
    const unsigned nb = static_cast<unsigned>((d_in + 31) / 32);
    dim3 grid(nb, nb, static_cast<unsigned>(g));
    {
        LaunchScope scope(GQ_KERNEL_MIRROR, static_cast<cudaStream_t>(stream));
        gq::mirror_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(H, static_cast<int>(d_in));
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

static int32_t hessian_exchange(float *const *H_ranks, int32_t ranks, int32_t rank, int64_t d_in, int32_t g,
                                void *stream, bool reduce)
{
    if (!H_ranks || ranks < 1 || ranks > gq::EX_MAX_RANKS || rank < 0 || rank >= ranks) return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, 0, g, false)) return rc;
    gq::ExchangeParams p{};
    for (int32_t r = 0; r < ranks; ++r) {
        if (!H_ranks[r]) return GQ_ERR_INVALID_ARG;
        if (!aligned(H_ranks[r], 16)) return GQ_ERR_ALIGNMENT;
        p.H[r] = H_ranks[r];
    }
    if (ranks == 1) return GQ_OK;
    p.ranks = ranks;
    p.rank = rank;
    p.d = static_cast<int>(d_in);
    p.g = g;
    p.nb = static_cast<int>((d_in + gq::EX_BLOCK - 1) / gq::EX_BLOCK);
    p.blocks = static_cast<long long>(g) * p.nb * (p.nb + 1) / 2;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    long long first = 0, count = p.blocks;
    if (reduce) {
        first = gq::exchange_share_begin(p.blocks, ranks, rank);
        count = gq::exchange_share_begin(p.blocks, ranks, rank + 1) - first;
    }
    if (count <= 0) return GQ_OK;
    {
        LaunchScope scope(GQ_KERNEL_EXCHANGE, st);
        if (reduce)
            gq::exchange_kernel<true><<<static_cast<unsigned>(count), 256, 0, st>>>(p, first);
        else
            gq::exchange_kernel<false><<<static_cast<unsigned>(count), 256, 0, st>>>(p, first);
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

int32_t gq_hessian_reduce_share(float *const *H_ranks, int32_t ranks, int32_t rank, int64_t d_in, int32_t g, void *stream)
{
    return hessian_exchange(H_ranks, ranks, rank, d_in, g, stream, true);
}

int32_t gq_hessian_gather_shares(float *const *H_ranks, int32_t ranks, int32_t rank, int64_t d_in, int32_t g, void *stream)
{
    return hessian_exchange(H_ranks, ranks, rank, d_in, g, stream, false);
}

size_t gq_objective_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g)
{
    if (check_layer_shape(d_in, d_out, g, true) != GQ_OK || d_in * d_out >= (1ll << 33)) return 0;
    return objective_layout(d_in, d_out, g).total;
}

int32_t gq_objective(const float *W, const float *W_hat, int64_t d_in, int64_t d_out, const float *H, int32_t g,
                     double *loss_out, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!W || !W_hat || !H || !loss_out) return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, d_out, g, true)) return rc;
    if (d_in * d_out >= (1ll << 33)) return GQ_ERR_UNSUPPORTED_SHAPE;      // 32-bit element indices in the preparation
    if (!aligned(W, 16) || !aligned(W_hat, 16) || !aligned(H, 128) || !aligned(loss_out, 8)) return GQ_ERR_ALIGNMENT;
    const ObjectiveLayout L = objective_layout(d_in, d_out, g);
    if (!workspace || workspace_bytes < L.total) return GQ_ERR_WORKSPACE;
    if (!aligned(workspace, 1024)) return GQ_ERR_ALIGNMENT;
    if (int32_t rc = check_objective_aliasing(W, W_hat, d_in, d_out, H, g, loss_out, workspace, L.total)) return rc;
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    gq::GramDotHeader *header = reinterpret_cast<gq::GramDotHeader *>(ws + L.header_off);
    __half *dh = reinterpret_cast<__half *>(ws + L.half_off);
    double *partials = reinterpret_cast<double *>(ws + L.partials_off);
    const int64_t m = d_out / g;
    // delta = W - W_hat as one fp16 matrix scaled by a power of two taken from max |delta| (two passes over W, W_hat)
    GQ_CUDA(cudaMemsetAsync(header, 0, sizeof(gq::GramDotHeader), st));
    {
        const unsigned count4 = static_cast<unsigned>(d_in * d_out / 4);
        const unsigned per_block = 256u * gq::DELTA_VEC_PER_THREAD;
        const unsigned blocks = (count4 + per_block - 1) / per_block;
        {
            LaunchScope scope(GQ_KERNEL_SPLIT_DELTA, st);
            gq::delta_absmax_kernel<<<blocks, 256, 0, st>>>(W, W_hat, count4, header);
        }
        GQ_CUDA(cudaGetLastError());
        {
            LaunchScope scope(GQ_KERNEL_SPLIT_DELTA, st);
            gq::delta_half_kernel<<<blocks, 256, 0, st>>>(W, W_hat, count4, header, dh);
        }
        GQ_CUDA(cudaGetLastError());
    }
    CUtensorMap mapD;
    if (int32_t rc = make_map(&mapD, dh, d_in, m, g, d_in, m * d_in, CU_TENSOR_MAP_DATA_TYPE_FLOAT16)) return rc;
    gq::GramDotParams p{};
    p.d = static_cast<int>(d_in);
    p.rows = static_cast<int>(m);
    p.g = g;
    p.nj = static_cast<int>((d_in + gq::TILE_N - 1) / gq::TILE_N);
    // units: (256 x 256 tile on the upper triangle, group), group-major (gq_gram_dot.cuh)
    p.tiles = tiles_for(d_in);
    const int slots = p.tiles;
    const int units = slots * g;
    const int ksteps = static_cast<int>((m + gq::TILE_K - 1) / gq::TILE_K);
    const int pairs = units < di->max_pairs ? units : di->max_pairs;
    p.raster = raster_for(pairs, 1);
    p.sched = gq::plan_schedule(units, ksteps, pairs, false);
    p.H = H;
    p.partials = partials;
    p.status = di->status_ptr;
    p.wait_budget_ns = wait_budget_ns();
    {
        LaunchScope scope(GQ_KERNEL_GRAM_DOT, st);
        gq::gram_dot_kernel<<<2 * p.sched.pairs, gq::GD_THREADS, gq::GD_SMEM_BYTES, st>>>(mapD, p);
    }
    GQ_CUDA(cudaGetLastError());
    {
        LaunchScope scope(GQ_KERNEL_REDUCE, st);
        gq::gram_dot_reduce_kernel<<<static_cast<unsigned>(g), 256, 0, st>>>(partials, slots, g, gq::GD_PARTIALS_PER_UNIT, header, loss_out);
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

// ------------------------------------------------------------------------------------------------
// gq_objective_noalloc: the objective with its scratch in a fixed device array of this library.
// Limits (see include/gq.h): d_in * d_out <= 2^20 weights, (256 x 256 tiles) * g <= 4096 work units.
#define GQ_NOALLOC_MAX_WEIGHTS (1ll << 20)
#define GQ_NOALLOC_MAX_UNITS 4096ll
#define GQ_NOALLOC_MATRIX_BYTES (GQ_NOALLOC_MAX_WEIGHTS * 2)                 /* one bf16 copy of delta */
#define GQ_NOALLOC_PARTIAL_BYTES (GQ_NOALLOC_MAX_UNITS * 8 * 8)              /* 8 fp64 sums per unit   */
#define GQ_NOALLOC_SCRATCH_BYTES (2 * GQ_NOALLOC_MATRIX_BYTES + GQ_NOALLOC_PARTIAL_BYTES)

}  // extern "C"

namespace {
// Lives in every CUDA context that loads the library, from load until exit: 4 MiB + 256 KiB.
static __device__ __align__(256) unsigned char g_noalloc_scratch[GQ_NOALLOC_SCRATCH_BYTES];
// Device address of g_noalloc_scratch per device, looked up once (the name above is only a handle
// on the host side and must never be passed to a kernel as if it were an address).
unsigned char *g_noalloc_scratch_ptr[kMaxDevices];
std::mutex g_noalloc_mutex;
}  // namespace

extern "C" {

int32_t gq_objective_noalloc(const float *W, const float *W_hat, int64_t d_in, int64_t d_out, const float *H,
                             int32_t g, double *loss_out, void *stream)
{
    if (!W || !W_hat || !H || !loss_out) return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, d_out, g, true)) return rc;
    if (!aligned(W, 16) || !aligned(W_hat, 16) || !aligned(H, 16) || !aligned(loss_out, 8)) return GQ_ERR_ALIGNMENT;
    const int tiles = tiles_for(d_in);
    if (d_in * d_out > GQ_NOALLOC_MAX_WEIGHTS || static_cast<int64_t>(tiles) * g > GQ_NOALLOC_MAX_UNITS)
        return GQ_ERR_UNSUPPORTED_SHAPE;       // larger layers must use gq_objective with a caller workspace
    if (int32_t rc = check_objective_aliasing(W, W_hat, d_in, d_out, H, g, loss_out, nullptr, 0)) return rc;
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;

    // One-time set-up per device (with that device current): ask the runtime where the array lives.
    int dev = 0;
    GQ_CUDA(cudaGetDevice(&dev));
    unsigned char *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_scratch_ptr[dev]) {
            unsigned char *ptr = nullptr;
            GQ_CUDA(cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_scratch));
            if (!ptr) {
                tl_last_cuda_error = static_cast<int32_t>(cudaErrorInvalidSymbol);
                return GQ_ERR_CUDA;
            }
            g_noalloc_scratch_ptr[dev] = ptr;
        }
        scratch = g_noalloc_scratch_ptr[dev];
    }

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    __nv_bfloat16 *hi = reinterpret_cast<__nv_bfloat16 *>(scratch);
    __nv_bfloat16 *lo = reinterpret_cast<__nv_bfloat16 *>(scratch + GQ_NOALLOC_MATRIX_BYTES);
    double *partials = reinterpret_cast<double *>(scratch + 2 * GQ_NOALLOC_MATRIX_BYTES);
    const int64_t m = d_out / g;
    // Every scratch byte that is read below is written first by this same call (hi/lo by the split
    // kernel, one partial per (unit, CTA, warp) by the objective kernel), so what an earlier call left behind
    // is never observed and nothing has to be cleared.
    {
        const long long count8 = d_in * d_out / 8;
        const int grid = grid_for(count8, 256, di->sm_count, 8);
        gq::split_delta_kernel<<<grid, 256, 0, st>>>(W, W_hat, count8, hi, lo);
        g_launches.fetch_add(1);
        GQ_CUDA(cudaGetLastError());
    }
    CUtensorMap mapHi, mapLo;
    if (int32_t rc = make_map(&mapHi, hi, d_in, m, g, d_in, m * d_in)) return rc;
    if (int32_t rc = make_map(&mapLo, lo, d_in, m, g, d_in, m * d_in)) return rc;
    gq::PairGemmParams p{};
    p.d = static_cast<int>(d_in);
    p.rows = static_cast<int>(m);
    p.g = g;
    p.n_terms = 3;
    p.nj = static_cast<int>((d_in + gq::TILE_N - 1) / gq::TILE_N);
    p.raster = raster_for(di->max_pairs, g);
    p.term_a[0] = 0; p.term_b[0] = 0;
    p.term_a[1] = 0; p.term_b[1] = 1;
    p.term_a[2] = 1; p.term_b[2] = 0;
    p.map_grouped[0] = 1;
    p.map_grouped[1] = 1;
    const int units = tiles * g;
    const int ksteps = 3 * static_cast<int>((m + gq::TILE_K - 1) / gq::TILE_K);
    p.sched = gq::plan_schedule(units, ksteps, units < di->max_pairs ? units : di->max_pairs, false);
    p.H = H;
    p.partials = partials;
    p.status = di->status_ptr;
    p.wait_budget_ns = wait_budget_ns();
    const int grid = 2 * p.sched.pairs;
    gq::pair_gemm_kernel<gq::MODE_OBJECTIVE><<<grid, gq::OBJ_THREADS, gq::OBJ_SMEM_BYTES, st>>>(mapHi, mapLo, mapHi, mapLo, mapHi,
                                                                                               mapLo, p);
    g_launches.fetch_add(1);
    GQ_CUDA(cudaGetLastError());
    gq::reduce_partials_kernel<<<1, 1024, 0, st>>>(partials, tiles, g, gq::PARTIALS_PER_UNIT, loss_out);
    g_launches.fetch_add(1);
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

size_t gq_cd_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g)
{
    if (check_layer_shape(d_in, d_out, g, true) != GQ_OK) return 0;
    return cd_layout(d_in, d_out, g).total;
}

int32_t gq_cd_cycles(const float *W, float *W_hat, uint8_t *Q, const float *codebook, int32_t m, int64_t d_in,
                     int64_t d_out, const float *H, int32_t g, int32_t cycles, void *workspace,
                     size_t workspace_bytes, void *stream)
{
    if (!W || !W_hat || !Q || !codebook || !H || cycles < 0 || m < 1) return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, d_out, g, true)) return rc;
    if (m > gq::CD_MAX_LEVELS) return GQ_ERR_UNSUPPORTED_SHAPE;
    if (!aligned(W, 16) || !aligned(W_hat, 16) || !aligned(H, 16) || !aligned(codebook, 4)) return GQ_ERR_ALIGNMENT;
    const CdLayout L = cd_layout(d_in, d_out, g);
    if (!workspace || workspace_bytes < L.total) return GQ_ERR_WORKSPACE;
    if (!aligned(workspace, 1024)) return GQ_ERR_ALIGNMENT;
    {
        const size_t w4 = static_cast<size_t>(d_out) * d_in * 4;
        const ByteRange wr[3] = {{W_hat, w4}, {Q, static_cast<size_t>(d_out) * d_in}, {workspace, L.total}};
        const ByteRange ro[3] = {{W, w4}, {codebook, static_cast<size_t>(d_out) * m * 4},
                                 {H, static_cast<size_t>(g) * d_in * d_in * 4}};
        if (int32_t rc = check_disjoint(wr, ro)) return rc;
    }
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    float *Wt = reinterpret_cast<float *>(ws + L.wt);
    float *Wht = reinterpret_cast<float *>(ws + L.wht);
    float *Et = reinterpret_cast<float *>(ws + L.et);
    __nv_bfloat16 *Ehi = reinterpret_cast<__nv_bfloat16 *>(ws + L.ehi);
    __nv_bfloat16 *Elo = reinterpret_cast<__nv_bfloat16 *>(ws + L.elo);
    __nv_bfloat16 *Hhi = reinterpret_cast<__nv_bfloat16 *>(ws + L.hhi);
    __nv_bfloat16 *Hlo = reinterpret_cast<__nv_bfloat16 *>(ws + L.hlo);
    float *rdiag = reinterpret_cast<float *>(ws + L.rdiag);
    float *P = reinterpret_cast<float *>(ws + L.p);
    uint8_t *Qt = ws + L.qt;
    const int64_t mk = d_out / g;
    const dim3 tgrid(static_cast<unsigned>((d_in + 31) / 32), static_cast<unsigned>((d_out + 31) / 32));
    {
        LaunchScope scope(GQ_KERNEL_CD_AUX, st);
        gq::cd_prepare_kernel<<<tgrid, 256, 0, st>>>(W, W_hat, static_cast<int>(d_in), static_cast<int>(d_out), Wt, Wht,
                                                     Et, Ehi, Elo);
    }
    GQ_CUDA(cudaGetLastError());
    {
        const long long count = static_cast<long long>(g) * d_in * d_in;
        LaunchScope scope(GQ_KERNEL_CD_AUX, st);
        gq::cd_split_h_kernel<<<grid_for(count, 256, di->sm_count, 8), 256, 0, st>>>(H, count, static_cast<int>(d_in), Hhi,
                                                                                 Hlo, rdiag);
    }
    GQ_CUDA(cudaGetLastError());

    CUtensorMap mapHhi, mapHlo, mapEhi, mapElo;
    if (int32_t rc = make_map(&mapHhi, Hhi, d_in, d_in, g, d_in, d_in * d_in)) return rc;
    if (int32_t rc = make_map(&mapHlo, Hlo, d_in, d_in, g, d_in, d_in * d_in)) return rc;
    if (int32_t rc = make_map(&mapEhi, Ehi, d_out, d_in, 1, d_out, d_in * d_out)) return rc;
    if (int32_t rc = make_map(&mapElo, Elo, d_out, d_in, 1, d_out, d_in * d_out)) return rc;
    const int kblocks = static_cast<int>((d_in + gq::TILE_K - 1) / gq::TILE_K);
    const int ch_tiles = static_cast<int>((mk + gq::TILE_N - 1) / gq::TILE_N);
    const int slices = static_cast<int>((mk + gq::CD_CH - 1) / gq::CD_CH);

    for (int32_t cyc = 0; cyc < cycles; ++cyc) {
        for (int64_t s0 = 0; s0 < d_in; s0 += gq::CD_BLOCK) {
            const int rows = static_cast<int>(d_in - s0 < gq::CD_BLOCK ? d_in - s0 : gq::CD_BLOCK);
            const int blk_ksteps = (rows + gq::TILE_K - 1) / gq::TILE_K;
            const int nk = kblocks - blk_ksteps;
            GQ_CUDA(cudaMemsetAsync(P, 0, static_cast<size_t>(gq::CD_BLOCK) * d_out * sizeof(float), st));
            if (nk > 0) {
                gq::PairGemmParams pp{};
                pp.d = static_cast<int>(d_in);
                pp.g = g;
                pp.n_terms = 3;                    // Hhi Ehi + Hhi Elo + Hlo Ehi
                pp.term_a[0] = 0; pp.term_b[0] = 2;
                pp.term_a[1] = 0; pp.term_b[1] = 3;
                pp.term_a[2] = 1; pp.term_b[2] = 2;
                pp.map_grouped[0] = 1; pp.map_grouped[1] = 1; pp.map_grouped[2] = 0; pp.map_grouped[3] = 0;
                pp.s0 = static_cast<int>(s0);
                pp.blk_ksteps = blk_ksteps;
                pp.nk = nk;
                pp.ch_tiles = ch_tiles;
                pp.mk = static_cast<int>(mk);
                pp.d_out = static_cast<int>(d_out);
                pp.P = P;
                const int tiles = g * ch_tiles;
                int pieces = di->max_pairs / tiles;              // cut the contraction so that every pair has work
                if (pieces < 1) pieces = 1;
                if (pieces > 3 * nk) pieces = 3 * nk;
                pp.pieces = pieces;
                const int ksteps = (3 * nk + pieces - 1) / pieces;
                const int units = tiles * pieces;
                pp.sched = gq::plan_schedule(units, ksteps, units < di->max_pairs ? units : di->max_pairs, false);
                pp.status = di->status_ptr;
                pp.wait_budget_ns = wait_budget_ns();
                {
                    LaunchScope scope(GQ_KERNEL_CD_PANEL, st);
                    gq::pair_gemm_kernel<gq::MODE_PANEL><<<2 * pp.sched.pairs, gq::OBJ_THREADS, gq::OBJ_SMEM_BYTES, st>>>(
                        mapHhi, mapHlo, mapEhi, mapElo, mapEhi, mapElo, pp);
                }
                GQ_CUDA(cudaGetLastError());
            }
            gq::CdBlockParams bp{};
            bp.H = H; bp.rdiag = rdiag; bp.P = P; bp.Wt = Wt; bp.codebook = codebook; bp.Wht = Wht; bp.Et = Et;
            bp.Ehi = Ehi; bp.Elo = Elo; bp.Qt = Qt;
            bp.d_in = static_cast<int>(d_in); bp.d_out = static_cast<int>(d_out); bp.g = g; bp.mk = static_cast<int>(mk);
            bp.m = m; bp.s0 = static_cast<int>(s0); bp.rows = rows; bp.slices = slices;
            {
                LaunchScope scope(GQ_KERNEL_CD_BLOCK, st);
                gq::cd_block_kernel<<<g * slices, gq::CD_THREADS, gq::CD_SMEM_BYTES, st>>>(bp);
            }
            GQ_CUDA(cudaGetLastError());
        }
    }
    {
        LaunchScope scope(GQ_KERNEL_CD_AUX, st);
        gq::cd_finish_kernel<<<tgrid, 256, 0, st>>>(Wht, Qt, static_cast<int>(d_in), static_cast<int>(d_out), W_hat, Q);
    }
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

size_t gq_codebook_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g, int32_t m)
{
    if (m < 1 || m > gq::CB_MAX_LEVELS || check_layer_shape(d_in, d_out, g, true) != GQ_OK) return 0;
    return codebook_layout(d_in, d_out, g, m).total;
}

int32_t gq_codebook_update(const float *W, const uint8_t *Q, int32_t m, int64_t d_in, int64_t d_out, const float *H,
                           int32_t g, double lambda, float *codebook, float *W_hat, void *workspace,
                           size_t workspace_bytes, void *stream)
{
    if (!W || !Q || !H || !codebook || m < 1 || !(lambda >= 0.0)) return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, d_out, g, true)) return rc;
    if (m > gq::CB_MAX_LEVELS) return GQ_ERR_UNSUPPORTED_SHAPE;
    if (!aligned(W, 16) || !aligned(H, 16) || !aligned(codebook, 4) || (W_hat && !aligned(W_hat, 16))) return GQ_ERR_ALIGNMENT;
    const CodebookLayout L = codebook_layout(d_in, d_out, g, m);
    if (!workspace || workspace_bytes < L.total) return GQ_ERR_WORKSPACE;
    if (!aligned(workspace, 1024)) return GQ_ERR_ALIGNMENT;
    {
        const size_t w4 = static_cast<size_t>(d_out) * d_in * 4;
        const ByteRange wr[3] = {{codebook, static_cast<size_t>(d_out) * m * 4}, {W_hat, W_hat ? w4 : 0}, {workspace, L.total}};
        const ByteRange ro[3] = {{W, w4}, {Q, static_cast<size_t>(d_out) * d_in}, {H, static_cast<size_t>(g) * d_in * d_in * 4}};
        if (int32_t rc = check_disjoint(wr, ro)) return rc;
    }
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    __nv_bfloat16 *H0 = reinterpret_cast<__nv_bfloat16 *>(ws + L.h0), *H1 = reinterpret_cast<__nv_bfloat16 *>(ws + L.h1);
    __nv_bfloat16 *W0 = reinterpret_cast<__nv_bfloat16 *>(ws + L.w0), *W1 = reinterpret_cast<__nv_bfloat16 *>(ws + L.w1);
    uint8_t *Qt = ws + L.qt;
    float *HW = reinterpret_cast<float *>(ws + L.hw);
    __nv_bfloat16 *Pm = reinterpret_cast<__nv_bfloat16 *>(ws + L.pm);
    float *HP = reinterpret_cast<float *>(ws + L.hp);
    double *Gm = reinterpret_cast<double *>(ws + L.gmat);
    double *Rv = reinterpret_cast<double *>(ws + L.rvec);
    const int64_t mk = d_out / g;
    const long long hcount = static_cast<long long>(g) * d_in * d_in;
    {
        LaunchScope scope(GQ_KERNEL_CB_AUX, st);
        gq::cb_split2_kernel<<<grid_for(hcount, 256, di->sm_count, 8), 256, 0, st>>>(H, hcount, H0, H1);
    }
    GQ_CUDA(cudaGetLastError());
    {
        const dim3 tgrid(static_cast<unsigned>((d_in + 31) / 32), static_cast<unsigned>((d_out + 31) / 32));
        LaunchScope scope(GQ_KERNEL_CB_AUX, st);
        gq::cb_transpose_kernel<<<tgrid, 256, 0, st>>>(W, Q, static_cast<int>(d_in), static_cast<int>(d_out), W0, W1, Qt);
    }
    GQ_CUDA(cudaGetLastError());
    CUtensorMap mH0, mH1, mW0, mW1, mPm;
    if (int32_t rc = make_map(&mH0, H0, d_in, d_in, g, d_in, d_in * d_in)) return rc;
    if (int32_t rc = make_map(&mH1, H1, d_in, d_in, g, d_in, d_in * d_in)) return rc;
    if (int32_t rc = make_map(&mW0, W0, d_out, d_in, 1, d_out, d_in * d_out)) return rc;
    if (int32_t rc = make_map(&mW1, W1, d_out, d_in, 1, d_out, d_in * d_out)) return rc;
    if (int32_t rc = make_map(&mPm, Pm, L.slab_ld, d_in, 1, L.slab_ld, d_in * L.slab_ld)) return rc;

    auto launch_full = [&](gq::PairGemmParams &pp, const CUtensorMap &b0, const CUtensorMap &b1, const CUtensorMap &b2,
                           int kernel_id, bool wide) -> int32_t {
        pp.d = static_cast<int>(d_in);
        pp.rows = static_cast<int>(d_in);
        pp.g = g;
        pp.map_grouped[0] = pp.map_grouped[1] = pp.map_grouped[2] = 1;
        pp.map_grouped[3] = pp.map_grouped[4] = pp.map_grouped[5] = 0;
        pp.col_tiles = (pp.cols + gq::TILE_N - 1) / gq::TILE_N;
        const int row_blocks = static_cast<int>((d_in + gq::TILE_M - 1) / gq::TILE_M);
        // wide: a unit is a row block times two neighbouring column tiles (gq_wide_gemm.cuh)
        const int units = row_blocks * (wide ? (pp.col_tiles + 1) / 2 : pp.col_tiles);
        const int ksteps = pp.n_terms * static_cast<int>((d_in + gq::TILE_K - 1) / gq::TILE_K);
        pp.sched = gq::plan_schedule(units, ksteps, units < di->max_pairs ? units : di->max_pairs, false);
        pp.status = di->status_ptr;
        pp.wait_budget_ns = wait_budget_ns();
        {
            LaunchScope scope(kernel_id, st);
            if (wide)
                gq::wide_gemm_kernel<gq::WG_FULL><<<2 * pp.sched.pairs, gq::WG_THREADS, gq::WG_SMEM_BYTES, st>>>(mH0, mH1, mH1, b0, b1, b2, pp);
            else
                gq::pair_gemm_kernel<gq::MODE_FULL><<<2 * pp.sched.pairs, gq::OBJ_THREADS, gq::OBJ_SMEM_BYTES, st>>>(
                    mH0, mH1, mH1, b0, b1, b2, pp);
        }
        GQ_CUDA(cudaGetLastError());
        return GQ_OK;
    };

    GQ_CUDA(cudaMemsetAsync(Gm, 0, static_cast<size_t>(d_out) * gq::CB_MAX_LEVELS * gq::CB_MAX_LEVELS * sizeof(double), st));
    GQ_CUDA(cudaMemsetAsync(Rv, 0, static_cast<size_t>(d_out) * gq::CB_MAX_LEVELS * sizeof(double), st));
    for (int32_t k = 0; k < g; ++k) {
        // HW[:, group k] = H_k W_k^T: H0 W0 + H0 W1 + H1 W0 (hi + lo splits, 16 significant bits per factor)
        gq::PairGemmParams pp{};
        pp.n_terms = 3;
        const int ta[3] = {0, 0, 1}, tb[3] = {3, 4, 3};
        for (int t = 0; t < 3; ++t) { pp.term_a[t] = ta[t]; pp.term_b[t] = tb[t]; }
        pp.full_k = k;
        pp.col0 = static_cast<int>(k * mk);
        pp.cols = static_cast<int>(mk);
        pp.C = HW + k * mk;
        pp.ldc = d_out;
        if (int32_t rc = launch_full(pp, mW0, mW1, mW1, GQ_KERNEL_CB_GEMM, false)) return rc;
        for (int64_t j0 = k * mk; j0 < (k + 1) * mk; j0 += L.slab_channels) {
            const int nch = static_cast<int>((k + 1) * mk - j0 < L.slab_channels ? (k + 1) * mk - j0 : L.slab_channels);
            {
                const long long total = static_cast<long long>(d_in) * nch;
                LaunchScope scope(GQ_KERNEL_CB_AUX, st);
                gq::cb_onehot_kernel<<<grid_for(total, 256, di->sm_count, 8), 256, 0, st>>>(
                    Qt, static_cast<int>(d_in), static_cast<int>(d_out), static_cast<int>(j0), nch, m, Pm, L.slab_ld);
            }
            GQ_CUDA(cudaGetLastError());
            // HP = H_k Pm: the one-hot columns are exact in bf16; the two leading terms of H carry 16 mantissa bits
            gq::PairGemmParams pq{};
            pq.n_terms = 2;
            pq.term_a[0] = 0; pq.term_b[0] = 3;
            pq.term_a[1] = 1; pq.term_b[1] = 3;
            pq.full_k = k;
            pq.col0 = 0;
            pq.cols = nch * m;
            pq.C = HP;
            pq.ldc = L.slab_ld;
            if (int32_t rc = launch_full(pq, mPm, mPm, mPm, GQ_KERNEL_CB_GEMM, pq.cols > 2 * gq::TILE_N)) return rc;
            {
                LaunchScope scope(GQ_KERNEL_CB_FOLD, st);
                if (m % 4 == 0)
                    gq::cb_fold4_kernel<<<dim3((nch + gq::CB_FOLD4_CH - 1) / gq::CB_FOLD4_CH, 16), gq::CB_FOLD4_CH * 4, 0, st>>>(
                        HP, L.slab_ld, HW, Qt, static_cast<int>(d_in), static_cast<int>(d_out), static_cast<int>(j0), nch, m, Gm, Rv);
                else
                    gq::cb_fold_kernel<<<dim3((nch + gq::CB_FOLD_CH - 1) / gq::CB_FOLD_CH, 16), gq::CB_FOLD_CH * 16, 0, st>>>(
                        HP, L.slab_ld, HW, Qt, static_cast<int>(d_in), static_cast<int>(d_out), static_cast<int>(j0), nch, m, Gm, Rv);
            }
            GQ_CUDA(cudaGetLastError());
        }
    }
    {
        LaunchScope scope(GQ_KERNEL_CB_FOLD, st);
        gq::cb_solve_kernel<<<static_cast<unsigned>((d_out + 127) / 128), 128, 0, st>>>(Gm, Rv, static_cast<int>(d_out), m,
                                                                                      lambda, codebook);
    }
    GQ_CUDA(cudaGetLastError());
    if (W_hat) {
        const long long count = static_cast<long long>(d_out) * d_in;
        LaunchScope scope(GQ_KERNEL_CB_AUX, st);
        gq::cb_apply_kernel<<<grid_for(count, 256, di->sm_count, 8), 256, 0, st>>>(codebook, Q, count, static_cast<int>(d_in),
                                                                                 m, W_hat);
        GQ_CUDA(cudaGetLastError());
    }
    return GQ_OK;
}

size_t gq_lnq_workspace_bytes(int64_t d_in, int64_t d_out, int32_t g, int32_t m)
{
    const size_t cb = gq_codebook_workspace_bytes(d_in, d_out, g, m);
    const size_t cd = gq_cd_workspace_bytes(d_in, d_out, g);
    if (cb == 0 || cd == 0) return 0;
    return cb > cd ? cb : cd;                     // the two steps alternate: one region serves both
}

int32_t gq_lnq(const float *W, uint8_t *Q, int32_t m, int64_t d_in, int64_t d_out, const float *H, int32_t g,
               int32_t T, int32_t K, double lambda, float *codebook, float *W_hat, void *workspace,
               size_t workspace_bytes, void *stream)
{
    if (!W || !Q || !H || !codebook || !W_hat || T < 0 || K < 0) return GQ_ERR_INVALID_ARG;
    const size_t need = gq_lnq_workspace_bytes(d_in, d_out, g, m);
    if (need == 0) {
        if (int32_t rc = check_layer_shape(d_in, d_out, g, true)) return rc;
        return (m < 1) ? GQ_ERR_INVALID_ARG : GQ_ERR_UNSUPPORTED_SHAPE;
    }
    if (!workspace || workspace_bytes < need) return GQ_ERR_WORKSPACE;
    {
        const size_t w4 = static_cast<size_t>(d_out) * d_in * 4;
        const ByteRange wr[4] = {{Q, static_cast<size_t>(d_out) * d_in}, {codebook, static_cast<size_t>(d_out) * m * 4},
                                 {W_hat, w4}, {workspace, need}};
        const ByteRange ro[2] = {{W, w4}, {H, static_cast<size_t>(g) * d_in * d_in * 4}};
        if (int32_t rc = check_disjoint(wr, ro)) return rc;
    }
    for (int32_t t = 0; t < T; ++t) {
        if (int32_t rc = gq_codebook_update(W, Q, m, d_in, d_out, H, g, lambda, codebook, W_hat, workspace,
                                            workspace_bytes, stream))
            return rc;
        if (K == 0) continue;
        if (int32_t rc = gq_cd_cycles(W, W_hat, Q, codebook, m, d_in, d_out, H, g, K, workspace, workspace_bytes, stream))
            return rc;
    }
    return gq_codebook_update(W, Q, m, d_in, d_out, H, g, lambda, codebook, W_hat, workspace, workspace_bytes, stream);
}

int32_t gq_selftest_wait_timeout(int32_t budget_ms, void *stream)
{
    if (budget_ms < 1 || budget_ms > 1000) return GQ_ERR_INVALID_ARG;
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    gq::wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        di->status_ptr, static_cast<unsigned long long>(budget_ms) * 1000000ull);
    g_launches.fetch_add(1);
    GQ_CUDA(cudaGetLastError());
    return GQ_OK;
}

int32_t gq_kernel_timing_enable(int32_t enable)
{
    // Only the switch: what has been recorded so far stays until gq_kernel_timing_read collects it, so that a
    // caller can time a sample of its launches (switch on, run, switch off, run untimed, ...).
    g_timing_on.store(enable ? 1 : 0);
    return GQ_OK;
}

int32_t gq_kernel_timing_read(double *ms_sum, uint64_t *launches)
{
    if (!ms_sum || !launches) return GQ_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    int32_t rc = GQ_OK;
    for (int id = 0; id < GQ_KERNEL_COUNT; ++id) {
        double total = 0.0;
        uint64_t count = 0;
        for (auto &pr : g_timing_events[id]) {
            float ms = 0.0f;
            cudaError_t e = cudaEventSynchronize(pr.second);
            if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, pr.first, pr.second);
            if (e != cudaSuccess) {
                tl_last_cuda_error = static_cast<int32_t>(e);
                rc = GQ_ERR_CUDA;
            } else {
                total += ms;
                ++count;
            }
            cudaEventDestroy(pr.first);
            cudaEventDestroy(pr.second);
        }
        g_timing_events[id].clear();
        ms_sum[id] = total;
        launches[id] = count;
    }
    return rc;
}

int32_t gq_check(void *stream, uint32_t *detail)
{
    DeviceInfo *di;
    if (int32_t rc = device_info(&di)) return rc;
    GQ_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    uint32_t word[4] = {0, 0, 0, 0};
    GQ_CUDA(cudaMemcpy(word, di->status_ptr, sizeof word, cudaMemcpyDeviceToHost));
    if (detail) std::memcpy(detail, word, sizeof word);
    if (word[0] == 0) return GQ_OK;
    GQ_CUDA(cudaMemset(di->status_ptr, 0, sizeof word));
    if (detail) detail[0] = static_cast<uint32_t>(GQ_ERR_TIMEOUT);
    return word[0] == gq::STATUS_TIMEOUT ? GQ_ERR_TIMEOUT : GQ_ERR_CUDA;
}

size_t gq_layer_host_arena_bytes(int64_t chunk, int64_t d_in, int64_t d_out, int32_t g)
{
    if (chunk < 1 || check_layer_shape(d_in, d_out, g, true) != GQ_OK) return 0;
    size_t total = 0;
    total += 2 * round_up(static_cast<size_t>(chunk) * d_in * 2, 1024);      // X chunk, double buffered
    total += 2 * round_up(static_cast<size_t>(chunk) * d_out * 2, 1024);     // grad chunk, double buffered
    total += round_up(static_cast<size_t>(g) * chunk * 4, 1024);             // s
    total += round_up(static_cast<size_t>(g) * d_in * d_in * 4, 1024);       // H
    total += 2 * round_up(static_cast<size_t>(d_out) * d_in * 4, 1024);      // W, W_hat
    total += round_up(static_cast<size_t>(g + 1) * sizeof(double), 1024);    // loss: g + 1 fp64 values
    total += hessian_ws_bytes(chunk, d_in, g);
    total += objective_layout(d_in, d_out, g).total;
    return total;
}

int32_t gq_layer_objective_host(const void *X_host, const void *grad_host, int64_t n, int64_t chunk, int64_t d_in,
                                int64_t d_out, int32_t g, float grad_scale, const float *W_host,
                                const float *W_hat_host, double *loss_host, float *H_host, void *arena,
                                size_t arena_bytes, void *stream)
{
    if (!X_host || !grad_host || !W_host || !W_hat_host || !loss_host || n < 0 || chunk < 1)
        return GQ_ERR_INVALID_ARG;
    if (int32_t rc = check_layer_shape(d_in, d_out, g, true)) return rc;
    const size_t need = gq_layer_host_arena_bytes(chunk, d_in, d_out, g);
    if (!arena || arena_bytes < need) return GQ_ERR_WORKSPACE;
    if (!aligned(arena, 1024)) return GQ_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    uint8_t *p = static_cast<uint8_t *>(arena);
    auto take = [&p](size_t bytes) { uint8_t *q = p; p += round_up(bytes, 1024); return q; };
    uint8_t *xbuf[2], *gbuf[2];
    xbuf[0] = take(static_cast<size_t>(chunk) * d_in * 2);
    xbuf[1] = take(static_cast<size_t>(chunk) * d_in * 2);
    gbuf[0] = take(static_cast<size_t>(chunk) * d_out * 2);
    gbuf[1] = take(static_cast<size_t>(chunk) * d_out * 2);
    float *s = reinterpret_cast<float *>(take(static_cast<size_t>(g) * chunk * 4));
    const size_t h_bytes = static_cast<size_t>(g) * d_in * d_in * 4;
    float *H = reinterpret_cast<float *>(take(h_bytes));
    const size_t w_bytes = static_cast<size_t>(d_out) * d_in * 4;
    float *W = reinterpret_cast<float *>(take(w_bytes));
    float *What = reinterpret_cast<float *>(take(w_bytes));
    double *loss = reinterpret_cast<double *>(take(static_cast<size_t>(g + 1) * sizeof(double)));
    const size_t hws_bytes = hessian_ws_bytes(chunk, d_in, g);
    void *hws = take(hws_bytes);
    const size_t ows_bytes = objective_layout(d_in, d_out, g).total;
    void *ows = take(ows_bytes);

    // Copies run on a second stream so that chunk c+1 is in flight while chunk c is processed.
    cudaStream_t copy_st = nullptr;
    cudaEvent_t copied[2] = {nullptr, nullptr}, consumed[2] = {nullptr, nullptr}, start = nullptr;
    int32_t rc = GQ_OK;
    auto fail = [&rc](cudaError_t e) {
        if (e != cudaSuccess && rc == GQ_OK) { tl_last_cuda_error = static_cast<int32_t>(e); rc = GQ_ERR_CUDA; }
        return e != cudaSuccess;
    };
    fail(cudaStreamCreateWithFlags(&copy_st, cudaStreamNonBlocking));
    for (int b = 0; b < 2 && rc == GQ_OK; ++b) {
        fail(cudaEventCreateWithFlags(&copied[b], cudaEventDisableTiming));
        fail(cudaEventCreateWithFlags(&consumed[b], cudaEventDisableTiming));
    }
    if (rc == GQ_OK) fail(cudaEventCreateWithFlags(&start, cudaEventDisableTiming));
    if (rc == GQ_OK) {
        fail(cudaEventRecord(start, st));              // the copy stream starts after prior work on `stream`
        fail(cudaStreamWaitEvent(copy_st, start, 0));
        fail(cudaMemsetAsync(H, 0, h_bytes, st));
        fail(cudaMemcpyAsync(W, W_host, w_bytes, cudaMemcpyHostToDevice, st));
        fail(cudaMemcpyAsync(What, W_hat_host, w_bytes, cudaMemcpyHostToDevice, st));
    }
    const int64_t n_chunks = (n + chunk - 1) / chunk;
    for (int64_t c = 0; c < n_chunks && rc == GQ_OK; ++c) {
        const int b = static_cast<int>(c & 1);
        const int64_t tok0 = c * chunk;
        const int64_t nt = (n - tok0 < chunk) ? (n - tok0) : chunk;
        if (c >= 2) fail(cudaStreamWaitEvent(copy_st, consumed[b], 0));
        fail(cudaMemcpyAsync(xbuf[b], static_cast<const uint8_t *>(X_host) + static_cast<size_t>(tok0) * d_in * 2,
                             static_cast<size_t>(nt) * d_in * 2, cudaMemcpyHostToDevice, copy_st));
        fail(cudaMemcpyAsync(gbuf[b], static_cast<const uint8_t *>(grad_host) + static_cast<size_t>(tok0) * d_out * 2,
                             static_cast<size_t>(nt) * d_out * 2, cudaMemcpyHostToDevice, copy_st));
        fail(cudaEventRecord(copied[b], copy_st));
        fail(cudaStreamWaitEvent(st, copied[b], 0));
        if (rc != GQ_OK) break;
        rc = gq_saliency_prepared(gbuf[b], nt, d_out, d_out, g, grad_scale, s, chunk, hws, hws_bytes, st);
        if (rc == GQ_OK)
            rc = gq_hessian_accumulate(xbuf[b], nt, d_in, d_in, s, chunk, g, H, GQ_HESSIAN_S_PREPARED, hws, hws_bytes, st);
        if (rc == GQ_OK) fail(cudaEventRecord(consumed[b], st));
    }
    if (rc == GQ_OK) rc = gq_hessian_finalize(H, d_in, g, st);
    if (rc == GQ_OK) rc = gq_objective(W, What, d_in, d_out, H, g, loss, ows, ows_bytes, st);
    if (rc == GQ_OK) {
        fail(cudaMemcpyAsync(loss_host, loss, sizeof(double) * (g + 1), cudaMemcpyDeviceToHost, st));
        if (H_host) fail(cudaMemcpyAsync(H_host, H, h_bytes, cudaMemcpyDeviceToHost, st));
    }
    // Always drain both streams before their events and the copy stream are destroyed.
    if (copy_st) cudaStreamSynchronize(copy_st);
    const int32_t chk = gq_check(stream, nullptr);
    if (rc == GQ_OK) rc = chk;
    for (int b = 0; b < 2; ++b) {
        if (copied[b]) cudaEventDestroy(copied[b]);
        if (consumed[b]) cudaEventDestroy(consumed[b]);
    }
    if (start) cudaEventDestroy(start);
    if (copy_st) cudaStreamDestroy(copy_st);
    return rc;
}

}  // extern "C"
