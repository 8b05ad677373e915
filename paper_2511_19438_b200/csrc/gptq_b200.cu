// C ABI of the gptq_b200 library: argument validation, workspace bookkeeping, dispatch.
// The library is one translation unit; the kernels live in the headers included below.
#include "gptq_common.cuh"
#include "gptq_layout.cuh"
#include "gptq_streamk.cuh"
#include "gptq_splitk.cuh"
#include "gptq_umma.cuh"
#include "gptq_umma2.cuh"
#include "gptq_w8.cuh"
#include "gptq_wn.cuh"

#include <atomic>
#include <cstdio>
#include <mutex>
#include <unordered_map>
#include <vector>

namespace gptq {

static std::atomic<int> g_last_cuda_error{0};
static std::atomic<int> g_use_cta_pairs{0};

int record_cuda_error(cudaError_t e)
{
    if (e == cudaSuccess) return GPTQ_OK;
    g_last_cuda_error.store((int)e);
    return GPTQ_ERR_CUDA;
}

int next_trace_slot()
{
#ifdef GPTQ_TIMELINE
    static std::atomic<int> next{0};
    return next.fetch_add(1) % kTraceLaunches;
#else
    return -1;
#endif
}

int ensure_dynamic_smem(const void *kernel, int *configured, int smem_bytes)
{
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return GPTQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (configured[dev] >= smem_bytes) return GPTQ_OK;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return record_cuda_error(e);
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return record_cuda_error(e);
    configured[dev] = smem_bytes;
    return GPTQ_OK;
}

constexpr int kMaxDevices = 64;
constexpr size_t kTicketAreaBytes = 16384;   // 4096 panels
constexpr int kStreamKMaxRows = 64;          // tokens per mma.sync launch
#ifndef GPTQ_UMMA_MIN_TOKENS
#define GPTQ_UMMA_MIN_TOKENS 17
#endif
constexpr int kUmmaMinTokens = GPTQ_UMMA_MIN_TOKENS;   // from this many tokens on, gptq_gemm uses the tcgen05 kernel

static Workspace g_workspace[kMaxDevices];
static int g_sm_count[kMaxDevices];
static std::mutex g_mutex;

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_shape(int M, int N, int K, int group_size)
{
    if (M < 1 || N < 8 || K < 8 || group_size < 1) return GPTQ_ERR_SHAPE;
    if (K % 8 || N % 8 || K % group_size) return GPTQ_ERR_SHAPE;
    return GPTQ_OK;
}
// On success `group_size` becomes the group size of the TILED layer: a checkpoint whose groups are a multiple of 128
// rows (256, 512, ..., K = one group per column) is tiled as groups of 128 rows that repeat their group's scales and
// zero points, so the kernels see an ordinary group-128 layer.
static int check_fast_path(int N, int K, int &group_size)
{
    const bool coarse = group_size > kGroup && group_size % kGroup == 0;
    if ((!coarse && group_size != 128 && group_size != 64 && group_size != 32) || N % kPanel || K % kGroup)
        return GPTQ_ERR_UNSUPPORTED;
    if (N / kPanel > (int)(kTicketAreaBytes / sizeof(int))) return GPTQ_ERR_UNSUPPORTED;
    if (coarse) group_size = kGroup;
    return GPTQ_OK;
}
static inline int tiled_group_size(int group_size) { return group_size > kGroup ? kGroup : group_size; }

static int current_device_sms(int *dev_out, int *sms_out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return GPTQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_sm_count[dev] == 0) {
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return record_cuda_error(e);
        g_sm_count[dev] = sms;
    }
    *dev_out = dev;
    *sms_out = g_sm_count[dev];
    return GPTQ_OK;
}

// Stream-K launch geometry and scratch need (the kernel behind gptq_gemm_noalloc).
struct StreamKGemmPlan {
    StreamKPlan sk;          // plan of one launch (for the largest chunk)
    int m_chunks;
    size_t x_perm_bytes;     // gathered activations (act-order)
    size_t workspace_bytes;  // 0 if nothing is needed
};

static StreamKGemmPlan make_streamk_plan(int M, int N, int K, int act_order, int sm_count)
{
    StreamKGemmPlan gp{};
    const int rows = M < kStreamKMaxRows ? M : kStreamKMaxRows;
    gp.sk = plan_streamk(rows, N, K, sm_count);
    gp.m_chunks = (M + kStreamKMaxRows - 1) / kStreamKMaxRows;
    gp.x_perm_bytes = act_order ? (((size_t)M * K * sizeof(__half) + 255) & ~(size_t)255) : 0;
    const size_t need = gp.sk.partial_bytes + gp.x_perm_bytes;
    gp.workspace_bytes = need ? kTicketAreaBytes + need : 0;
    return gp;
}

// gptq_gemm keeps its split-K partials on chip; its only scratch is the gathered x of act-order layers.
static size_t gemm_workspace_need(int M, int K, int act_order)
{
    return act_order == 1 ? (((size_t)M * K * sizeof(__half) + 255) & ~(size_t)255) : 0;   // 2: x arrives sorted
}

// Copy streams and events of gptq_gemm_host_batch (per device, created on first use; no device memory).
struct HostPipe {
    std::mutex enqueue;   // held for a whole gptq_gemm_host_batch call: the streams and events are per device
    cudaStream_t in = nullptr, out = nullptr;
    std::vector<cudaEvent_t> events;
};
static HostPipe g_host_pipe[kMaxDevices];

static int ensure_host_pipe(int dev, size_t n_events, HostPipe **out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    HostPipe &p = g_host_pipe[dev];
    cudaError_t e;
    if (p.in == nullptr && (e = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking)) != cudaSuccess)
        return record_cuda_error(e);
    if (p.out == nullptr && (e = cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking)) != cudaSuccess)
        return record_cuda_error(e);
    while (p.events.size() < n_events) {
        cudaEvent_t ev;
        if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return record_cuda_error(e);
        p.events.push_back(ev);
    }
    *out = &p;
    return GPTQ_OK;
}

}  // namespace gptq

using namespace gptq;

extern "C" {

const char *gptq_status_string(int status)
{
    switch (status) {
    case GPTQ_OK: return "ok";
    case GPTQ_ERR_NULL: return "a required pointer is NULL";
    case GPTQ_ERR_SHAPE: return "invalid shape (need M>=1, K%8==0, N%8==0, K%group_size==0)";
    case GPTQ_ERR_ALIGN: return "a pointer is not 16-byte aligned";
    case GPTQ_ERR_UNSUPPORTED: return "shape outside the tiled fast path (group_size 32, 64 or a multiple of 128, N%128==0, K%128==0)";
    case GPTQ_ERR_LAYOUT: return "invalid layout selector or flag";
    case GPTQ_ERR_GIDX: return "g_idx entry out of range, or groups of unequal size";
    case GPTQ_ERR_WORKSPACE: return "workspace missing or too small (see gptq_workspace_bytes)";
    case GPTQ_ERR_CUDA: return "a CUDA runtime call failed (see gptq_last_cuda_error)";
    case GPTQ_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    default: return "unknown status";
    }
}

int gptq_last_cuda_error(void) { return g_last_cuda_error.load(); }

int gptq_set_cta_pairs(int enable)
{
    g_use_cta_pairs.store(enable ? 1 : 0);
    return GPTQ_OK;
}

int gptq_unpack_u8(const int32_t *qweight, const int32_t *qzeros, uint8_t *q_out, uint8_t *z_out, int N, int K,
                   int group_size, void *stream)
{
    if ((q_out && !qweight) || (z_out && !qzeros) || (!q_out && !z_out)) return GPTQ_ERR_NULL;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    return launch_unpack_u8(qweight, qzeros, q_out, z_out, N, K, K / group_size, (cudaStream_t)stream);
}

int gptq_dequant_f32(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                     float *w_out, int N, int K, int group_size, int act_order, int repacked, void *stream)
{
    return gptq_dequant_f32_format(qweight, qzeros, scales, g_idx, w_out, N, K, group_size, act_order, repacked, 0, stream);
}

int gptq_dequant_f32_format(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                            float *w_out, int N, int K, int group_size, int act_order, int repacked, int format,
                            void *stream)
{
    if (format & ~(GPTQ_FORMAT_ZEROS_MINUS_ONE | GPTQ_FORMAT_GATE_UP | GPTQ_FORMAT_BF16)) return GPTQ_ERR_LAYOUT;
    if (!qweight || !qzeros || !scales || !w_out || (act_order && !g_idx)) return GPTQ_ERR_NULL;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    if (repacked != 0 && repacked != 1) return GPTQ_ERR_LAYOUT;
    if (!repacked && (format & GPTQ_FORMAT_GATE_UP)) return GPTQ_ERR_LAYOUT;   // a property of the tiled layout only
    if (repacked) {
        st = check_fast_path(N, K, group_size);
        if (st) return st;
    }
    return launch_dequant_f32(qweight, qzeros, scales, g_idx, w_out, N, K, group_size, act_order, repacked, format,
                              (cudaStream_t)stream);
}

size_t gptq_repack_bytes(int which, int N, int K, int group_size, int act_order)
{
    if (check_shape(1, N, K, group_size) != GPTQ_OK) return 0;
    const size_t G = (size_t)(K / tiled_group_size(group_size));   // coarser groups are stored once per 128 rows
    switch (which) {
    case 0: return (size_t)K / 8 * N * 4;
    case 1: return G * (N / 8) * 4 + kTrailerBytes;   // + the format trailer
    case 2: return G * N * 2;
    case 3: return act_order ? (size_t)K * 4 : 0;
    default: return 0;
    }
}

int gptq_repack(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, int N, int K,
                int group_size, int act_order, void *stream)
{
    return gptq_repack_format(qweight, qzeros, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, N, K,
                              group_size, act_order, 0, stream);
}

int gptq_repack_format(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                       void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, int N, int K,
                       int group_size, int act_order, int format, void *stream)
{
    if (format & ~(GPTQ_FORMAT_ZEROS_MINUS_ONE | GPTQ_FORMAT_GATE_UP | GPTQ_FORMAT_BF16)) return GPTQ_ERR_LAYOUT;
    if (!qweight || !qzeros || !scales || !qweight_out || !qzeros_out || !scales_out) return GPTQ_ERR_NULL;
    if (act_order && (!g_idx || !perm_out)) return GPTQ_ERR_NULL;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    const int source_group_size = group_size;
    st = check_fast_path(N, K, group_size);
    if (st) return st;
    if (!aligned16(qweight_out) || !aligned16(qzeros_out) || !aligned16(scales_out)) return GPTQ_ERR_ALIGN;
    if (qweight_out == (const void *)qweight || qzeros_out == (const void *)qzeros || scales_out == scales)
        return GPTQ_ERR_LAYOUT;
    return launch_repack(qweight, qzeros, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, N, K,
                         source_group_size, act_order, format, (cudaStream_t)stream);
}

static void set_kernel_name(gptq_plan_t *out, const char *fmt, int a, int b = 0, int c = 0, int d = 0)
{
    snprintf(out->kernel_name, sizeof(out->kernel_name), fmt, a, b, c, d);
}

int gptq_plan(int M, int N, int K, int group_size, int act_order, int sm_count, gptq_plan_t *out)
{
    if (!out) return GPTQ_ERR_NULL;
    int st = check_shape(M, N, K, group_size);
    if (st) return st;
    st = check_fast_path(N, K, group_size);
    if (st) return st;
    if (sm_count < 1) return GPTQ_ERR_SHAPE;
    if (M >= kUmmaMinTokens) {
        const UmmaPlan up = plan_umma(M, N, K, sm_count);
        out->kernel = 2;
        out->m_tile = up.tok;
        out->m_chunks = 1;
        out->stages = up.stages;
        out->ctas = up.ctas;
        out->items = (N / kPanel) * (K / kGroup);
        out->split_panels = 0;
        out->smem_bytes = up.smem_bytes;
        out->workspace_bytes = gemm_workspace_need(M, K, act_order);
        out->cluster_size = up.S;
        out->tail_ctas = up.tail_tiles * up.tail_S;
        out->tail_cluster_size = up.tail_S;
        out->split_panels = up.S > 1 ? N / kPanel : 0;
        if (g_use_cta_pairs.load() && umma2_applicable(M, N) && group_size == kGroup)
            set_kernel_name(out, "umma2_kernel", 0);
        else
            snprintf(out->kernel_name, sizeof(out->kernel_name), "umma_kernel<%d,%d,%d,%d,%d>", up.tok,
                     umma_a_stages(up.tok, up.np), up.np, up.sets, kGroup / group_size);
        return GPTQ_OK;
    }
    const int rows = M < kStreamKMaxRows ? M : kStreamKMaxRows;
    const SplitKPlan pl = plan_splitk(rows, N, K, group_size, sm_count);
    out->kernel = 1;
    out->m_tile = pl.m_tile;
    out->m_chunks = (M + kStreamKMaxRows - 1) / kStreamKMaxRows;
    out->stages = pl.stages;
    out->ctas = pl.ctas;
    out->items = (N / kPanel) * (K / kGroup);
    out->split_panels = pl.S > 1 ? N / kPanel : 0;
    out->smem_bytes = pl.smem_bytes;
    out->workspace_bytes = gemm_workspace_need(M, K, act_order);
    out->cluster_size = pl.S;
    out->tail_ctas = 0;
    out->tail_cluster_size = 1;
    set_kernel_name(out, "splitk_kernel<%d,%d>", pl.m_tile / 8, pl.sub);
    return GPTQ_OK;
}

int gptq_plan_noalloc(int M, int N, int K, int group_size, int act_order, int sm_count, gptq_plan_t *out)
{
    if (!out) return GPTQ_ERR_NULL;
    int st = check_shape(M, N, K, group_size);
    if (st) return st;
    st = check_fast_path(N, K, group_size);
    if (st) return st;
    if (group_size != kGroup) return GPTQ_ERR_UNSUPPORTED;   // the stream-K kernel is built for group size 128 only
    if (sm_count < 1) return GPTQ_ERR_SHAPE;
    const StreamKGemmPlan gp = make_streamk_plan(M, N, K, act_order, sm_count);
    out->kernel = 3;
    out->m_tile = gp.sk.m_tile;
    out->m_chunks = gp.m_chunks;
    out->stages = gp.sk.stages;
    out->ctas = gp.sk.ctas;
    out->items = gp.sk.items;
    out->split_panels = gp.sk.split_panels;
    out->smem_bytes = gp.sk.smem_bytes;
    out->workspace_bytes = gp.workspace_bytes;
    out->cluster_size = 1;
    out->tail_ctas = 0;
    out->tail_cluster_size = 1;
    set_kernel_name(out, "streamk_kernel<%d>", gp.sk.m_tile / 8);
    return GPTQ_OK;
}

int gptq_plan_cta_range(int items, int ctas, int cta, int *first_item, int *end_item)
{
    if (!first_item || !end_item) return GPTQ_ERR_NULL;
    if (items < 1 || ctas < 1 || ctas > items || cta < 0 || cta >= ctas) return GPTQ_ERR_SHAPE;
    *first_item = sk_range_begin(items, ctas, cta);
    *end_item = sk_range_begin(items, ctas, cta + 1);
    return GPTQ_OK;
}

int gptq_plan_panel_owners(int items, int ctas, int groups, int panel, int *first_cta, int *last_cta)
{
    if (!first_cta || !last_cta) return GPTQ_ERR_NULL;
    if (items < 1 || ctas < 1 || ctas > items || groups < 1 || items % groups || panel < 0 ||
        panel >= items / groups)
        return GPTQ_ERR_SHAPE;
    const long long first_item = (long long)panel * groups;
    *first_cta = sk_owner(items, ctas, first_item);
    *last_cta = sk_owner(items, ctas, first_item + groups - 1);
    return GPTQ_OK;
}

size_t gptq_workspace_bytes(int M, int N, int K, int group_size, int act_order)
{
    if (check_shape(M, N, K, group_size) != GPTQ_OK || check_fast_path(N, K, group_size) != GPTQ_OK) return 0;
    return gemm_workspace_need(M, K, act_order);
}

int gptq_set_workspace(void *ptr, size_t bytes)
{
    int dev, sms;
    int st = current_device_sms(&dev, &sms);
    if (st) return st;
    if (ptr != nullptr && !aligned16(ptr)) return GPTQ_ERR_ALIGN;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_workspace[dev].ptr = ptr;
    g_workspace[dev].bytes = ptr ? bytes : 0;
    return GPTQ_OK;
}

} // extern "C"

// y = x W (fuse == 0, y is [M, N]) or silu(gate) * up of y's column halves (fuse == 1, y is [M, N / 2])
static int gemm_dispatch(const void *x, const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                         void *y, int M, int N, int K, int group_size, int act_order, int fuse, const void *bias,
                         const void *residual, const int32_t *out_index, void *stream, int bf16 = 0)
{
    if (act_order < 0 || act_order > GPTQ_ACT_ORDER_PRESORTED) return GPTQ_ERR_LAYOUT;
    if (!x || !qweight || !qzeros || !scales || !y || (act_order == 1 && !g_idx)) return GPTQ_ERR_NULL;
    int st = check_shape(M, N, K, group_size);
    if (st) return st;
    if (!aligned16(x) || !aligned16(qweight) || !aligned16(qzeros) || !aligned16(scales) || !aligned16(y))
        return GPTQ_ERR_ALIGN;
    if (act_order == 1 && !aligned16(g_idx)) return GPTQ_ERR_ALIGN;
    if (!aligned16(bias) || !aligned16(residual) || !aligned16(out_index)) return GPTQ_ERR_ALIGN;     // a null pointer passes
    st = check_fast_path(N, K, group_size);
    if (st) return st;

    int dev, sms;
    st = current_device_sms(&dev, &sms);
    if (st) return st;
    cudaStream_t s = (cudaStream_t)stream;
    const __half *xin = (const __half *)x;
    const bool extras = bias != nullptr || residual != nullptr;
    if (bf16 && (fuse || extras)) return GPTQ_ERR_UNSUPPORTED;     // the fused epilogues exist for fp16 only
    if (act_order == 1) {
        Workspace ws;
        {
            std::lock_guard<std::mutex> lock(g_mutex);
            ws = g_workspace[dev];
        }
        if (ws.ptr == nullptr || ws.bytes < gemm_workspace_need(M, K, act_order)) return GPTQ_ERR_WORKSPACE;
        __half *x_perm = (__half *)ws.ptr;
        st = launch_gather_x((const __half *)x, g_idx, x_perm, M, K, s);
        if (st) return st;
        xin = x_perm;
    }
    const size_t ldy = fuse ? (size_t)N / 2 : (size_t)N;
    if (M >= kUmmaMinTokens) {
        if (!fuse && !extras && !bf16 && g_use_cta_pairs.load() && umma2_applicable(M, N) && group_size == kGroup) {
            const Umma2Plan p2 = plan_umma2(M, N, K);
            return launch_umma2(xin, qweight, qzeros, scales, (__half *)y, M, N, K, p2, s);
        }
        // tcgen05 kernel: 32- to 256-token tiles
        const UmmaPlan pl = plan_umma(M, N, K, sms);
        return launch_umma(xin, qweight, qzeros, scales, (__half *)y, M, N, K, group_size, pl, fuse, (const __half *)bias,
                           (const __half *)residual, out_index, bf16, s);
    }
    for (int m0 = 0; m0 < M; m0 += kStreamKMaxRows) {
        const int rows = (M - m0) < kStreamKMaxRows ? (M - m0) : kStreamKMaxRows;
        const SplitKPlan pl = plan_splitk(rows, N, K, group_size, sms);
        st = launch_splitk(xin + (size_t)m0 * K, qweight, qzeros, scales, (__half *)y + (size_t)m0 * ldy, rows, N, K,
                           pl, fuse, (const __half *)bias,
                           residual ? (const __half *)residual + (size_t)m0 * N : nullptr, out_index, bf16, s);
        if (st) return st;
    }
    return GPTQ_OK;
}

extern "C" {

int gptq_gemm(const void *x, const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
              void *y, int M, int N, int K, int group_size, int act_order, void *stream)
{
    return gemm_dispatch(x, qweight, qzeros, scales, g_idx, y, M, N, K, group_size, act_order, 0, nullptr, nullptr, nullptr, stream);
}

int gptq_gemm_bf16(const void *x, const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                   void *y, int M, int N, int K, int group_size, int act_order, void *stream)
{
    return gemm_dispatch(x, qweight, qzeros, scales, g_idx, y, M, N, K, group_size, act_order, 0, nullptr, nullptr, nullptr, stream,
                         1);
}

int gptq_gemm_bias_residual(const void *x, const void *qweight, const void *qzeros, const void *scales,
                            const int32_t *g_idx, const void *bias, const void *residual, void *y, int M, int N, int K,
                            int group_size, int act_order, void *stream)
{
    return gemm_dispatch(x, qweight, qzeros, scales, g_idx, y, M, N, K, group_size, act_order, 0, bias, residual, nullptr, stream);
}

int gptq_gemm_silu_mul(const void *x, const void *qweight, const void *qzeros, const void *scales,
                       const int32_t *g_idx, void *out, int M, int N, int K, int group_size, int act_order,
                       void *stream)
{
    return gemm_dispatch(x, qweight, qzeros, scales, g_idx, out, M, N, K, group_size, act_order, 1, nullptr, nullptr, nullptr,
                         stream);
}

int gptq_gemm_silu_mul_scatter(const void *x, const void *qweight, const void *qzeros, const void *scales,
                               const int32_t *g_idx, const int32_t *out_index, void *out, int M, int N, int K,
                               int group_size, int act_order, void *stream)
{
    if (!out_index) return GPTQ_ERR_NULL;
    return gemm_dispatch(x, qweight, qzeros, scales, g_idx, out, M, N, K, group_size, act_order, 1, nullptr, nullptr, out_index,
                         stream);
}

// ---- 8-bit weights: two stacked 4-bit planes (gptq_w8.cuh) ----------------------------------------------------------

static int check_w8(int N, int K, int &group_size, int format)
{
    if (format & ~GPTQ_FORMAT_ZEROS_MINUS_ONE) return GPTQ_ERR_LAYOUT;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    return check_fast_path(N, K, group_size);     // K % 128 == 0: a 128-row tile never spans the two planes
}

size_t gptq_repack_w8_bytes(int which, int N, int K, int group_size)
{
    int tiled = group_size;
    if (K < 8 || K > (1 << 29) || check_w8(N, K, tiled, 0) != GPTQ_OK) return 0;
    return gptq_repack_bytes(which, N, 2 * K, group_size, 1);
}

size_t gptq_repack_w8_scratch_bytes(int N, int K, int group_size)
{
    int tiled = group_size;
    if (K < 8 || K > (1 << 29) || check_w8(N, K, tiled, 0) != GPTQ_OK) return 0;
    return w8_scratch_layout(N, K, group_size).total;
}

int gptq_repack_w8(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                   void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, void *scratch,
                   size_t scratch_bytes, int N, int K, int group_size, int act_order, int format, void *stream)
{
    if (!qweight || !qzeros || !scales || !qweight_out || !qzeros_out || !scales_out || !perm_out || !scratch)
        return GPTQ_ERR_NULL;
    if (act_order && !g_idx) return GPTQ_ERR_NULL;
    if (K > (1 << 29)) return GPTQ_ERR_SHAPE;
    int tiled = group_size;
    int st = check_w8(N, K, tiled, format);
    if (st) return st;
    if (!aligned16(qweight_out) || !aligned16(qzeros_out) || !aligned16(scales_out) || !aligned16(perm_out) ||
        (reinterpret_cast<uintptr_t>(scratch) & 255u))
        return GPTQ_ERR_ALIGN;
    if (scratch_bytes < w8_scratch_layout(N, K, group_size).total) return GPTQ_ERR_WORKSPACE;
    return launch_w8_repack(qweight, qzeros, scales, act_order ? g_idx : nullptr, qweight_out, qzeros_out, scales_out,
                            perm_out, scratch, N, K, group_size, (format & GPTQ_FORMAT_ZEROS_MINUS_ONE) ? 1 : 0,
                            (cudaStream_t)stream);
}

int gptq_dequant_f32_w8(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx, float *w_out,
                        int N, int K, int group_size, int act_order, int repacked, int format, void *stream)
{
    if (!qweight || !qzeros || !scales || !w_out || ((act_order || repacked) && !g_idx)) return GPTQ_ERR_NULL;
    if (repacked != 0 && repacked != 1) return GPTQ_ERR_LAYOUT;
    if (format & ~GPTQ_FORMAT_ZEROS_MINUS_ONE) return GPTQ_ERR_LAYOUT;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    if (N % 4) return GPTQ_ERR_SHAPE;
    if (repacked) {
        st = check_fast_path(N, K, group_size);
        if (st) return st;
    }
    return launch_w8_dequant_f32(qweight, qzeros, scales, (act_order || repacked) ? g_idx : nullptr, w_out, N, K,
                                 group_size, repacked, (format & GPTQ_FORMAT_ZEROS_MINUS_ONE) ? 1 : 0, (cudaStream_t)stream);
}

int gptq_gemm_w8(const void *x, const void *qweight, const void *qzeros, const void *scales, const int32_t *perm,
                 void *y, int M, int N, int K, int group_size, void *stream)
{
    if (!x || !qweight || !qzeros || !scales || !perm || !y) return GPTQ_ERR_NULL;
    if (K > (1 << 29)) return GPTQ_ERR_SHAPE;
    int st = check_shape(M, N, K, group_size);
    if (st) return st;
    if (!aligned16(x) || !aligned16(qweight) || !aligned16(qzeros) || !aligned16(scales) || !aligned16(y) || !aligned16(perm))
        return GPTQ_ERR_ALIGN;
    int tiled = group_size;
    st = check_fast_path(N, K, tiled);
    if (st) return st;
    int dev, sms;
    st = current_device_sms(&dev, &sms);
    if (st) return st;
    Workspace ws;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = g_workspace[dev];
    }
    if (ws.ptr == nullptr || ws.bytes < gemm_workspace_need(M, 2 * K, 1)) return GPTQ_ERR_WORKSPACE;
    st = launch_w8_gather_x((const __half *)x, perm, (__half *)ws.ptr, M, K, (cudaStream_t)stream);
    if (st) return st;
    // the stacked layer, its activations already in its row order
    return gemm_dispatch(ws.ptr, qweight, qzeros, scales, nullptr, y, M, N, 2 * K, group_size, GPTQ_ACT_ORDER_PRESORTED, 0,
                         nullptr, nullptr, nullptr, stream);
}

// ---- 2- and 3-bit weights: widened to nibbles by the repack (gptq_wn.cuh) ------------------------------------------

static int check_bits(int bits, int N, int K, int format)
{
    if (bits != 2 && bits != 3) return GPTQ_ERR_UNSUPPORTED;
    if (format & ~GPTQ_FORMAT_ZEROS_MINUS_ONE) return GPTQ_ERR_LAYOUT;
    if (K % 32 || N % 32) return GPTQ_ERR_SHAPE;     // whole words per column and per zero-point row
    return GPTQ_OK;
}

size_t gptq_repack_bits_scratch_bytes(int bits, int N, int K, int group_size)
{
    int tiled = group_size;
    if (check_shape(1, N, K, group_size) != GPTQ_OK || check_bits(bits, N, K, 0) != GPTQ_OK ||
        check_fast_path(N, K, tiled) != GPTQ_OK)
        return 0;
    return wn_scratch_bytes(N, K, group_size);
}

int gptq_repack_bits(int bits, const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                     void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, void *scratch,
                     size_t scratch_bytes, int N, int K, int group_size, int act_order, int format, void *stream)
{
    if (!qweight || !qzeros || !scales || !qweight_out || !qzeros_out || !scales_out || !scratch) return GPTQ_ERR_NULL;
    if (act_order && (!g_idx || !perm_out)) return GPTQ_ERR_NULL;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    st = check_bits(bits, N, K, format);
    if (st) return st;
    int tiled = group_size;
    st = check_fast_path(N, K, tiled);
    if (st) return st;
    if (!aligned16(qweight_out) || !aligned16(qzeros_out) || !aligned16(scales_out) || (reinterpret_cast<uintptr_t>(scratch) & 255u))
        return GPTQ_ERR_ALIGN;
    if (scratch_bytes < wn_scratch_bytes(N, K, group_size)) return GPTQ_ERR_WORKSPACE;
    return launch_wn_repack(qweight, qzeros, scales, act_order ? g_idx : nullptr, qweight_out, qzeros_out, scales_out, perm_out,
                            scratch, N, K, group_size, bits, act_order, (format & GPTQ_FORMAT_ZEROS_MINUS_ONE) ? 1 : 0,
                            (cudaStream_t)stream);
}

int gptq_dequant_f32_bits(int bits, const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                          float *w_out, int N, int K, int group_size, int act_order, int format, void *stream)
{
    if (!qweight || !qzeros || !scales || !w_out || (act_order && !g_idx)) return GPTQ_ERR_NULL;
    int st = check_shape(1, N, K, group_size);
    if (st) return st;
    st = check_bits(bits, N, K, format);
    if (st) return st;
    return launch_wn_dequant_f32(qweight, qzeros, scales, act_order ? g_idx : nullptr, w_out, N, K, group_size, bits,
                                 (format & GPTQ_FORMAT_ZEROS_MINUS_ONE) ? 1 : 0, (cudaStream_t)stream);
}

int gptq_invert_perm(const int32_t *perm, int32_t *inverse, int K, void *stream)
{
    if (!perm || !inverse) return GPTQ_ERR_NULL;
    if (K < 1) return GPTQ_ERR_SHAPE;
    return launch_invert_perm(perm, inverse, K, (cudaStream_t)stream);
}

int gptq_gemm_host(const void *x_host, const void *qweight, const void *qzeros, const void *scales,
                   const int32_t *g_idx, void *y_host, void *x_stage, void *y_stage, int M, int N, int K,
                   int group_size, int act_order, void *stream)
{
    if (!x_host || !y_host || !x_stage || !y_stage) return GPTQ_ERR_NULL;
    int st = check_shape(M, N, K, group_size);
    if (st) return st;
    cudaStream_t s = (cudaStream_t)stream;
    st = record_cuda_error(cudaMemcpyAsync(x_stage, x_host, (size_t)M * K * sizeof(__half), cudaMemcpyHostToDevice, s));
    if (st) return st;
    st = gptq_gemm(x_stage, qweight, qzeros, scales, g_idx, y_stage, M, N, K, group_size, act_order, stream);
    if (st) return st;
    return record_cuda_error(cudaMemcpyAsync(y_host, y_stage, (size_t)M * N * sizeof(__half), cudaMemcpyDeviceToHost, s));
}

// ---- matmul with built-in scratch -----------------------------------------------------------
// Scratch for gptq_gemm_noalloc: lives in the library's device image, so every GPU that loads
// the library holds these 8 MiB until the process exits.  Layout = the registered workspace's:
// [tickets 16 KB][fp32 partial tiles][gathered x (act-order)].
constexpr size_t kStaticScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
// In host code `g_static_scratch` is only a handle for the runtime, never a device address; the
// address a kernel can use is looked up once per device and cached here.
static void *g_static_scratch_addr[kMaxDevices];

static int static_scratch_address(int dev, void **out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);   // device `dev` is current
        if (e != cudaSuccess) return record_cuda_error(e);
        if (p == nullptr) return GPTQ_ERR_CUDA;
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return GPTQ_OK;
}

size_t gptq_noalloc_scratch_bytes(void) { return kStaticScratchBytes; }

int gptq_gemm_noalloc(const void *x, const void *qweight, const void *qzeros, const void *scales,
                      const int32_t *g_idx, void *y, int M, int N, int K, int group_size, int act_order,
                      void *stream)
{
    if (act_order < 0 || act_order > 1) return GPTQ_ERR_LAYOUT;   // the pre-sorted mode belongs to gptq_gemm only
    if (!x || !qweight || !qzeros || !scales || !y || (act_order && !g_idx)) return GPTQ_ERR_NULL;
    int st = check_shape(M, N, K, group_size);
    if (st) return st;
    if (!aligned16(x) || !aligned16(qweight) || !aligned16(qzeros) || !aligned16(scales) || !aligned16(y))
        return GPTQ_ERR_ALIGN;
    if (act_order && !aligned16(g_idx)) return GPTQ_ERR_ALIGN;
    st = check_fast_path(N, K, group_size);
    if (st) return st;
    if (group_size != kGroup) return GPTQ_ERR_UNSUPPORTED;   // the stream-K kernel is built for group size 128 only
    int dev, sms;
    st = current_device_sms(&dev, &sms);
    if (st) return st;
    const StreamKGemmPlan gp = make_streamk_plan(M, N, K, act_order, sms);
    // the built-in scratch has a fixed size: larger problems must use gptq_gemm with a workspace
    if (gp.workspace_bytes > kStaticScratchBytes) return GPTQ_ERR_WORKSPACE;
    void *base = nullptr;
    st = static_scratch_address(dev, &base);
    if (st) return st;

    cudaStream_t s = (cudaStream_t)stream;
    uint8_t *wsb = (uint8_t *)base;
    int *tickets = (int *)wsb;
    float *partials = (float *)(wsb + kTicketAreaBytes);
    // the array keeps whatever the previous call left; the tickets are the only part that must be zero
    st = record_cuda_error(cudaMemsetAsync(tickets, 0, (size_t)(N / kPanel) * sizeof(int), s));
    if (st) return st;
    const __half *xin = (const __half *)x;
    if (act_order) {
        __half *x_perm = (__half *)(wsb + kTicketAreaBytes + gp.sk.partial_bytes);
        st = launch_gather_x((const __half *)x, g_idx, x_perm, M, K, s);
        if (st) return st;
        xin = x_perm;
    }
    for (int m0 = 0; m0 < M; m0 += kStreamKMaxRows) {
        const int rows = (M - m0) < kStreamKMaxRows ? (M - m0) : kStreamKMaxRows;
        const StreamKPlan pl = plan_streamk(rows, N, K, sms);
        st = launch_streamk(xin + (size_t)m0 * K, qweight, qzeros, scales, (__half *)y + (size_t)m0 * N, rows, N, K,
                            pl, partials, tickets, s);
        if (st) return st;
    }
    return GPTQ_OK;
}

} // extern "C"

// mode: 0 = fp16 layers (gptq_gemm), 1 = bfloat16 layers (gptq_gemm_bf16), 2 = 8-bit layers (gptq_gemm_w8)
static int host_batch(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index, int mode)
{
    if (!problems || count < 0) return GPTQ_ERR_NULL;
    for (int i = 0; i < count; ++i) {
        const gptq_host_problem_t &q = problems[i];
        int st = GPTQ_OK;
        if (!q.x_host || !q.y_host || !q.x_stage || !q.y_stage || !q.qweight || !q.qzeros || !q.scales ||
            ((q.act_order == 1 || mode == 2) && !q.g_idx))
            st = GPTQ_ERR_NULL;
        if (!st) st = check_shape(q.M, q.N, q.K, q.group_size);
        if (!st && (!aligned16(q.x_stage) || !aligned16(q.y_stage) || !aligned16(q.qweight) || !aligned16(q.qzeros) ||
                    !aligned16(q.scales)))
            st = GPTQ_ERR_ALIGN;
        int tiled_group = q.group_size;
        if (!st) st = check_fast_path(q.N, q.K, tiled_group);
        if (st) {
            if (bad_index) *bad_index = i;
            return st;
        }
    }
    if (count == 0) return GPTQ_OK;
    // Three-stage pipeline over two internal copy streams: activations go up while earlier matmuls run and their results come down.
    int dev, sms;
    int st = current_device_sms(&dev, &sms);
    if (st) return st;
    HostPipe *pipe = nullptr;
    st = ensure_host_pipe(dev, 3 * (size_t)count + 1, &pipe);
    if (st) return st;
    // one caller at a time per device: the copy streams and events belong to the device, not to the call
    std::lock_guard<std::mutex> enqueue_lock(pipe->enqueue);
    std::vector<cudaEvent_t> events;   // handles copied out: another caller may grow (and move) the device's vector
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        events.assign(pipe->events.begin(), pipe->events.begin() + (3 * (size_t)count + 1));
    }
    cudaStream_t s = (cudaStream_t)stream;
    cudaEvent_t *ev_x = events.data(), *ev_g = ev_x + count, *ev_y = ev_g + count, ev_start = ev_y[count];
    auto check = [&](cudaError_t e) { return record_cuda_error(e); };
    // copies must not start before earlier work on `stream` (which may still use the staging buffers)
    if ((st = check(cudaEventRecord(ev_start, s)))) return st;
    if ((st = check(cudaStreamWaitEvent(pipe->in, ev_start, 0)))) return st;
    if ((st = check(cudaStreamWaitEvent(pipe->out, ev_start, 0)))) return st;
    // from here on the internal streams are forked off `stream`: every exit goes through the join below
    // The problems go through the pipeline in CHUNKS: a chunk is a run of consecutive problems that share no staging
    // buffer (at most kChunk of them).  All x of a chunk are copied up, then its matmuls run back to back on `stream`
    // (consecutive launches overlap through programmatic dependent launch - a dependency on another stream between
    // every two of them would cost about a microsecond each), then all its y are copied down; chunk c + 1 is copied up
    // while chunk c computes and chunk c - 1 comes down.  Events: ev_x[c] chunk c is up, ev_g[c] computed, ev_y[c] down.
    // A chunk that reaches back to a staging buffer used d problems earlier must wait for that problem's chunk, so the
    // pipeline only overlaps if chunks are short against d: a chunk holds at most d / 3 problems (one problem when
    // buffers are reused every few problems, kChunk when every problem has its own).
    constexpr int kChunk = 16;
    std::vector<int> reuse((size_t)count);
    {
        std::unordered_map<const void *, int> last_index;     // staging buffer -> the last problem that used it
        for (int i = 0; i < count; ++i) {
            int d = 3 * kChunk;
            for (const void *buf : {(const void *)problems[i].x_stage, (const void *)problems[i].y_stage}) {
                auto it = last_index.find(buf);
                if (it != last_index.end() && i - it->second < d) d = i - it->second;
            }
            reuse[(size_t)i] = d;
            last_index[problems[i].x_stage] = i;
            last_index[problems[i].y_stage] = i;
        }
    }
    // staging buffer -> the latest chunk whose matmuls read it as x / whose copies down read it as y
    std::unordered_map<const void *, int> read_as_x, copied_as_y;
    int n_chunks = 0;
    for (int i0 = 0; i0 < count && !st;) {
        // ... and at most kChunkBytes of activations and results: large problems (prefill) keep one problem per chunk,
        // where the copies, not the dependencies, set the pace
        constexpr size_t kChunkBytes = 2u << 20;
        auto io_bytes = [&](int i) { return (size_t)problems[i].M * ((size_t)problems[i].K + problems[i].N) * sizeof(__half); };
        int i1 = i0 + 1, limit = reuse[(size_t)i0] / 3;
        size_t bytes = io_bytes(i0);
        for (; i1 < count; ++i1) {
            if (reuse[(size_t)i1] / 3 < limit) limit = reuse[(size_t)i1] / 3;
            if (i1 - i0 >= limit) break;      // (also ends the chunk before a problem that shares a buffer with it)
            bytes += io_bytes(i1);
            if (bytes > kChunkBytes) break;
        }
        const int c = n_chunks++;
        // a staging buffer used by an earlier chunk is overwritten only after that chunk is done with it: after its
        // matmuls (ev_g) where it was their x, after its copies down (ev_y) where it was their y; the streams are in
        // order, so the latest such chunk suffices
        int wait_g = -1, wait_y_in = -1, wait_y = -1;
        for (int i = i0; i < i1; ++i) {
            auto it = read_as_x.find(problems[i].x_stage);
            if (it != read_as_x.end() && it->second > wait_g) wait_g = it->second;
            it = copied_as_y.find(problems[i].x_stage);
            if (it != copied_as_y.end() && it->second > wait_y_in) wait_y_in = it->second;
            it = copied_as_y.find(problems[i].y_stage);
            if (it != copied_as_y.end() && it->second > wait_y) wait_y = it->second;
        }
        for (int i = i0; i < i1; ++i) {
            read_as_x[problems[i].x_stage] = c;
            copied_as_y[problems[i].y_stage] = c;
        }
        if (wait_y_in >= 0) st = check(cudaStreamWaitEvent(pipe->in, ev_y[wait_y_in], 0));
        if (!st && wait_g >= 0 && wait_g > wait_y_in) st = check(cudaStreamWaitEvent(pipe->in, ev_g[wait_g], 0));
        for (int i = i0; i < i1 && !st; ++i) {
            const gptq_host_problem_t &q = problems[i];
            st = check(cudaMemcpyAsync(q.x_stage, q.x_host, (size_t)q.M * q.K * sizeof(__half), cudaMemcpyHostToDevice, pipe->in));
        }
        if (!st) st = check(cudaEventRecord(ev_x[c], pipe->in));
        if (!st) st = check(cudaStreamWaitEvent(s, ev_x[c], 0));
        if (!st && wait_y >= 0) st = check(cudaStreamWaitEvent(s, ev_y[wait_y], 0));
        for (int i = i0; i < i1 && !st; ++i) {
            const gptq_host_problem_t &q = problems[i];
            if (mode == 2)
                st = gptq_gemm_w8(q.x_stage, q.qweight, q.qzeros, q.scales, q.g_idx, q.y_stage, q.M, q.N, q.K, q.group_size, stream);
            else
                st = gemm_dispatch(q.x_stage, q.qweight, q.qzeros, q.scales, q.g_idx, q.y_stage, q.M, q.N, q.K, q.group_size,
                                   q.act_order, 0, nullptr, nullptr, nullptr, stream, mode);
            if (st && bad_index) *bad_index = i;
        }
        if (st) break;
        st = check(cudaEventRecord(ev_g[c], s));
        if (!st) st = check(cudaStreamWaitEvent(pipe->out, ev_g[c], 0));
        for (int i = i0; i < i1 && !st; ++i) {
            const gptq_host_problem_t &q = problems[i];
            st = check(cudaMemcpyAsync(q.y_host, q.y_stage, (size_t)q.M * q.N * sizeof(__half), cudaMemcpyDeviceToHost, pipe->out));
        }
        if (!st) st = check(cudaEventRecord(ev_y[c], pipe->out));
        i0 = i1;
    }
    // join: `stream` finishes after the last copy of each direction, also after an error
    int st2 = check(cudaEventRecord(ev_start, pipe->in));
    if (!st2) st2 = check(cudaStreamWaitEvent(s, ev_start, 0));
    if (!st2) st2 = check(cudaEventRecord(ev_x[0], pipe->out));
    if (!st2) st2 = check(cudaStreamWaitEvent(s, ev_x[0], 0));
    return st ? st : st2;
}

extern "C" {

int gptq_gemm_host_batch(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index)
{
    return host_batch(problems, count, stream, bad_index, 0);
}

int gptq_gemm_host_batch_bf16(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index)
{
    return host_batch(problems, count, stream, bad_index, 1);
}

int gptq_gemm_host_batch_w8(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index)
{
    return host_batch(problems, count, stream, bad_index, 2);
}

// ---- self-test of the bounded waits ------------------------------------------------------------
// One thread waits (for at most `limit_ns`) on an mbarrier that nothing will ever complete, exactly as the
// matmul kernels wait, gives up, records the time-out in the status word and returns normally.
__global__ void wait_selftest_kernel(unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = smem_u32(&bar);
    mbar_init(b, 1);
    fence_barrier_init();
    mbar_wait_limited(b, 0, limit_ns);
}

int gptq_selftest_wait_timeout(unsigned int limit_us, void *stream)
{
    if (limit_us < 1 || limit_us > 1000000) return GPTQ_ERR_SHAPE;
    wait_selftest_kernel<<<1, 1, 0, (cudaStream_t)stream>>>((unsigned long long)limit_us * 1000ull);
    return record_cuda_error(cudaGetLastError());
}

int gptq_trace_reset(void *stream)
{
#ifdef GPTQ_TIMELINE
    static TraceRow blank[kTraceLaunches];
    for (int i = 0; i < kTraceLaunches; ++i) {
        blank[i].first_entry = blank[i].first_weight_issue = blank[i].first_wait_done = blank[i].first_data = ~0ull;
        blank[i].last_wait_done = blank[i].last_exit = blank[i].kernel_and_ctas = blank[i].last_entry = 0;
    }
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyToSymbolAsync(g_trace, blank, sizeof(blank), 0, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    return record_cuda_error(e);
#else
    (void)stream;
    return GPTQ_ERR_UNSUPPORTED;
#endif
}

int gptq_trace_read(unsigned long long *rows_out, int max_rows, void *stream)
{
#ifdef GPTQ_TIMELINE
    if (!rows_out || max_rows < 0) return GPTQ_ERR_NULL;
    const int n = max_rows < kTraceLaunches ? max_rows : kTraceLaunches;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyFromSymbolAsync(rows_out, g_trace, (size_t)n * sizeof(TraceRow), 0, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return record_cuda_error(e);
    return n;
#else
    (void)rows_out; (void)max_rows; (void)stream;
    return GPTQ_ERR_UNSUPPORTED;
#endif
}

int gptq_check_status(void *stream)
{
    cudaStream_t s = (cudaStream_t)stream;
    int status = 0;
    cudaError_t e = cudaMemcpyFromSymbolAsync(&status, g_device_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (status == kStatusOk) return GPTQ_OK;
    int zero = 0;
    e = cudaMemcpyToSymbolAsync(g_device_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return record_cuda_error(e);
    return status == kStatusLayoutMismatch ? GPTQ_ERR_LAYOUT : GPTQ_ERR_TIMEOUT;
}

}  // extern "C"
