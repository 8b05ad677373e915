// Streaming GPTQ matmul for small token counts (decode, M <= 64 per launch): HBM-bound.
//
// One launch covers all (panel, group) items of the layer; CTA c works through the contiguous
// item range [c*T/C, (c+1)*T/C) ("stream-K"), so every SM streams the same number of bytes no
// matter how N/128 compares with the SM count.  Per item a producer thread issues bulk copies
// (8 KB of packed weights, 256 B of scales, 64 B of zeros, one 256 B row of x per token) into
// a multi-stage shared-memory ring guarded by mbarriers.  Eight consumer warps each own 16
// columns: a lane reads its 16-byte chunk, turns nibbles into fp16 pairs with lop3 (1024+q or
// 64+q, exact), subtracts the matching zero constant as packed half2 (exact integer q - z) and
// feeds them as the 16-row A operand of mma.sync.m16n8k16 with the tokens as the 8-wide B
// operand.  The group's scale is applied to the fp32 group sum once per group, so the inner
// loop carries no multiply and the weights are never rounded to fp16.
//
// A panel whose K range is shared by several CTAs is finished through fp32 partial tiles in
// the workspace: every contributor stores its tile, takes a ticket, and the last one sums the
// tiles in CTA order (a fixed order, so results are reproducible) and writes fp16 y once.
#pragma once
#include "gptq_common.cuh"

namespace gptq {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kStreamKThreads = kConsumerThreads + 32;
constexpr int kXRowBytes = 320;   // 256 B of x + 64 B pad: conflict-free 128-bit fragment loads
constexpr int kBarrierBytes = 128;

__host__ __device__ constexpr int streamk_stage_bytes(int MT)
{
    return kItemWBytes + kItemSBytes + kItemZBytes + MT * 8 * kXRowBytes;
}

// Stream-K index arithmetic (shared by the kernel, the planner and the host-side introspection
// entry points).  T items are cut into C contiguous ranges; CTA c owns [begin(c), begin(c+1)).
__host__ __device__ inline int sk_range_begin(long long T, int C, int c) { return (int)((long long)c * T / C); }
// the CTA whose range contains item t
__host__ __device__ inline int sk_owner(long long T, int C, long long t) { return (int)(((t + 1) * C - 1) / T); }

struct StreamKArgs {
    const __half *x;        // [M, K] (already in sorted row order for act-order layers)
    const uint8_t *qweight; // tiled
    const uint8_t *scales;
    const uint8_t *qzeros;
    __half *y;              // [M, N]
    float *partials;        // [ctas][2][M][128]
    int *tickets;           // [panels], zero between launches
    int M, N, K, G;
    int items;              // T = panels * G
    int stages;
};

template <int MT>
__global__ void __launch_bounds__(kStreamKThreads, 1) streamk_kernel(const StreamKArgs a)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int kStage = streamk_stage_bytes(MT);
    constexpr int kOffS = kItemWBytes, kOffZ = kOffS + kItemSBytes, kOffX = kOffZ + kItemZBytes;

    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t bar_full = smem_base;                  // stages x 8 B
    const uint32_t bar_empty = smem_base + 64;            // stages x 8 B
    const uint32_t ring = smem_base + kBarrierBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int C = gridDim.x, c = blockIdx.x;
    const long long T = a.items;
    const int t0 = sk_range_begin(T, C, c), t1 = sk_range_begin(T, C, c + 1);
    const int stages = a.stages;

    if (threadIdx.x == kConsumerThreads) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, kConsumerWarps);
        }
        fence_barrier_init();
        fence_proxy_async();
    }
    // token rows beyond M stay zero for the whole kernel (the bulk copies never touch them)
    {
        const int zero_rows = MT * 8 - a.M;   // rows a.M .. MT*8-1 of every stage
        const int vec_per_row = kXRowBytes / 16;
        for (int i = threadIdx.x; i < stages * zero_rows * vec_per_row; i += kStreamKThreads) {
            int s = i / (zero_rows * vec_per_row), rem = i % (zero_rows * vec_per_row);
            int row = a.M + rem / vec_per_row, v = rem % vec_per_row;
            *reinterpret_cast<uint4 *>(smem_raw + kBarrierBytes + s * kStage + kOffX + row * kXRowBytes + v * 16) =
                make_uint4(0, 0, 0, 0);
        }
    }
    __syncthreads();
    pdl_launch_dependents();

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        const uint64_t policy = l2_policy_evict_first();
        const uint32_t meta_bytes = kItemWBytes + kItemSBytes + kItemZBytes;
        const int n_items = t1 - t0;
        const int n_pre = n_items < stages ? n_items : stages;
        auto issue_weights = [&](int t, int s) {
            uint32_t dst = ring + s * kStage, bar = bar_full + 8 * s;
            mbar_expect_tx(bar, meta_bytes);
            bulk_g2s_hint(dst, a.qweight + (size_t)t * kItemWBytes, kItemWBytes, bar, policy);
            bulk_g2s_hint(dst + kOffS, a.scales + (size_t)t * kItemSBytes, kItemSBytes, bar, policy);
            bulk_g2s_hint(dst + kOffZ, a.qzeros + (size_t)t * kItemZBytes, kItemZBytes, bar, policy);
        };
        // weights never depend on earlier work in the stream: fill the ring before waiting on it
        if (lane == 0)
            for (int i = 0; i < n_pre; ++i) issue_weights(t0 + i, i);
        pdl_wait();
        int s = 0, round = 0;
        bool ok = true;
        for (int it = 0; it < n_items && ok; ++it) {
            const int t = t0 + it;
            const uint32_t bar = bar_full + 8 * s;
            if (lane == 0) {
                if (it >= stages) {
                    ok = mbar_wait(bar_empty + 8 * s, (uint32_t)((round - 1) & 1));
                    if (ok) issue_weights(t, s);
                }
                if (ok) mbar_arrive_expect_tx(bar, (uint32_t)a.M * 256u);
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (ok) {
                const int grp = t % a.G;
                const uint32_t dst = ring + s * kStage + kOffX;
                for (int m = lane; m < a.M; m += 32)
                    bulk_g2s(dst + m * kXRowBytes, a.x + (size_t)m * a.K + (size_t)grp * kGroup, 256, bar);
            }
            if (++s == stages) { s = 0; ++round; }
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    pdl_wait();
    const int g = lane >> 2, t4 = lane & 3;
    const uint32_t w_off = warp * kUnitBytes + lane * 16;
    const uint32_t s_off = kOffS + (warp * 16 + 2 * g) * 2;
    const uint32_t z_off = kOffZ + warp * 8 + g;
    const uint32_t x_off = kOffX + g * kXRowBytes + t4 * 16;
    constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, MAGIC_LO = 0x64006400u, MAGIC_HI = 0x54005400u;

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;

    int s = 0;
    uint32_t phase = 0;
    int p = t0 / a.G, grp = t0 % a.G;
    int seg_first_grp = grp;
    const int first_panel = p;
    __shared__ int s_last;

    bool ok = true;   // false after a wait gave up: keep taking part in barriers, skip the data
    for (int t = t0; t < t1; ++t) {
        const uint32_t st = ring + s * kStage;
        if (ok) ok = mbar_wait(bar_full + 8 * s, phase);   // on failure: stale data, status word set

        const uint4 wq0 = lds128(st + w_off);
        const uint4 wq1 = lds128(st + kBlockWBytes + w_off);
        const uint32_t sc = lds32(st + s_off);
        const uint32_t zb = lds8(st + z_off);
        const uint32_t zA = zb & 15u, zB = zb >> 4;
        const uint32_t zloA = (zA * 0x00010001u) | MAGIC_LO, zhiA = (zA * 0x00100010u) | MAGIC_HI;
        const uint32_t zloB = (zB * 0x00010001u) | MAGIC_LO, zhiB = (zB * 0x00100010u) | MAGIC_HI;

        float accg[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) accg[mt][i] = 0.f;

#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {
            const uint4 wq = blk ? wq1 : wq0;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                uint32_t wA = j ? wq.y : wq.x, wB = j ? wq.w : wq.z;
                const uint32_t a0 = hsub2_u32(lop3_and_or(wA, LO, MAGIC_LO), zloA);
                const uint32_t a2 = hsub2_u32(lop3_and_or(wA, HI, MAGIC_HI), zhiA);
                const uint32_t a1 = hsub2_u32(lop3_and_or(wB, LO, MAGIC_LO), zloB);
                const uint32_t a3 = hsub2_u32(lop3_and_or(wB, HI, MAGIC_HI), zhiB);
                wA >>= 8;
                wB >>= 8;
                const uint32_t c0 = hsub2_u32(lop3_and_or(wA, LO, MAGIC_LO), zloA);
                const uint32_t c2 = hsub2_u32(lop3_and_or(wA, HI, MAGIC_HI), zhiA);
                const uint32_t c1 = hsub2_u32(lop3_and_or(wB, LO, MAGIC_LO), zloB);
                const uint32_t c3 = hsub2_u32(lop3_and_or(wB, HI, MAGIC_HI), zhiB);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const uint4 xb = lds128(st + x_off + mt * 8 * kXRowBytes + (blk * 64 + j * 32) * 2);
                    mma_m16n8k16(accg[mt], a0, a1, a2, a3, xb.x, xb.y);
                    mma_m16n8k16(accg[mt], c0, c1, c2, c3, xb.z, xb.w);
                }
            }
        }
        // release the stage, then fold the group sum into the running sum with the group's scale
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * s);
        if (++s == stages) { s = 0; phase ^= 1u; }

        const float2 sf = __half22float2(*reinterpret_cast<const __half2 *>(&sc));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            acc[mt][0] = fmaf(sf.x, accg[mt][0], acc[mt][0]);
            acc[mt][1] = fmaf(sf.x, accg[mt][1], acc[mt][1]);
            acc[mt][2] = fmaf(sf.y, accg[mt][2], acc[mt][2]);
            acc[mt][3] = fmaf(sf.y, accg[mt][3], acc[mt][3]);
        }

        const bool seg_end = (grp == a.G - 1) || (t == t1 - 1);
        if (seg_end) {
            const int col = warp * 16 + g;
            if (seg_first_grp == 0 && grp == a.G - 1) {
                // this CTA saw the panel's whole K range: round once and store
                __half *yp = a.y + (size_t)p * kPanel + col;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = mt * 8 + 2 * t4 + (i & 1);
                        if (m < a.M) yp[(size_t)m * a.N + 8 * (i >> 1)] = __float2half_rn(acc[mt][i]);
                    }
            } else {
                const int slot = (p == first_panel) ? 0 : 1;
                float *pp = a.partials + ((size_t)(c * 2 + slot) * a.M) * kPanel + col;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = mt * 8 + 2 * t4 + (i & 1);
                        if (m < a.M) pp[(size_t)m * kPanel + 8 * (i >> 1)] = acc[mt][i];
                    }
                __threadfence();
                named_bar_sync(1, kConsumerThreads);
                // contributors of panel p: the CTAs that own its first and last item, and all between
                const long long first_item = (long long)p * a.G, last_item = first_item + a.G - 1;
                const int c_first = sk_owner(T, C, first_item), c_last = sk_owner(T, C, last_item);
                if (threadIdx.x == 0) {
                    const int old = atomicAdd(a.tickets + p, 1);
                    s_last = (old == c_last - c_first);
                }
                named_bar_sync(1, kConsumerThreads);
                if (s_last) {
                    __threadfence();
                    for (int idx = threadIdx.x; idx < a.M * kPanel; idx += kConsumerThreads) {
                        const int m = idx / kPanel, cc_col = idx % kPanel;
                        float sum = 0.f;
                        for (int cc = c_first; cc <= c_last; ++cc) {
                            const int cc_first_panel = sk_range_begin(T, C, cc) / a.G;
                            const int cc_slot = (cc_first_panel == p) ? 0 : 1;
                            sum += __ldcg(a.partials + ((size_t)(cc * 2 + cc_slot) * a.M + m) * kPanel + cc_col);
                        }
                        a.y[(size_t)m * a.N + (size_t)p * kPanel + cc_col] = __float2half_rn(sum);
                    }
                    if (threadIdx.x == 0) a.tickets[p] = 0;   // ready for the next launch
                }
                named_bar_sync(1, kConsumerThreads);   // s_last is reused by the next segment
            }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
            seg_first_grp = 0;
        }
        if (++grp == a.G) { grp = 0; ++p; }
    }
}

inline int streamk_m_tile(int m_rows) { return m_rows <= 8 ? 1 : m_rows <= 16 ? 2 : m_rows <= 32 ? 4 : 8; }

StreamKPlan plan_streamk(int m_rows, int N, int K, int sm_count)
{
    StreamKPlan pl{};
    const int MT = streamk_m_tile(m_rows);
    const int G = K / kGroup, panels = N / kPanel;
    const int stage = streamk_stage_bytes(MT);
    // MT <= 2 keeps two CTAs per SM (<= 113 registers per thread, ~110 KB of ring each); wider
    // token tiles need more registers, so they run one CTA per SM with a deeper ring.
    const int ctas_per_sm = MT <= 2 ? 2 : 1;
    const int ring_budget = (ctas_per_sm == 2 ? 110 : 220) * 1024 - kBarrierBytes;
    int stages = ring_budget / stage;
    if (stages > 8) stages = 8;
    pl.m_tile = MT * 8;
    pl.stages = stages;
    pl.items = panels * G;
    const int max_ctas = sm_count * ctas_per_sm;
    pl.ctas = pl.items < max_ctas ? pl.items : max_ctas;
    pl.smem_bytes = kBarrierBytes + stages * stage;
    // panels that are not covered by a single CTA
    int split = 0;
    const long long T = pl.items, C = pl.ctas;
    for (int p = 0; p < panels; ++p) {
        const long long first_item = (long long)p * G, last_item = first_item + G - 1;
        if (sk_owner(T, (int)C, first_item) != sk_owner(T, (int)C, last_item)) ++split;
    }
    pl.split_panels = split;
    pl.partial_bytes = split ? (size_t)pl.ctas * 2 * m_rows * kPanel * sizeof(float) : 0;
    pl.ticket_bytes = (size_t)panels * sizeof(int);
    return pl;
}

template <int MT>
static int launch_streamk_mt(const StreamKArgs &args, const StreamKPlan &plan, cudaStream_t s)
{
    static int configured_smem[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (dev < 0 || dev >= 64) return GPTQ_ERR_UNSUPPORTED;
    if (configured_smem[dev] < plan.smem_bytes) {
        e = cudaFuncSetAttribute(streamk_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e != cudaSuccess) return record_cuda_error(e);
        e = cudaFuncSetAttribute(streamk_kernel<MT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return record_cuda_error(e);
        configured_smem[dev] = plan.smem_bytes;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)plan.ctas);
    cfg.blockDim = dim3(kStreamKThreads);
    cfg.dynamicSmemBytes = (size_t)plan.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return record_cuda_error(cudaLaunchKernelEx(&cfg, streamk_kernel<MT>, args));
}

int launch_streamk(const __half *x, const void *qweight, const void *qzeros, const void *scales, __half *y,
                   int M, int N, int K, const StreamKPlan &plan, float *partials, int *tickets, cudaStream_t s)
{
    StreamKArgs args;
    args.x = x;
    args.qweight = (const uint8_t *)qweight;
    args.scales = (const uint8_t *)scales;
    args.qzeros = (const uint8_t *)qzeros;
    args.y = y;
    args.partials = partials;
    args.tickets = tickets;
    args.M = M;
    args.N = N;
    args.K = K;
    args.G = K / kGroup;
    args.items = plan.items;
    args.stages = plan.stages;
    switch (plan.m_tile) {
    case 8: return launch_streamk_mt<1>(args, plan, s);
    case 16: return launch_streamk_mt<2>(args, plan, s);
    case 32: return launch_streamk_mt<4>(args, plan, s);
    case 64: return launch_streamk_mt<8>(args, plan, s);
    default: return GPTQ_ERR_UNSUPPORTED;
    }
}

}  // namespace gptq
