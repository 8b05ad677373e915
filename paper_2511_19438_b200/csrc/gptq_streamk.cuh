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
#include "gptq_tma.cuh"

namespace gptq {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kStreamKThreads = kConsumerThreads + 32;
constexpr int kRingOffset = 1024;   // barriers live below the ring; the ring is 1024-byte aligned

// A ring stage: [x: two K64 tiles of MT*8 token rows x 128 B, 128-byte swizzled by the tensor-map load]
//               [8192 B packed weights][256 B scales][64 B zeros], rounded up to 1024 B.
__host__ __device__ constexpr int streamk_x_bytes(int MT) { return MT * 2048; }
__host__ __device__ constexpr int streamk_stage_bytes(int MT, int SUB = 1)
{
    return (streamk_x_bytes(MT) + kItemWBytes + SUB * (kItemSBytes + kItemZBytes) + 1023) & ~1023;
}

// Stream-K index arithmetic (shared by the kernel, the planner and the host-side introspection
// entry points).  T items are cut into C contiguous ranges; CTA c owns [begin(c), begin(c+1)).
__host__ __device__ inline int sk_range_begin(long long T, int C, int c) { return (int)((long long)c * T / C); }
// the CTA whose range contains item t
__host__ __device__ inline int sk_owner(long long T, int C, long long t) { return (int)(((t + 1) * C - 1) / T); }

// MMA token slot n (0..7) -> token row inside an 8-row tile: bit reversal.  With this choice the
// eight lanes of a quarter warp (two token slots x four k chunks) read eight different 16-byte
// chunks of the swizzled x tile, so the 128-bit fragment loads are bank-conflict free.
__host__ __device__ constexpr int token_row_of_slot(int n) { return ((n & 1) << 2) | (n & 2) | ((n >> 2) & 1); }

// The arithmetic of one (panel, 128-row) item for one consumer warp, shared by the mma.sync kernels.  The lane reads
// its two 16-byte chunks of packed weights from ring stage `st`; for each of the item's SUB quantisation groups
// (128 / group_size: the whole item, a K64 block, or half of one) it reads the scale pair and the zero byte of its
// columns, turns nibbles into exact fp16 integers q - z (z_add = 1 when the stored zero points are one too small),
// multiplies them with the stage's x tiles and folds the fp32 group sums into `acc` with the group's scales.
// The stage may be released once `consume_item` has returned; `fold_item` needs registers only.
template <int MT, int SUB>
struct ItemSums {
    float g[SUB][MT][4];
    uint32_t sc[SUB];
};
// BF: x and the scales are bfloat16 instead of fp16 (the exact integers q - z are built as bfloat16 too).
template <int MT, int SUB, bool BF = false>
__device__ __forceinline__ void consume_item(uint32_t st, uint32_t w_off, uint32_t s_off, uint32_t z_off,
                                             uint32_t x_off0, uint32_t x_off1, uint32_t z_add, ItemSums<MT, SUB> &out)
{
    constexpr int kXTile = MT * 1024;
    constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, MAGIC_LO = 0x64006400u, MAGIC_HI = 0x54005400u;
    const uint4 wq0 = lds128(st + w_off);
    const uint4 wq1 = lds128(st + kBlockWBytes + w_off);
    uint32_t zloA = 0, zhiA = 0, zloB = 0, zhiB = 0;
#pragma unroll
    for (int sub = 0; sub < SUB; ++sub)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) out.g[sub][mt][i] = 0.f;
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
        const uint4 wq = blk ? wq1 : wq0;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int q4 = blk * 2 + j;              // quarter of the item: 32 rows
            const int sub = q4 * SUB / 4;
            if (q4 * SUB % 4 == 0) {                 // first quarter of a group
                out.sc[sub] = lds32(st + s_off + sub * kItemSBytes);
                const uint32_t zb = lds8(st + z_off + sub * kItemZBytes);
                const uint32_t zA = (zb & 15u) + z_add, zB = (zb >> 4) + z_add;   // up to 16: still exact below
                if constexpr (BF) {
                    zero_constants<true>(zA, zloA, zhiA);
                    zero_constants<true>(zB, zloB, zhiB);
                } else {
                    zloA = (zA * 0x00010001u) | MAGIC_LO, zhiA = (zA * 0x00100010u) | MAGIC_HI;
                    zloB = (zB * 0x00010001u) | MAGIC_LO, zhiB = (zB * 0x00100010u) | MAGIC_HI;
                }
            }
            uint32_t wA = j ? wq.y : wq.x, wB = j ? wq.w : wq.z;
            if constexpr (BF) {
                uint32_t pA[4], pB[4];    // pairs of rows (0,1) (2,3) (4,5) (6,7) of columns g and g + 8
                nibble_pairs_minus_zero<true>(wA, zloA, zhiA, pA);
                nibble_pairs_minus_zero<true>(wB, zloB, zhiB, pB);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    const uint4 xb = lds128(st + blk * kXTile + mt * 1024 + (j ? x_off1 : x_off0));
                    mma_m16n8k16_bf16(out.g[sub][mt], pA[0], pB[0], pA[1], pB[1], xb.x, xb.y);
                    mma_m16n8k16_bf16(out.g[sub][mt], pA[2], pB[2], pA[3], pB[3], xb.z, xb.w);
                }
                continue;
            }
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
                const uint4 xb = lds128(st + blk * kXTile + mt * 1024 + (j ? x_off1 : x_off0));
                mma_m16n8k16(out.g[sub][mt], a0, a1, a2, a3, xb.x, xb.y);
                mma_m16n8k16(out.g[sub][mt], c0, c1, c2, c3, xb.z, xb.w);
            }
        }
    }
}
// folds the item's group sums into the running sums with each group's scales
template <int MT, int SUB, bool BF = false>
__device__ __forceinline__ void fold_item(float (&acc)[MT][4], const ItemSums<MT, SUB> &it)
{
#pragma unroll
    for (int sub = 0; sub < SUB; ++sub) {
        const float2 sf = pair_to_float2<BF>(it.sc[sub]);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            acc[mt][0] = fmaf(sf.x, it.g[sub][mt][0], acc[mt][0]);
            acc[mt][1] = fmaf(sf.x, it.g[sub][mt][1], acc[mt][1]);
            acc[mt][2] = fmaf(sf.y, it.g[sub][mt][2], acc[mt][2]);
            acc[mt][3] = fmaf(sf.y, it.g[sub][mt][3], acc[mt][3]);
        }
    }
}

struct StreamKArgs {
    const uint8_t *qweight; // tiled
    const uint8_t *scales;
    const uint8_t *qzeros;
    __half *y;              // [M, N]
    float *partials;        // [ctas][2][M][128]
    int *tickets;           // [panels], zero between launches
    int M, N, K, G;
    int items;              // T = panels * G
    int stages;
    const TiledTrailer *trailer;   // behind the tiled zero points: says whether the stored zero points are one too small
};

template <int MT>
__global__ void __launch_bounds__(kStreamKThreads, MT <= 2 ? 2 : 1)
streamk_kernel(const StreamKArgs a, const __grid_constant__ CUtensorMap x_map)
{
    extern __shared__ uint8_t smem_raw[];
    constexpr int kStage = streamk_stage_bytes(MT);
    constexpr int kXTile = MT * 1024;                       // one K64 tile of x
    constexpr int kOffW = streamk_x_bytes(MT), kOffS = kOffW + kItemWBytes, kOffZ = kOffS + kItemSBytes;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_full = smem_base;                  // stages x 8 B
    const uint32_t bar_empty = smem_base + 64;            // stages x 8 B
    const uint32_t ring = smem_base + kRingOffset;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int C = gridDim.x, c = blockIdx.x;
    const long long T = a.items;
    const int t0 = sk_range_begin(T, C, c), t1 = sk_range_begin(T, C, c + 1);
    const int stages = a.stages;
    __shared__ int s_last;
    const uint32_t flags = __ldg(&a.trailer->flags);   // needed by the consumers only; asked for first to hide the round trip

    if (threadIdx.x == kConsumerThreads) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, kConsumerWarps);
        }
        fence_barrier_init();
        fence_proxy_async();
    }
    __syncthreads();
    pdl_launch_dependents();

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer (one thread)
        if (lane != 0) return;
        const uint64_t policy = l2_policy_evict_first();
        tma_prefetch_descriptor(&x_map);
        const uint32_t meta_bytes = kItemWBytes + kItemSBytes + kItemZBytes;
        const int n_items = t1 - t0;
        const int n_pre = n_items < stages ? n_items : stages;
        auto issue_weights = [&](int t, int s) {
            const uint32_t dst = ring + s * kStage, bar = bar_full + 8 * s;
            mbar_expect_tx(bar, meta_bytes);
            bulk_g2s_hint(dst + kOffW, a.qweight + (size_t)t * kItemWBytes, kItemWBytes, bar, policy);
            bulk_g2s_hint(dst + kOffS, a.scales + (size_t)t * kItemSBytes, kItemSBytes, bar, policy);
            bulk_g2s_hint(dst + kOffZ, a.qzeros + (size_t)t * kItemZBytes, kItemZBytes, bar, policy);
        };
        // weights never depend on earlier work in the stream: fill the ring before waiting on it
        for (int i = 0; i < n_pre; ++i) issue_weights(t0 + i, i);
        pdl_wait();
        int s = 0, round = 0, grp = t0 % a.G;
        for (int it = 0; it < n_items; ++it) {
            const uint32_t bar = bar_full + 8 * s;
            if (it >= stages) {
                if (!mbar_wait(bar_empty + 8 * s, (uint32_t)((round - 1) & 1))) break;
                issue_weights(t0 + it, s);
            }
            // the group's activations for all token rows: two swizzled K64 tiles, rows >= M read as zero
            mbar_arrive_expect_tx(bar, (uint32_t)streamk_x_bytes(MT));
            const uint32_t dst = ring + s * kStage;
            tma_load_2d(dst, &x_map, grp * kGroup, 0, bar);
            tma_load_2d(dst + kXTile, &x_map, grp * kGroup + 64, 0, bar);
            if (++s == stages) { s = 0; ++round; }
            if (++grp == a.G) grp = 0;
        }
        return;
    }

    // -------------------------------------------------------------------- consumer warps
    const uint32_t z_add = flags & kFormatZerosMinusOne;   // weights-side data: no need to wait
    // this kernel has no fused gate/up epilogue: a layer tiled for one is computed but not stored, and reported
    const bool layout_ok = (flags & (kFormatGateUp | kFormatBf16)) == 0;   // fp16, plain column order only
    if (!layout_ok && threadIdx.x == 0) atomicMax(&g_device_status, (int)kStatusLayoutMismatch);
    pdl_wait();
    const int g = lane >> 2, t4 = lane & 3;
    const int r = token_row_of_slot(g);
    const uint32_t w_off = kOffW + warp * kUnitBytes + lane * 16;
    const uint32_t s_off = kOffS + (warp * 16 + 2 * g) * 2;
    const uint32_t z_off = kOffZ + warp * 8 + g;
    // x fragment of k chunk (4j + t4) for token slot g: row r of the swizzled tile
    const uint32_t x_off0 = r * 128 + ((uint32_t)(t4 ^ r) << 4);          // j = 0
    const uint32_t x_off1 = r * 128 + ((uint32_t)((4 + t4) ^ r) << 4);    // j = 1
    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;

    int s = 0;
    uint32_t phase = 0;
    int p = t0 / a.G, grp = t0 - p * a.G;
    int seg_first_grp = grp;
    const int first_panel = p;

    bool ok = true;   // false after a wait gave up: keep taking part in barriers, skip the data
    for (int t = t0; t < t1; ++t) {
        const uint32_t st = ring + s * kStage;
        if (ok) ok = mbar_wait(bar_full + 8 * s, phase);   // on failure: stale data, status word set

        ItemSums<MT, 1> sums;
        consume_item<MT, 1>(st, w_off, s_off, z_off, x_off0, x_off1, z_add, sums);
        // release the stage, then fold the group sum into the running sum with the group's scale
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * s);
        if (++s == stages) { s = 0; phase ^= 1u; }
        fold_item<MT, 1>(acc, sums);

        const bool seg_end = (grp == a.G - 1) || (t == t1 - 1);
        if (seg_end) {
            const int col = warp * 16 + g;
            // accumulator i of tile mt: weight column col + 8*(i>>1), token slot 2*t4 + (i&1)
            const int m_lo = token_row_of_slot(2 * t4), m_hi = token_row_of_slot(2 * t4 + 1);
            if (seg_first_grp == 0 && grp == a.G - 1) {
                // this CTA saw the panel's whole K range: round once and store
                __half *yp = a.y + (size_t)p * kPanel + col;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = mt * 8 + ((i & 1) ? m_hi : m_lo);
                        if (m < a.M && layout_ok) yp[(size_t)m * a.N + 8 * (i >> 1)] = __float2half_rn(acc[mt][i]);
                    }
            } else {
                const int slot = (p == first_panel) ? 0 : 1;
                float *pp = a.partials + ((size_t)(c * 2 + slot) * a.M) * kPanel + col;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = mt * 8 + ((i & 1) ? m_hi : m_lo);
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
                    // every contributor after the first starts inside this panel (slot 0); the first one
                    // starts inside it only if its range begins exactly at the panel's first item
                    const int slot_first = (sk_range_begin(T, C, c_first) >= first_item) ? 0 : 1;
                    const int nc = c_last - c_first + 1;
                    const size_t tile = (size_t)a.M * kPanel;
                    for (int idx = threadIdx.x; idx < a.M * kPanel; idx += kConsumerThreads) {
                        const float *src = a.partials + (size_t)c_first * 2 * tile + idx;
                        float sum = 0.f;
                        // fixed summation order (CTA order), eight loads in flight at a time
                        for (int c0 = 0; c0 < nc; c0 += 8) {
                            float v[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const int ci = c0 + u;
                                const int sl = (ci == 0) ? slot_first : 0;
                                v[u] = (ci < nc) ? __ldcg(src + (size_t)(ci * 2 + sl) * tile) : 0.f;
                            }
#pragma unroll
                            for (int u = 0; u < 8; ++u) sum += v[u];
                        }
                        const int m = idx / kPanel, cc_col = idx % kPanel;
                        if (layout_ok) a.y[(size_t)m * a.N + (size_t)p * kPanel + cc_col] = __float2half_rn(sum);
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
    const int ring_budget = (ctas_per_sm == 2 ? 112 : 224) * 1024 - 2 * kRingOffset;
    int stages = ring_budget / stage;
    if (stages > 8) stages = 8;
    pl.m_tile = MT * 8;
    pl.stages = stages;
    pl.items = panels * G;
    const int max_ctas = sm_count * ctas_per_sm;
    pl.ctas = pl.items < max_ctas ? pl.items : max_ctas;
    pl.smem_bytes = 2 * kRingOffset + stages * stage;   // barrier block + alignment slack + ring
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
static int launch_streamk_mt(const StreamKArgs &args, const CUtensorMap &x_map, const StreamKPlan &plan,
                             cudaStream_t s)
{
    static int configured_smem[64] = {};
    const int cfg_st = ensure_dynamic_smem((const void *)streamk_kernel<MT>, configured_smem, plan.smem_bytes);
    if (cfg_st) return cfg_st;
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
    return record_cuda_error(cudaLaunchKernelEx(&cfg, streamk_kernel<MT>, args, x_map));
}

int launch_streamk(const __half *x, const void *qweight, const void *qzeros, const void *scales, __half *y,
                   int M, int N, int K, const StreamKPlan &plan, float *partials, int *tickets, cudaStream_t s)
{
    StreamKArgs args;
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
    args.trailer = reinterpret_cast<const TiledTrailer *>((const uint8_t *)qzeros + tiled_zero_bytes(N, K, kGroup));
    // x as a 2-D tensor [M rows, K halves]; a box is one K64 tile of all token rows of the CTA tile
    CUtensorMap x_map;
    int st = make_tensor_map_2d(&x_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, x, (uint64_t)K, (uint64_t)M,
                                (uint64_t)K * sizeof(__half), 64, (uint32_t)plan.m_tile, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st) return st;
    switch (plan.m_tile) {
    case 8: return launch_streamk_mt<1>(args, x_map, plan, s);
    case 16: return launch_streamk_mt<2>(args, x_map, plan, s);
    case 32: return launch_streamk_mt<4>(args, x_map, plan, s);
    case 64: return launch_streamk_mt<8>(args, x_map, plan, s);
    default: return GPTQ_ERR_UNSUPPORTED;
    }
}

}  // namespace gptq
