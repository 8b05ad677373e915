// Decode / small-batch GPTQ matmul (M <= 64 per launch): HBM-bound streaming with split-K inside a
// thread-block cluster.
//
// A CTA owns one 128-column panel and a contiguous range of its K groups; the S CTAs that share a
// panel form one cluster (S = 1..8, chosen so that panels * S fills the SMs once).  A producer
// thread streams the CTA's items (8 KB of packed weights, 256 B of scales, 64 B of zeros, one
// swizzled tensor-map tile of x per K64 block) through a shared-memory ring guarded by
// mbarriers; weights are fetched before griddepcontrol.wait, so they overlap the previous kernel.
// Eight consumer warps each own 16 columns: a lane reads its 16-byte chunk, turns nibbles into
// fp16 pairs with lop3 (1024+q or 64+q, exact), subtracts the zero as packed half2 (exact integer
// q - z) and feeds them as the 16-row A operand of mma.sync.m16n8k16, tokens as the 8-wide B
// operand.  The group's scale multiplies the fp32 group sum once per group.
//
// The K-partials of a panel never touch global memory: CTA r owns columns [128 r / S, 128 (r+1) / S);
// every CTA sends each owner its slice of its fp32 tile with st.async into the owner's shared
// memory (counted in bytes on the owner's mbarrier), and each owner, once all S slices have landed,
// sums them in rank order (a fixed order: results are reproducible), rounds once to fp16 and
// stores y.  The only cluster-wide barrier is split around the main loop (arrive after the
// barriers are armed, wait before the first send), so no CTA waits for a slower neighbour.
#pragma once
#include "gptq_common.cuh"
#include "gptq_tma.cuh"
#include "gptq_streamk.cuh"   // ring geometry (streamk_stage_bytes, token_row_of_slot, thread counts)

namespace gptq {

__device__ __forceinline__ void cluster_arrive_release()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire()
{
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cluster_rank(uint32_t local_addr, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    return remote;
}
// fire-and-forget 4-byte store into another CTA's shared memory; the 4 bytes are counted on that CTA's mbarrier
__device__ __forceinline__ void st_async_f32(uint32_t cluster_addr, float v, uint32_t cluster_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(cluster_addr), "r"(__float_as_uint(v)), "r"(cluster_bar)
                 : "memory");
}
__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded like mbar_wait, but observing arrivals and stores from other CTAs of the cluster
__device__ __noinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity)
{
    const uint64_t start = global_timer_ns();
    for (;;) {
        for (int it = 0; it < 256; ++it)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (global_timer_ns() - start > kWaitLimitNs) break;
    }
    atomicMax(&g_device_status, (int)kStatusWaitTimeout);
    return false;
}

__device__ __forceinline__ void sts_f32(uint32_t addr, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

struct SplitKArgs {
    const uint8_t *qweight; // tiled
    const uint8_t *scales;
    const uint8_t *qzeros;
    __half *y;              // [M, N]
    int M, N, K, G;
    int S;                  // CTAs per panel = cluster size
    int stages;
    const TiledTrailer *trailer;   // behind the tiled zero points
    int fuse;               // 1: y[M, N / 2] = silu(gate) * up of a layer tiled with its column halves interleaved
    const __half *bias;     // fp16 [N] added to every row of y, or nullptr (not with fuse)
    const __half *residual; // fp16 [M, N] added to y, or nullptr (not with fuse); may be y itself
    int trace_slot;         // row of the launch timeline, or -1
    const int32_t *out_index; // with fuse: output column i is stored at column out_index[i] (nullptr: at i)
    // split-K column slices: the panel is one run of 128 columns, or with fuse two runs of 64 (gate, up); within a run
    // owner q finishes columns [lo(q), lo(q + 1)), lo(q) = q * run / S (byte q of slice_lo, q < 8; lo(S) = run);
    // slice_max = the widest slice
    unsigned long long slice_lo;
    int slice_max;
};

// silu(g) * u in fp32
__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.f + __expf(-g)) * u; }

struct SplitKPlan {
    int m_tile;     // 8 or 16
    int sub;        // quantisation groups per 128-row item: 128 / group_size
    int S;
    int stages;
    int ctas;       // panels * S
    int smem_bytes;
};

// The 8-row, group-128 instantiation compiles to 56 registers, which plan_splitk counts on for four resident CTAs; the
// timeline build's extra code would push it over, so there the bound is stated (a stated bound of 4 in the normal build
// made the compiler choose 52 registers and a 1-2 % slower schedule).
#ifdef GPTQ_TIMELINE
constexpr int kSplitKWideCtas = 4;
#else
constexpr int kSplitKWideCtas = 3;
#endif
template <int MT, int SUB, bool BF = false>
__global__ void __launch_bounds__(kStreamKThreads, (MT == 1 && SUB == 1) ? kSplitKWideCtas : 3)
splitk_kernel(const SplitKArgs a, const __grid_constant__ CUtensorMap x_map)
{
    extern __shared__ uint8_t smem_raw[];
    constexpr int kStage = streamk_stage_bytes(MT, SUB);
    constexpr int kXTile = MT * 1024;                       // one K64 tile of x
    constexpr int kOffW = streamk_x_bytes(MT), kOffS = kOffW + kItemWBytes, kOffZ = kOffS + SUB * kItemSBytes;

    // the layer's format flags are needed late (first item, epilogue): ask for them first, so that the round trip to
    // HBM hides behind the set-up
    const uint32_t flags = __ldg(&a.trailer->flags);
    if (threadIdx.x == 0) {
        GPTQ_TRACE_MIN(a.trace_slot, first_entry);
        GPTQ_TRACE_MAX(a.trace_slot, last_entry);
        if (blockIdx.x == 0) {
            GPTQ_TRACE_SET(a.trace_slot, kernel_and_ctas, (1ull << 32) | gridDim.x);
        }
    }
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_full = smem_base;                  // stages x 8 B
    const uint32_t bar_empty = smem_base + 64;            // stages x 8 B
    const uint32_t bar_recv = smem_base + 128;
    const uint32_t ring = smem_base + kRingOffset;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = a.S;
    const int p = blockIdx.x / S, rank = blockIdx.x - p * S;   // cluster = the S CTAs of panel p
    const int g0 = rank * a.G / S, g1 = (rank + 1) * a.G / S;  // this CTA's groups
    const int n_items = g1 - g0;
    const int t0 = p * a.G + g0;
    const int stages = a.stages;

    if (threadIdx.x == kConsumerThreads) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, kConsumerWarps);
        }
        mbar_init(bar_recv, 1);
        fence_barrier_init();
        fence_proxy_async();
        // split-K: S slices of a.M x (128 / S) floats will arrive in this CTA's receive buffer
        if (S > 1) {
            const int run = a.fuse ? 64 : kPanel;
            const int mine = (rank + 1 < S ? (int)((a.slice_lo >> (8 * (rank + 1))) & 255) : run) - (int)((a.slice_lo >> (8 * rank)) & 255);
            mbar_arrive_expect_tx(bar_recv, (uint32_t)(S * a.M * (a.fuse ? 2 : 1) * mine * 4));
        }
    }
    __syncthreads();
    if (S > 1) cluster_arrive_release();   // "my receive barrier is armed"; waited for before the first send
    pdl_launch_dependents();

    float acc[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[mt][i] = 0.f;
    const int g = lane >> 2, t4 = lane & 3;
    bool layout_ok = true;   // set by the consumer warps; the producer must not wait for the trailer

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer (one thread)
        if (lane == 0) {
            const uint64_t policy = l2_policy_evict_first();
            tma_prefetch_descriptor(&x_map);
            const uint32_t meta_bytes = kItemWBytes + SUB * (kItemSBytes + kItemZBytes);
            const int n_pre = n_items < stages ? n_items : stages;
            auto issue_weights = [&](int t, int s) {
                const uint32_t dst = ring + s * kStage, bar = bar_full + 8 * s;
                mbar_expect_tx(bar, meta_bytes);
                bulk_g2s_hint(dst + kOffW, a.qweight + (size_t)t * kItemWBytes, kItemWBytes, bar, policy);
                bulk_g2s_hint(dst + kOffS, a.scales + (size_t)t * (SUB * kItemSBytes), SUB * kItemSBytes, bar, policy);
                bulk_g2s_hint(dst + kOffZ, a.qzeros + (size_t)t * (SUB * kItemZBytes), SUB * kItemZBytes, bar, policy);
            };
            // weights never depend on earlier work in the stream: fill the ring before waiting on it
            GPTQ_TRACE_MIN(a.trace_slot, first_weight_issue);
            for (int i = 0; i < n_pre; ++i) issue_weights(t0 + i, i);
            pdl_wait();
            GPTQ_TRACE_MIN(a.trace_slot, first_wait_done);
            GPTQ_TRACE_MAX(a.trace_slot, last_wait_done);
            int s = 0, round = 0;
            for (int it = 0; it < n_items; ++it) {
                const uint32_t bar = bar_full + 8 * s;
                if (it >= stages) {
                    if (!mbar_wait(bar_empty + 8 * s, (uint32_t)((round - 1) & 1))) break;
                    issue_weights(t0 + it, s);
                }
                // the group's activations for all token rows: two swizzled K64 tiles, rows >= M read as zero
                mbar_arrive_expect_tx(bar, (uint32_t)streamk_x_bytes(MT));
                const uint32_t dst = ring + s * kStage;
                const int k0 = (g0 + it) * kGroup;
                tma_load_2d(dst, &x_map, k0, 0, bar);
                tma_load_2d(dst + kXTile, &x_map, k0 + 64, 0, bar);
                if (++s == stages) { s = 0; ++round; }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        // weights-side data (no need to wait for earlier kernels); requested at the top of the kernel
        const uint32_t z_add = flags & kFormatZerosMinusOne;
        // a layer tiled for the fused gate/up epilogue must be used with it, and only with it: otherwise nothing is
        // stored and the status word says so
        layout_ok = ((flags & kFormatGateUp) != 0) == (a.fuse != 0) && ((flags & kFormatBf16) != 0) == BF;
        if (!layout_ok && threadIdx.x == 0) atomicMax(&g_device_status, (int)kStatusLayoutMismatch);
        pdl_wait();
        const int r = token_row_of_slot(g);
        const uint32_t w_off = kOffW + warp * kUnitBytes + lane * 16;
        const uint32_t s_off = kOffS + (warp * 16 + 2 * g) * 2;
        const uint32_t z_off = kOffZ + warp * 8 + g;
        // x fragment of k chunk (4j + t4) for token slot g: row r of the swizzled tile
        const uint32_t x_off0 = r * 128 + ((uint32_t)(t4 ^ r) << 4);          // j = 0
        const uint32_t x_off1 = r * 128 + ((uint32_t)((4 + t4) ^ r) << 4);    // j = 1
        int s = 0;
        uint32_t phase = 0;
        bool ok = true;   // false after a wait gave up: keep taking part in barriers, skip the data
        for (int it = 0; it < n_items; ++it) {
            const uint32_t st = ring + s * kStage;
            if (ok) ok = mbar_wait(bar_full + 8 * s, phase);   // on failure: stale data, status word set
            if (it == 0 && threadIdx.x == 0) GPTQ_TRACE_MIN(a.trace_slot, first_data);

            ItemSums<MT, SUB> sums;
            consume_item<MT, SUB, BF>(st, w_off, s_off, z_off, x_off0, x_off1, z_add, sums);
            // release the stage, then fold the group sums into the running sums with the groups' scales
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * s);
            if (++s == stages) { s = 0; phase ^= 1u; }
            fold_item<MT, SUB, BF>(acc, sums);
        }
    }

    // accumulator i of tile mt: weight column col + 8*(i>>1), token slot 2*t4 + (i&1)
    const int col = warp * 16 + g;
    const int m_lo = token_row_of_slot(2 * t4), m_hi = token_row_of_slot(2 * t4 + 1);
    // what the epilogue adds to the fp32 sum of output (m, n) before the one rounding: bias[n] + residual[m][n]
    // (read after griddepcontrol.wait: an earlier kernel may have produced them; the thread that reads an element of
    // the residual is the one that writes the same element of y, so the two may be one buffer)
    auto addend = [&](int m, int n) {
        float v = 0.f;
        if (a.bias) v += __half2float(a.bias[n]);
        if (a.residual) v += __half2float(a.residual[(size_t)m * a.N + n]);
        return v;
    };
    if (S == 1) {
        if (warp < kConsumerWarps && layout_ok) {
            if (!a.fuse) {
                __half *yp = a.y + (size_t)p * kPanel + col;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int m = mt * 8 + ((i & 1) ? m_hi : m_lo);
                        if (m < a.M) store_out16<BF>(yp + (size_t)m * a.N + 8 * (i >> 1), acc[mt][i] + addend(m, p * kPanel + col + 8 * (i >> 1)));
                    }
            } else {
                // warps 4-7 hold the up columns of the gate columns of warps 0-3: hand them over through the
                // (unused) receive buffer, [token][64 columns] floats
                const uint32_t hand = ring + (uint32_t)a.stages * kStage;
                if (warp >= 4) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int m = mt * 8 + ((i & 1) ? m_hi : m_lo);
                            if (m < a.M) sts_f32(hand + (uint32_t)(m * 64 + col - 64 + 8 * (i >> 1)) * 4u, acc[mt][i]);
                        }
                }
                named_bar_sync(1, kConsumerThreads);
                if (warp < 4) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int m = mt * 8 + ((i & 1) ? m_hi : m_lo);
                            if (m < a.M) {
                                const float up = lds_f32(hand + (uint32_t)(m * 64 + col + 8 * (i >> 1)) * 4u);
                                const int oc = p * 64 + col + 8 * (i >> 1);
                                store_out16<BF>(a.y + (size_t)m * (a.N / 2) + (a.out_index ? a.out_index[oc] : oc),
                                                silu_mul(acc[mt][i], up));
                            }
                        }
                }
            }
        }
        if (threadIdx.x == 0) GPTQ_TRACE_MAX(a.trace_slot, last_exit);
        return;
    }

    // ---- split-K: send each owner its column slice, then finish the own slice ------------------------
    __syncwarp();
    cluster_wait_acquire();                 // every CTA of the cluster has armed its receive barrier
    if (warp < kConsumerWarps) {
        // One run of 128 columns, or with the fused epilogue two runs of 64 (gate | up).  Within a run owner q finishes
        // columns [lo(q), lo(q + 1)); S is any value from 2 to 8, so the slices may differ by one column.
        // Receive buffer of an owner: [sender rank][token row][run][slice_max] floats.
        const int hsh = a.fuse ? 6 : 7, hmask = (1 << hsh) - 1;            // log2(run), column within the run
        const int runs = a.fuse ? 2 : 1;
        const int hwmax = a.slice_max, wstride = runs * hwmax;
        const uint32_t recv = ring + (uint32_t)a.stages * kStage;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = mt * 8 + ((i & 1) ? m_hi : m_lo);
                if (m < a.M) {
                    const int c = col + 8 * (i >> 1), cc = c & hmask;
                    const int q = ((cc + 1) * S - 1) >> hsh;                 // the q with lo(q) <= cc < lo(q + 1)
                    const int pos = (c >> hsh) * hwmax + cc - (int)((a.slice_lo >> (8 * q)) & 255);
                    const uint32_t off = (uint32_t)((rank * a.M + m) * wstride + pos) * 4u;
                    st_async_f32(map_to_cluster_rank(recv + off, (uint32_t)q), acc[mt][i],
                                 map_to_cluster_rank(bar_recv, (uint32_t)q));
                }
            }
        if (mbar_wait_cluster(bar_recv, 0) && layout_ok) {
            auto slice_sum = [&](int m, int j) {   // rank order
                float v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    v[q] = q < S ? lds_f32(recv + (uint32_t)((q * a.M + m) * wstride + j) * 4u) : 0.f;
                float sum = 0.f;
#pragma unroll
                for (int q = 0; q < 8; ++q) sum += v[q];
                return sum;
            };
            const int lo = (int)((a.slice_lo >> (8 * rank)) & 255);
            const int hw = (rank + 1 < S ? (int)((a.slice_lo >> (8 * (rank + 1))) & 255) : (1 << hsh)) - lo;   // at most 64 columns per run
            // threads as [rows per pass][jw columns], jw the power of two that holds the slice (8 .. 64)
            const int jsh = hw <= 8 ? 3 : hw <= 16 ? 4 : hw <= 32 ? 5 : 6;
            const int j = threadIdx.x & ((1 << jsh) - 1);
            if (j < hw) {
                for (int m = threadIdx.x >> jsh; m < a.M; m += kConsumerThreads >> jsh) {
                    if (!a.fuse) {
                        const int n = p * kPanel + lo + j;
                        store_out16<BF>(a.y + (size_t)m * a.N + n, slice_sum(m, j) + addend(m, n));
                    } else {
                        const int oc = p * 64 + lo + j;
                        store_out16<BF>(a.y + (size_t)m * (a.N / 2) + (a.out_index ? a.out_index[oc] : oc),
                                        silu_mul(slice_sum(m, j), slice_sum(m, hwmax + j)));
                    }
                }
            }
        }
        if (threadIdx.x == 0) GPTQ_TRACE_MAX(a.trace_slot, last_exit);
    }
}

// Resident CTAs per SM by token tile: registers and ring size are set so that three CTAs of the
// narrowest tile fit, which lets the next kernel's first CTAs start (and prefetch weights) early.
__host__ __device__ constexpr int splitk_ctas_per_sm(int MT) { return 3; }

// Picks the cluster size S in {1, 2, 4, 8} with the smallest estimated time among those whose
// panels * S CTAs are all resident at once (falling back to all S if none is).  The estimate is
// the busiest SM's item count at the measured per-SM item rate, bounded below by one CTA's own
// serial rate, plus the cluster reduction when S > 1 (hundredths of a microsecond; only ratios
// matter).  Shared memory is then padded so that exactly ceil(CTAs / SMs) CTAs fit on an SM: the
// cluster scheduler otherwise packs three CTAs onto some SMs and leaves others empty.
SplitKPlan plan_splitk(int m_rows, int N, int K, int group_size, int sm_count)
{
    SplitKPlan pl{};
    const int MT = streamk_m_tile(m_rows);
    const int G = K / kGroup, panels = N / kPanel;
    pl.sub = kGroup / group_size;
    const int stage = streamk_stage_bytes(MT, pl.sub);
    // The 8-row, group-128 instantiation needs 56 registers, so four of its CTAs fit an SM, and for it cluster sizes 3
    // and 6 are candidates too (5 and 7 measured badly: clusters of that size often find no room): the 7B gate_up
    // (172 panels) takes 13.8 us with 3 x 172 CTAs against 14.9 with 2 x 172, the 13B qkv 12.6 us with S = 4 against 13.9
    // with S = 2.  The other instantiations keep powers of two and three CTAs per SM.
    const bool wide = (MT == 1 && pl.sub == 1);
    const int cps_max = wide ? 4 : splitk_ctas_per_sm(MT);
    static const int kSizesWide[] = {1, 2, 3, 4, 6, 8}, kSizes[] = {1, 2, 4, 8};
    const int *sizes = wide ? kSizesWide : kSizes;
    const int n_sizes = wide ? 6 : 4;
    int best_S = 1;
    long long best_t = -1;
    for (int pass = 0; pass < 2 && best_t < 0; ++pass) {
        for (int si = 0; si < n_sizes; ++si) {
            const int S = sizes[si];
            if (S > G || (pass == 1 && S > 1)) break;          // nothing fits at once: several waves, no split
            const long long ctas = (long long)panels * S, ipc = (G + S - 1) / S;
            const long long on_busiest_sm = (ctas + sm_count - 1) / sm_count;
            if (pass == 0 && on_busiest_sm > cps_max) continue;
            // per item and SM: about 0.33 us with two resident CTAs, 0.28 with three or four (measured, hundredths of a us)
            const long long per_item = !wide ? 30 : on_busiest_sm >= 3 ? 28 : 33;
            const long long serial = ipc * 45, shared = on_busiest_sm * ipc * per_item;
            const long long t = (serial > shared ? serial : shared) + (S > 1 ? 100 : 0);
            if (best_t < 0 || t < best_t) { best_t = t; best_S = S; }
        }
    }
    const int S = best_S;
    const int items_per_cta = (G + S - 1) / S;
    int per_sm = (panels * S + sm_count - 1) / sm_count;
    if (per_sm > cps_max) per_sm = cps_max;
    const int smem_cap = (227 * 1024) / per_sm - 1024;                 // per_sm CTAs fit ...
    const int smem_floor = (227 * 1024) / (per_sm + 1) + 512;          // ... per_sm + 1 do not
    const int recv_bytes = MT * 4480;   // receive buffer of the split-K exchange, after the ring: rows x (S slices: at most 140) floats
    int stages = (smem_cap - 2 * kRingOffset - recv_bytes) / stage;
    if (stages > 8) stages = 8;
    if (stages > items_per_cta) stages = items_per_cta;
    pl.m_tile = MT * 8;
    pl.S = S;
    pl.stages = stages;
    pl.ctas = panels * S;
    pl.smem_bytes = 2 * kRingOffset + stages * stage + recv_bytes;
    if (pl.smem_bytes < smem_floor) pl.smem_bytes = smem_floor;
    return pl;
}

template <int MT, int SUB, bool BF>
static int launch_splitk_mt(const SplitKArgs &args, const CUtensorMap &x_map, const SplitKPlan &plan, cudaStream_t s)
{
    static int configured_smem[64] = {};
    const int cfg_st = ensure_dynamic_smem((const void *)splitk_kernel<MT, SUB, BF>, configured_smem, plan.smem_bytes);
    if (cfg_st) return cfg_st;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)plan.ctas);
    cfg.blockDim = dim3(kStreamKThreads);
    cfg.dynamicSmemBytes = (size_t)plan.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[3];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)plan.S;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    // Let the hardware balance clusters over the SMs.  With the default policy, in a chain of launches of different
    // shapes a cluster of 8 now and then found no room until another cluster of its own grid had finished (seen in the
    // launch timeline: a 256-CTA launch taking 15 instead of 8.6 us); with this preference a decode layer's four matmuls
    // take 37.6 instead of 40.6 us.  (In the tcgen05 kernel's split-K launches it measured slightly slower: not set there.)
    attr[2].id = cudaLaunchAttributeClusterSchedulingPolicyPreference;
    attr[2].val.clusterSchedulingPolicyPreference = cudaClusterSchedulingPolicyLoadBalancing;
    cfg.attrs = attr;
    cfg.numAttrs = 3;
    return record_cuda_error(cudaLaunchKernelEx(&cfg, splitk_kernel<MT, SUB, BF>, args, x_map));
}

int launch_splitk(const __half *x, const void *qweight, const void *qzeros, const void *scales, __half *y,
                  int M, int N, int K, const SplitKPlan &plan, int fuse, const __half *bias, const __half *residual,
                  const int32_t *out_index, int bf16, cudaStream_t s)
{
    SplitKArgs args;
    args.qweight = (const uint8_t *)qweight;
    args.scales = (const uint8_t *)scales;
    args.qzeros = (const uint8_t *)qzeros;
    args.y = y;
    args.M = M;
    args.N = N;
    args.K = K;
    args.G = K / kGroup;
    args.S = plan.S;
    args.stages = plan.stages;
    args.fuse = fuse;
    args.bias = bias;
    args.residual = residual;
    args.trace_slot = next_trace_slot();
    args.out_index = out_index;
    {
        const int run = fuse ? 64 : kPanel;
        args.slice_lo = 0;
        for (int q = 0; q < 8; ++q) args.slice_lo |= (unsigned long long)(q < plan.S ? q * run / plan.S : run) << (8 * q);
        args.slice_max = (run + plan.S - 1) / plan.S;
    }
    args.trailer = reinterpret_cast<const TiledTrailer *>((const uint8_t *)qzeros + tiled_zero_bytes(N, K, kGroup / plan.sub));
    // x as a 2-D tensor [M rows, K halves]; a box is one K64 tile of all token rows of the CTA tile
    CUtensorMap x_map;
    int st = make_tensor_map_2d(&x_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, x, (uint64_t)K, (uint64_t)M,
                                (uint64_t)K * sizeof(__half), 64, (uint32_t)plan.m_tile, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st) return st;
    // (the tensor map only moves 16-bit words and zero-fills rows beyond M: the same for fp16 and bfloat16)
    switch ((bf16 ? 1000 : 0) + plan.m_tile * 10 + plan.sub) {
    case 81: return launch_splitk_mt<1, 1, false>(args, x_map, plan, s);
    case 82: return launch_splitk_mt<1, 2, false>(args, x_map, plan, s);
    case 84: return launch_splitk_mt<1, 4, false>(args, x_map, plan, s);
    case 161: return launch_splitk_mt<2, 1, false>(args, x_map, plan, s);
    case 162: return launch_splitk_mt<2, 2, false>(args, x_map, plan, s);
    case 164: return launch_splitk_mt<2, 4, false>(args, x_map, plan, s);
    case 1081: return launch_splitk_mt<1, 1, true>(args, x_map, plan, s);
    case 1082: return launch_splitk_mt<1, 2, true>(args, x_map, plan, s);
    case 1084: return launch_splitk_mt<1, 4, true>(args, x_map, plan, s);
    case 1161: return launch_splitk_mt<2, 1, true>(args, x_map, plan, s);
    case 1162: return launch_splitk_mt<2, 2, true>(args, x_map, plan, s);
    case 1164: return launch_splitk_mt<2, 4, true>(args, x_map, plan, s);
    default: return GPTQ_ERR_UNSUPPORTED;
    }
}

}  // namespace gptq
