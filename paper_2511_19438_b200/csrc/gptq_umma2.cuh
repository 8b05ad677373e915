// Prefill GPTQ matmul on CTA pairs: the tcgen05 kernel of gptq_umma.cuh with cta_group::2.
//
// Two CTAs of a cluster (two SMs) share one MMA of shape 256 x 256 x 16: CTA r owns weight panel
// 2 t + r (its 128 rows of the A operand, dequantised into its own tensor memory, and its 128 lanes
// of the accumulator) and loads only tokens [128 r, 128 r + 128) of the 256-token x tile; the
// tensor cores of the pair read both halves of the B operand from the two shared memories.  Per
// flop this halves the x traffic from L2 to shared memory, which is what bounds the single-CTA
// kernel, and halves the dequantisation work per MMA cycle.
//
// Synchronisation across the pair uses no multicast load: every CTA's TMA completes on its own
// mbarriers; the dequant warps of both CTAs arrive (cluster scope) on the LEADER's a_full barrier
// after they have waited for their own stage - so an arrival says "my A stage is in tensor memory
// and my half of the x tile has landed"; the leader's MMA thread issues tcgen05.mma.cta_group::2
// and hands slots back to both CTAs with tcgen05.commit ... multicast::cluster.
#pragma once
#include "gptq_umma.cuh"

namespace gptq {

constexpr int kUmma2Threads = 320;     // TMA warp, MMA/TMEM warp, two sets of four dequant warps
constexpr int kUmma2Tok = 256;         // tokens per pair tile (128 loaded by each CTA)
constexpr int kUmma2AStages = 8;
constexpr uint32_t kUmma2Cols = 512;   // accumulator 256 + A ring 8 x 32
constexpr int kUmma2StageBytes = 2 * (kUmma2Tok / 2) * 128 + 2 * kUmmaWBlockBytes;   // one K group: two x half-tiles + 8 KB of W

__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_slot, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// arrives on the barrier at this shared-memory offset in every CTA of `cta_mask` once all tcgen05
// operations issued so far by this thread have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"(cta_mask)
        : "memory");
}
__device__ __forceinline__ void umma_f16_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on a barrier of another CTA of the cluster, given its cluster-window address.  Default semantics
// (as the tensor-memory hand-off needs no more: the data is ordered by tcgen05.wait::st and
// tcgen05.fence::before_thread_sync on this side and tcgen05.fence::after_thread_sync on the other); an
// explicit .release.cluster here stalls the arriving thread for about 1100 cycles.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__global__ void __launch_bounds__(kUmma2Threads, 1)
umma2_kernel(const UmmaArgs a, const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map)
{
    extern __shared__ uint8_t smem_raw[];
    constexpr int kHalfTok = kUmma2Tok / 2;                 // tokens whose x rows this CTA loads
    // ring slot = one K group: [x half-tile of block 0][x half-tile of block 1][8 KB of packed weights]
    constexpr int kXTile = kHalfTok * 128, kStage = kUmma2StageBytes, kOffW = 2 * kXTile;
    constexpr uint32_t kAcol = kUmma2Tok;                  // accumulator first, then the A ring
    constexpr int NA = kUmma2AStages, SETS = 2;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // full[s]: this CTA's TMA data of ring slot s has landed; a_full (the leader's copy is used): the A stage of a block
    // is in tensor memory in both CTAs; done[b mod 16] (in both CTAs, by a multicast commit): the pair's MMAs of block b
    // have completed - the block's ring slot (with its group's second block) and its A stage may be overwritten
    const uint32_t bar_full = base, bar_afull = base + 128, bar_done = base + 320;
    const uint32_t bar_dfull = base + 256, tmem_slot = base + 264;
    const uint32_t ring = base + 1024;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NS = a.stages;
    const int ptiles = a.N / kPanel / 2;
    const int pair = blockIdx.x >> 1, rank = blockIdx.x & 1;             // cluster = CTAs 2 pair, 2 pair + 1
    const int mt = pair / ptiles, p = (pair - mt * ptiles) * 2 + rank;   // this CTA's weight panel
    const int m0 = mt * kUmma2Tok;
    const int NB = a.K / kUmmaBlockK;
    const uint32_t flags = __ldg(&a.trailer->flags);   // needed by the dequant warps only; asked for first to hide the round trip

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(bar_full + 8 * s, 1);
        for (int s = 0; s < kUmmaDoneRing; ++s) mbar_init(bar_done + 8 * s, 1);
        for (int s = 0; s < NA; ++s) {
            mbar_init(bar_afull + 8 * s, kUmmaDequantWarps);           // leader's copy is used: its four warps arrive, the
                                                                       // peer's four send 4 bytes each (transaction count)
        }
        mbar_init(bar_dfull, 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kUmma2Cols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    // both CTAs' barriers exist before anything arrives on them from the other CTA
    cluster_arrive_release();
    cluster_wait_acquire();
    tc_fence_after_sync();
    const uint32_t tmem_base = lds32(tmem_slot);
    pdl_launch_dependents();

    const int G = a.G;
    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer (one thread per CTA)
        if (lane == 0) {
            tma_prefetch_descriptor(&w_map);
            tma_prefetch_descriptor(&x_map);
            constexpr uint32_t kWBytes = 2 * kUmmaWBlockBytes, kXBytes = 2 * kXTile;
            const int n_pre = G < NS ? G : NS;
            for (int i = 0; i < n_pre; ++i) {                // weights do not depend on earlier kernels
                mbar_expect_tx(bar_full + 8 * i, kWBytes);
                tma_load_2d(ring + i * kStage + kOffW, &w_map, 0, (2 * G * p + 2 * i) * 64, bar_full + 8 * i);
            }
            pdl_wait();
            // as in the single-CTA kernel: a refill is one wait (the pair's MMAs of the slot's previous group are
            // done, which also means its weights were read), one arrive-and-expect and two copies
            int s = 0;
            for (int i = 0; i < G; ++i) {
                const uint32_t bar = bar_full + 8 * s, st = ring + s * kStage;
                if (i >= NS) {
                    const int c = 2 * (i - NS) + 1;
                    if (!mbar_wait(bar_done + 8 * (c & (kUmmaDoneRing - 1)), (uint32_t)((c / kUmmaDoneRing) & 1))) break;
                    mbar_arrive_expect_tx(bar, kXBytes + kWBytes);
                    tma_load_2d(st + kOffW, &w_map, 0, (2 * G * p + 2 * i) * 64, bar);
                } else {
                    mbar_arrive_expect_tx(bar, kXBytes);
                }
                // this CTA's half of the token tile: rows m0 + 128 rank .. + 127 (rows >= M read as zero), both K64 tiles
                tma_load_3d(st, &x_map, 0, m0 + rank * kHalfTok, 2 * i, bar);
                if (++s == NS) s = 0;
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issue (one thread of the leader CTA)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = umma_idesc_f16(256, kUmma2Tok);
            int s = 0, sa = 0;
            uint32_t pha = 0;
            bool ok = true;
            for (int b = 0; b < NB && ok; ++b) {
                // both CTAs' A stages written - which implies that both halves of the x tile have landed, since the
                // dequant warps waited for their slot before they wrote
                ok = mbar_wait_cluster(bar_afull + 8 * sa, pha);
                if (!ok) break;
                tc_fence_after_sync();
                const uint64_t bdesc = umma_desc_k_major_sw128(ring + s * kStage + (b & 1) * kXTile);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_f16_ts_pair(tmem_base, tmem_base + kAcol + sa * 32 + kk * 8, bdesc + (uint64_t)(kk * 2), idesc,
                                     (uint32_t)((b | kk) != 0));
                umma_commit_pair(bar_done + 8 * (b & (kUmmaDoneRing - 1)), 3);   // both CTAs: block b has been multiplied
                if ((b & 1) && ++s == NS) s = 0;
                if (++sa == NA) { sa = 0; pha ^= 1u; }
            }
            umma_commit_pair(bar_dfull, 3);
        }
    } else {
        // ---------------------------------------------------------------- dequant warps, then epilogue
        const int q = warp & 3;                 // the 32 TMEM lanes this warp may touch
        const int set = (warp - 2) >> 2;        // which K groups: set, set + 2, ...
        const int n = 32 * q + lane;            // weight column inside the panel = TMEM lane
        const int u = n >> 4, g = n & 7, h = (n >> 3) & 1;
        uint32_t w_rd[4];
#pragma unroll
        for (int t4 = 0; t4 < 4; ++t4) w_rd[t4] = kOffW + (u * 8 + g) * 64 + ((uint32_t)(t4 ^ (g >> 1)) << 4) + 8 * h;
        // scale and zero point of the lane's column: straight from L2, one group ahead
        const uint8_t *s_gl = a.scales + (size_t)p * G * kItemSBytes + (16 * u + 2 * g + h) * 2;
        const uint8_t *z_gl = a.qzeros + (size_t)p * G * kItemZBytes + 8 * u + g;
        auto load_sz = [&](int gg, uint32_t &sc, uint32_t &zb) {
            sc = __ldcg(reinterpret_cast<const unsigned short *>(s_gl + (size_t)gg * kItemSBytes));
            zb = __ldcg(z_gl + (size_t)gg * kItemZBytes);
        };
        uint32_t sc_next = 0, zb_next = 0;
        if (set < G) load_sz(set, sc_next, zb_next);
        constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, MAGIC_LO = 0x64006400u, MAGIC_HI = 0x54005400u;
        // The peer's warps signal the leader's a_full barrier with a fire-and-forget 4-byte st.async that is counted
        // on the barrier's transaction count (a remote mbarrier.arrive holds the issuing thread up for hundreds of
        // cycles); the leader's warp 0 of the set arms those 16 bytes with its own arrival.
        const uint32_t leader_afull = map_to_cluster_rank(bar_afull, 0);
        const uint32_t leader_slot = map_to_cluster_rank(base + 512 + 4 * warp, 0);
        int b = 2 * set;
        int s = set % NS, sa = b % NA;
        uint32_t ph = (uint32_t)(set / NS) & 1u;
        uint32_t s2 = 0, zlo = MAGIC_LO, zhi = MAGIC_HI;
        const uint32_t z_add = flags & kFormatZerosMinusOne;   // stored zero points one too small
        // this kernel has no fused gate/up epilogue: a layer tiled for one is multiplied but not stored, and reported
        const bool layout_ok = (flags & (kFormatGateUp | kFormatBf16)) == 0;   // fp16, plain column order only
        if (!layout_ok && threadIdx.x == 64) atomicMax(&g_device_status, (int)kStatusLayoutMismatch);
        bool ok = true;
        for (; b < NB && ok; b += ((b & 1) ? 2 * SETS - 1 : 1)) {
            const uint32_t st = ring + s * kStage;
            if ((b & 1) == 0) {
                // a set skips the other set's slots: its parity wait on a slot is unambiguous once the slot's previous
                // refill is known to have landed, i.e. that group's last block has been multiplied
                const int c = b - 2 * NS + 1;
                if (c > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_done + 8 * (c & (kUmmaDoneRing - 1)), (uint32_t)((c / kUmmaDoneRing) & 1)));
                ok = ok && __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, ph));   // warp-uniform
                if (!ok) break;
                s2 = sc_next * 0x00010001u;
                const uint32_t z = (h ? (zb_next >> 4) : (zb_next & 15u)) + z_add;
                zlo = (z * 0x00010001u) | MAGIC_LO;
                zhi = (z * 0x00100010u) | MAGIC_HI;
                if (b + 2 * SETS < NB) load_sz((b >> 1) + SETS, sc_next, zb_next);   // this set's next group
            }
            const uint32_t wb = st + (b & 1) * kUmmaWBlockBytes;
            uint2 wv[4];
#pragma unroll
            for (int t4 = 0; t4 < 4; ++t4) wv[t4] = lds64(wb + w_rd[t4]);
            uint32_t r[32];
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int t4 = 0; t4 < 4; ++t4) {
                    uint32_t w = jj ? wv[t4].y : wv[t4].x;       // rows 32 jj + 8 t4 + (0..7), TMEM columns 16 jj + 4 t4 + (0..3)
                    uint32_t *o = r + 16 * jj + 4 * t4;
                    o[0] = hmul2_u32(hsub2_u32(lop3_and_or(w, LO, MAGIC_LO), zlo), s2);
                    o[1] = hmul2_u32(hsub2_u32(lop3_and_or(w, HI, MAGIC_HI), zhi), s2);
                    w >>= 8;
                    o[2] = hmul2_u32(hsub2_u32(lop3_and_or(w, LO, MAGIC_LO), zlo), s2);
                    o[3] = hmul2_u32(hsub2_u32(lop3_and_or(w, HI, MAGIC_HI), zhi), s2);
                }
            if (b >= NA) {     // the stage's previous block b - NA must have been multiplied
                ok = __all_sync(0xffffffffu, mbar_wait(bar_done + 8 * ((b - NA) & (kUmmaDoneRing - 1)), (uint32_t)(((b - NA) / kUmmaDoneRing) & 1)));
                if (!ok) break;
                tc_fence_after_sync();
            }
            tmem_st_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + kAcol + sa * 32, r);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                // "my A stage and my x half are ready" to the leader
                if (rank == 0) {
                    if (q == 0) mbar_arrive_expect_tx(bar_afull + 8 * sa, 4 * kUmmaDequantWarps);
                    else mbar_arrive(bar_afull + 8 * sa);
                } else {
                    st_async_f32(leader_slot, 0.f, leader_afull + 8 * sa);
                }
            }
            const int step = (b & 1) ? 2 * SETS - 1 : 1;   // to this set's next block
            if (b & 1) {                                   // and to its next group's ring slot
                s += SETS;
                while (s >= NS) { s -= NS; ph ^= 1u; }
            }
            sa += step;
            while (sa >= NA) sa -= NA;
        }
        // ---- epilogue: lane n of this CTA's accumulator holds y[m0 .. m0+256, 128 p + n]
        pdl_wait();
        ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_dfull, 0));
        if (ok) tc_fence_after_sync();
        ok = ok && layout_ok;
        {
            // as in the single-CTA kernel: each set's four warps turn a 32-token chunk around through the idle ring
            // and write whole 128-byte lines of y; every warp takes part in the named barriers
            const uint32_t stg = ring + (uint32_t)(set * (32 * kPanel * 2));
            const int bar_id = 1 + set;
            const int tq = 32 * q + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < kUmma2Tok; c0 += 32) {
                if (m0 + c0 >= a.M) break;
                if (((c0 >> 5) & 1) != set) continue;       // the two warp sets share the token chunks
                if (ok) {
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + c0, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        sts_f16(stg + (uint32_t)(i * (kPanel * 2) + n * 2), __float2half_rn(__uint_as_float(r[i])));
                }
                named_bar_sync(bar_id, 128);
                if (ok) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int piece = tq + 128 * t, row = piece >> 4, c16 = piece & 15;
                        const int m = m0 + c0 + row;
                        if (m < a.M) {
                            const uint4 v = lds128(stg + (uint32_t)piece * 16u);
                            *reinterpret_cast<uint4 *>(a.y + (size_t)m * a.N + (size_t)p * kPanel + c16 * 8) = v;
                        }
                    }
                }
                named_bar_sync(bar_id, 128);
            }
        }
    }
    // neither CTA may free tensor memory or exit while the pair's MMAs or the peer's arrivals can still touch it
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();
    cluster_wait_acquire();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kUmma2Cols);
    }
}

struct Umma2Plan {
    int stages;
    int ctas;        // 2 * (panel pairs) * (256-token tiles)
    int smem_bytes;
};

inline bool umma2_applicable(int M, int N) { return M >= 256 && (N / kPanel) % 2 == 0; }

inline Umma2Plan plan_umma2(int M, int N, int K)
{
    Umma2Plan pl{};
    const int stage = kUmma2StageBytes;
    int stages = (227 * 1024 - 1024 - 2048) / stage;
    if (stages > 7) stages = 7;                               // fewer than 16 blocks in the ring (the done barriers)
    if (stages > K / kGroup) stages = K / kGroup;
    pl.stages = stages;
    pl.ctas = (N / kPanel) * ((M + kUmma2Tok - 1) / kUmma2Tok);
    pl.smem_bytes = 2048 + stages * stage;
    const int floor_one_per_sm = (227 * 1024) / 2 + 512;     // one CTA per SM: the pair owns all tensor memory
    if (pl.smem_bytes < floor_one_per_sm) pl.smem_bytes = floor_one_per_sm;
    return pl;
}

int launch_umma2(const __half *x, const void *qweight, const void *qzeros, const void *scales, __half *y, int M, int N,
                 int K, const Umma2Plan &plan, cudaStream_t s)
{
    UmmaArgs args;
    args.scales = (const uint8_t *)scales;
    args.qzeros = (const uint8_t *)qzeros;
    args.y = y;
    args.M = M;
    args.N = N;
    args.K = K;
    args.G = K / kGroup;
    args.S = 1;
    args.stages = plan.stages;
    args.fuse = 0;
    args.bias = nullptr;
    args.residual = nullptr;
    args.trace_slot = -1;
    args.out_index = nullptr;
    args.trailer = reinterpret_cast<const TiledTrailer *>((const uint8_t *)qzeros + tiled_zero_bytes(N, K, kGroup));
    CUtensorMap w_map, x_map;
    const uint64_t w_rows = (uint64_t)K * N / 2 / 64;
    int st = make_tensor_map_2d(&w_map, CU_TENSOR_MAP_DATA_TYPE_UINT32, qweight, 16, w_rows, 64, 16, 128,
                                CU_TENSOR_MAP_SWIZZLE_64B);
    if (st) return st;
    // x as K / 64 tiles of [M rows, 64 k]; a box is the two tiles of a K group, one CTA's half (128 rows) of the token tile
    st = make_tensor_map_ktiles(&x_map, x, (uint64_t)K, (uint64_t)M, kUmma2Tok / 2, 2);
    if (st) return st;
    static int configured_smem[64] = {};
    const int cfg_st = ensure_dynamic_smem((const void *)umma2_kernel, configured_smem, plan.smem_bytes);
    if (cfg_st) return cfg_st;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)plan.ctas);
    cfg.blockDim = dim3(kUmma2Threads);
    cfg.dynamicSmemBytes = (size_t)plan.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return record_cuda_error(cudaLaunchKernelEx(&cfg, umma2_kernel, args, w_map, x_map));
}

}  // namespace gptq
