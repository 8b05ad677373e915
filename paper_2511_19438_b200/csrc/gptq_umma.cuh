// Prefill GPTQ matmul (many tokens): tcgen05 tensor cores with the dequantisation fused in front
// of the MMA.
//
// Swap-AB: a CTA computes D[n, m] = sum_k W^T[n, k] x^T[k, m] for one 128-column panel (the MMA's
// M = 128 rows, one TMEM lane per weight column) and a tile of TOK tokens (the MMA's N).  x[M, K]
// row-major is already the K-major B operand, so it goes from global memory to swizzled shared
// memory by TMA and is read by the tensor core through a shared-memory descriptor.  The weights
// need arithmetic, so they take another road: TMA brings the packed weights of a K group of the
// panel (8 KB, 64-byte swizzle) to shared memory, two sets of four dequant warps (one warp per 32
// TMEM lanes, the sets taking alternate groups) read the eight words of "their" column per K64
// block, turn nibbles into fp16 with lop3 (1024+q / 64+q), subtract the zero (exact integer) and
// multiply by the group scale as packed half2 (scale and zero come straight from L2, one group
// ahead), and write the 64 fp16 values with tcgen05.st into a ring of A-operand stages in tensor
// memory.  One thread issues tcgen05.mma (kind::f16, A from TMEM, B from shared memory, fp32
// accumulator in TMEM); one tcgen05.commit per K64 block tells everybody that the block's ring
// slot and A stage are free again.  At the end of the K loop the dequant warps read the
// accumulator with tcgen05.ld, round once to fp16, turn each 32-token chunk around through the
// idle ring and store whole lines of y.
//
// The two single threads (TMA producer, MMA issue) pay 60-110 cycles for every instruction, so
// both loops are kept short: a ring refill is one wait, one arrive-and-expect, one weight copy and
// one 3-D x copy per K group; an MMA step is one wait, four MMAs and one commit per K64 block.
//
// Small problems split K over a thread-block cluster (partial tiles meet through distributed
// shared memory in rank order); when the tiles fill the SMs more than once, the partly filled
// last wave is launched separately with such a split.  Every wait is bounded.
#pragma once
#include "gptq_common.cuh"
#include "gptq_tma.cuh"
#include "gptq_splitk.cuh"   // cluster barrier and distributed-shared-memory helpers

namespace gptq {

// warp 0: TMA producer, warp 1: MMA issue + TMEM, then four dequant/epilogue warps per panel of the CTA
// (two sets of them, taking alternate K groups, when one warp per scheduler cannot keep up with the MMA)
// MMA-issuing warps: one thread pays 60-110 cycles for every instruction it issues (and more when its scheduler is
// shared with busy dequant warps).  With 64-token tiles each dequant warp set gets an issuing warp and an accumulator
// of its own, and the epilogue adds the accumulators (measured 0-6 % faster there; with 32-token tiles the third
// resident CTA that a single accumulator leaves room for is worth more).
__host__ __device__ constexpr int umma_issuers(int TOK, int SETS) { return (TOK == 64 && SETS == 2) ? 2 : 1; }
// warp 0: TMA producer; warps 1 .. ISS: MMA issue; then four dequant warps per panel and set
__host__ __device__ constexpr int umma_threads(int TOK, int NP, int SETS)
{
    return 32 * (1 + umma_issuers(TOK, SETS)) + 128 * NP * SETS;
}
constexpr int kUmmaDequantWarps = 4;     // per panel: one warp per 32 TMEM lanes
constexpr int kUmmaBlockK = 64;
constexpr int kUmmaWBlockBytes = 4096;   // packed weights of one K64 block of a panel
constexpr int kUmmaDoneRing = 16;        // "block multiplied" barriers, indexed by block number mod 16

// ---- tcgen05 wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_slot, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// arrives on the mbarrier once every tcgen05 operation issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor]; M, N and the operand types come from idesc
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 columns of 32 bits: thread t of the warp writes / reads lane (base + t), register i <-> column i
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,"
        "%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (what a tensor-map load with SWIZZLE_128B writes): groups of 8 rows are 1024
// bytes apart (stride byte offset), the leading byte offset is unused for swizzled K-major tiles.
__device__ __forceinline__ uint64_t umma_desc_k_major_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);          // start address, bits 0..13
    d |= (uint64_t)1 << 16;                                // leading byte offset (ignored), bits 16..29
    d |= (uint64_t)(1024 >> 4) << 32;                      // stride byte offset, bits 32..45
    d |= (uint64_t)1 << 46;                                // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                                // layout type: 128-byte swizzle
    return d;
}
// Instruction descriptor: fp16 A and B, both K-major, fp32 accumulator, MMA shape M x N (K = 16).
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N)
{
    return (1u << 4) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// the same with bfloat16 A and B: operand format fields (bits 7..9 and 10..12) 1 instead of 0
constexpr uint32_t kUmmaIdescBf16 = (1u << 7) | (1u << 10);

__device__ __forceinline__ void sts_f16(uint32_t addr, __half v)
{
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(__half_as_ushort(v)) : "memory");
}

__device__ __forceinline__ void sts_b16(uint32_t addr, unsigned short v)
{
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}

__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(addr)
                 : "memory");
    return v;
}

struct UmmaArgs {
    const uint8_t *scales;  // tiled
    const uint8_t *qzeros;  // tiled
    __half *y;              // [M, N]
    int M, N, K, G;
    int S;                  // CTAs that share one output tile along K (cluster size)
    int tile0;              // first output tile of this launch (a matmul may take a main and a tail launch)
    int stages;             // shared-memory ring depth
    const TiledTrailer *trailer;   // behind the tiled zero points
    int fuse;               // 1: y[M, N / 2] = silu(gate) * up of a layer tiled with its column halves interleaved
    const __half *bias;     // fp16 [N] added to every row of y, or nullptr (not with fuse)
    const __half *residual; // fp16 [M, N] added to y, or nullptr (not with fuse); may be y itself
    int trace_slot;         // row of the launch timeline, or -1
    const int32_t *out_index; // with fuse: output column i is stored at column out_index[i] (nullptr: at i)
};

// K64 blocks per ring slot of the single-CTA kernel: a whole K group (two blocks: fewer, larger copies for the
// producer thread) except for 128-token tiles, where two CTAs share an SM and group-sized slots would leave each
// a ring of only two
__host__ __device__ constexpr int umma_blocks_per_slot(int TOK) { return TOK == 128 ? 1 : 2; }
// one ring slot: x tile(s) and packed weights of each panel (scales and zeros do not pass through shared memory)
__host__ __device__ constexpr int umma_slot_bytes(int TOK, int NP)
{
    return (umma_blocks_per_slot(TOK) * (TOK * 128 + NP * kUmmaWBlockBytes) + 1023) & ~1023;
}
__host__ __device__ constexpr int umma_tmem_cols(int TOK, int NA, int NP, int ISS)
{
    // per panel: accumulators (TOK columns each) + A ring (32 columns = one K64 block per stage); a power of two >= 32
    int need = NP * (ISS * TOK + NA * 32), c = 32;
    while (c < need) c <<= 1;
    return c;
}

template <int TOK, int NA, int NP, int SETS, int SUB, bool BF = false>
__global__ void __launch_bounds__(umma_threads(TOK, NP, SETS), (NP > 1 || TOK > 128) ? 1 : TOK <= 32 ? 3 : 2)
umma_kernel(const UmmaArgs a, const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap x_map)
{
    extern __shared__ uint8_t smem_raw[];
    // the layer's format flags are needed by the dequant warps only: requested first, so that the round trip to HBM
    // hides behind the set-up
    const uint32_t flags = __ldg(&a.trailer->flags);
    if (threadIdx.x == 0) {
        GPTQ_TRACE_MIN(a.trace_slot, first_entry);
        GPTQ_TRACE_MAX(a.trace_slot, last_entry);
        if (blockIdx.x == 0) {
            GPTQ_TRACE_SET(a.trace_slot, kernel_and_ctas, (2ull << 32) | gridDim.x);
        }
    }
    constexpr int kStage = umma_slot_bytes(TOK, NP);
    // ring slot = BPS K64 blocks: [x tile of each block][W blocks of each panel]
    constexpr int BPS = umma_blocks_per_slot(TOK);
    constexpr int kXTile = TOK * 128;
    constexpr int kOffW = BPS * kXTile;
    constexpr int ISS = umma_issuers(TOK, SETS);
    constexpr int kFirstDq = 1 + ISS;                       // first dequant warp
    constexpr uint32_t kCols = umma_tmem_cols(TOK, NA, NP, ISS);
    constexpr uint32_t kAcol = NP * ISS * TOK;             // accumulators first, then the A rings (panel-major)

    // A warp set jumps 2 SETS - 1 blocks from one K group to its next.  Its parity wait on an A stage is only
    // unambiguous if that jump is no longer than the A ring: then the wait it passed for the previous block implies
    // that the stage's completion before the awaited one has already happened.
    static_assert(SETS == 1 || NA >= 2 * SETS - 1, "A ring too short for this many dequant warp sets");
    // With two issuers each dequant set must own its A stages (blocks b and b + NA belong to the same set), so that
    // an issuer sees every completion of the barriers it waits on.
    static_assert(umma_issuers(TOK, SETS) == 1 || NA == 2 * SETS, "issuers need A stages of their own");
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // full[s]: the TMA data of ring slot s has landed; a_full: an A stage has been written; done[b mod 16]: the MMAs
    // of K64 block b have completed (one tcgen05.commit per block tells the producer that the block's ring slot and
    // the dequant warps that its A stage may be overwritten).  A parity wait for block c must look at done[c mod 16]
    // before block c + 16 completes, so fewer than 16 blocks may be in the ring at once (the planner sees to that).
    const uint32_t bar_full = base, bar_afull = base + 128, bar_done = base + 320;
    const uint32_t bar_dfull = base + 256, tmem_slot = base + 264, bar_recv = base + 272;
    const uint32_t ring = base + 1024;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NS = a.stages;
    const int panels = a.N / kPanel;
    const int S = a.S;
    const int cl = blockIdx.x / S, rank = blockIdx.x - cl * S;          // cluster = the S CTAs of one tile
    const int tile = cl + a.tile0;
    const int ptiles = panels / NP;
    const int mt = tile / ptiles, p0 = (tile - mt * ptiles) * NP;       // first panel; neighbours share the x tile
    const int m0 = mt * TOK;
    const int g0 = rank * a.G / S, g1 = (rank + 1) * a.G / S;           // this CTA's K groups
    const int NB = 2 * (g1 - g0), b_first = 2 * g0;                     // its K64 blocks

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar_full + 8 * s, 1);
        }
        for (int s = 0; s < NP * NA; ++s) mbar_init(bar_afull + 8 * s, kUmmaDequantWarps);
        for (int s = 0; s < kUmmaDoneRing; ++s) mbar_init(bar_done + 8 * s, 1);
        mbar_init(bar_dfull, ISS);
        mbar_init(bar_recv, 1);
        fence_barrier_init();
        fence_proxy_async();
        // split-K: every CTA of the cluster (this one included) will push its partial sums of this CTA's 128 / S columns
        // for every 32-token chunk that holds rows of y
        if (S > 2) {
            const int rows = (a.M - m0) < TOK ? (a.M - m0) : TOK;
            mbar_arrive_expect_tx(bar_recv, (uint32_t)(S * ((rows + 31) & ~31) * (kPanel / S) * 4));
        }
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = lds32(tmem_slot);
    pdl_launch_dependents();
    bool layout_ok = true;   // set by the dequant warps; the producer and the MMA issuers must not wait for the trailer

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer (one thread)
        if (lane == 0) {
            tma_prefetch_descriptor(&w_map);
            tma_prefetch_descriptor(&x_map);
            constexpr uint32_t kXBytes = BPS * kXTile;
            const int NR = NB / BPS;                         // ring refills of this CTA
            constexpr uint32_t kWBytes = NP * BPS * kUmmaWBlockBytes;
            // the packed weights of refill i (scales and zeros are read by the dequant warps themselves)
            auto issue_w = [&](int i, int s) {
                const uint32_t st = ring + s * kStage, bar = bar_full + 8 * s;
                const int b = i * BPS;                       // first K64 block of the refill
#pragma unroll
                for (int j = 0; j < NP; ++j)
                    // packed weights viewed as rows of 64 bytes; block b of panel p starts at row (2 G p + b) * 64
                    tma_load_2d(st + kOffW + j * BPS * kUmmaWBlockBytes, &w_map, 0, (2 * a.G * (p0 + j) + b_first + b) * 64, bar);
            };
            const int n_pre = NR < NS ? NR : NS;
            GPTQ_TRACE_MIN(a.trace_slot, first_weight_issue);
            for (int i = 0; i < n_pre; ++i) {                // weights do not depend on earlier kernels
                mbar_expect_tx(bar_full + 8 * i, kWBytes);
                issue_w(i, i);
            }
            pdl_wait();
            GPTQ_TRACE_MIN(a.trace_slot, first_wait_done);
            GPTQ_TRACE_MAX(a.trace_slot, last_wait_done);
            // Every instruction of this thread (a wait, an expect, a copy) costs it about 0.1 us, which bounds
            // the kernel when there are many of them per byte, so a ring slot holds a whole K group where shared
            // memory allows and a refill is one wait, one arrive-and-expect and the copies.  The slot is free
            // once the MMAs of its previous refill's last block have completed: that also means that its packed
            // weights were read (the A stages those MMAs used were written from them).
            int s = 0;
            for (int i = 0; i < NR; ++i) {
                const uint32_t bar = bar_full + 8 * s, st = ring + s * kStage;
                if (i >= NS) {
                    const int c = (i - NS) * BPS + BPS - 1;
                    if (!mbar_wait(bar_done + 8 * (c & (kUmmaDoneRing - 1)), (uint32_t)((c / kUmmaDoneRing) & 1))) break;
                    mbar_arrive_expect_tx(bar, kXBytes + kWBytes);
                    issue_w(i, s);
                } else {
                    mbar_arrive_expect_tx(bar, kXBytes);
                }
                tma_load_3d(st, &x_map, 0, m0, b_first + i * BPS, bar);   // the refill's BPS x tiles in one copy
                if (++s == NS) s = 0;
            }
        }
    } else if (warp <= ISS) {
        // ---------------------------------------------------------------- MMA issue (one thread per issuing warp)
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_f16(128, TOK) | (BF ? kUmmaIdescBf16 : 0u);
            // Every instruction this thread issues costs it 60-110 cycles (a tcgen05.mma about 60, a commit
            // about 80, a barrier wait about 100 even when the barrier is ready), so the loop is kept to one wait
            // per panel, the four MMAs and one commit per K64 block.  It does not wait for the slot's TMA data
            // itself: the dequant warps did before they wrote the A stage, and their a_full arrival orders it.
            // With one issuer it takes the blocks in order; with two, issuer t takes the blocks of dequant set t
            // (K groups t, t + SETS, ...) and accumulates them in its own tensor-memory columns.
            const int t = ISS == 1 ? 0 : warp - 1;          // a constant for the single issuer: nothing to compute per MMA
            const int b_begin = ISS == 1 ? 0 : 2 * t;
            const uint32_t d_tmem = tmem_base + (uint32_t)(t * TOK);
            bool ok = true;
            // one block: wait for its A stage(s), four MMAs per panel, one commit (every extra instruction of this
            // thread shows in the prefill rate, so the bookkeeping below is kept incremental)
            auto issue_block = [&](int b, int s, int sa, uint32_t pha) {
                const uint64_t bdesc = umma_desc_k_major_sw128(ring + s * kStage + (b % BPS) * kXTile);
#pragma unroll
                for (int j = 0; j < NP; ++j) {
                    ok = mbar_wait(bar_afull + 8 * (j * NA + sa), pha);
                    if (!ok) return;
                    tc_fence_after_sync();
                    if (b == b_begin) GPTQ_TRACE_MIN(a.trace_slot, first_data);   // (nothing in a normal build)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)   // 16 k per MMA: 8 TMEM columns of A, 32 bytes of each x row
                        umma_f16_ts(d_tmem + j * ISS * TOK, tmem_base + kAcol + (j * NA + sa) * 32 + kk * 8,
                                    bdesc + (uint64_t)(kk * 2), idesc, (uint32_t)(b != b_begin || kk != 0));
                }
                umma_commit(bar_done + 8 * (b & (kUmmaDoneRing - 1)));     // this block's A stage(s) and x tile may be overwritten
            };
            if (ISS == 1) {
                int s = 0, sa = 0;
                uint32_t pha = 0;
                for (int b = 0; b < NB && ok; ++b) {
                    issue_block(b, s, sa, pha);
                    if ((b % BPS) == BPS - 1 && ++s == NS) s = 0;
                    if (++sa == NA) { sa = 0; pha ^= 1u; }
                }
            } else {
                // the blocks of dequant set t: K groups t, t + SETS, ...; A stage b mod NA, filled for the (b / NA)-th time
                int b = b_begin;
                int s = (b / BPS) % NS;
                while (b < NB && ok) {
                    issue_block(b, s, b % NA, (uint32_t)(b / NA) & 1u);
                    const int step = (b & 1) ? 2 * SETS - 1 : 1;   // to this issuer's next block
                    s += (b + step) / BPS - b / BPS;                // and to that block's ring slot
                    while (s >= NS) s -= NS;
                    b += step;
                }
            }
            if (b_begin < NB) umma_commit(bar_dfull);
            else mbar_arrive(bar_dfull);            // this issuer had no block
        }
    } else {
        // ---------------------------------------------------------------- dequant warps, then epilogue
        const int q = warp & 3;                 // the 32 TMEM lanes this warp may touch
        const int j = ((warp - kFirstDq) >> 2) % NP;   // which of the CTA's panels this warp dequantises
        const int set = ((warp - kFirstDq) >> 2) / NP; // and which K64 blocks: set, set + SETS, ...
        const int p = p0 + j;
        const int n = 32 * q + lane;            // weight column inside the panel = TMEM lane
        const int u = n >> 4, g = n & 7, h = (n >> 3) & 1;
        // the column's 8 bytes (two words: rows +0..7 and +32..39) in each of the four 16-byte chunks
        uint32_t w_rd[4];
#pragma unroll
        for (int t4 = 0; t4 < 4; ++t4) w_rd[t4] = kOffW + j * BPS * kUmmaWBlockBytes + (u * 8 + g) * 64 + ((uint32_t)(t4 ^ (g >> 1)) << 4) + 8 * h;
        // The column's scale and zero point of a group come straight from global memory (2 bytes and a nibble per
        // lane: 64 + 16 bytes per warp), fetched one group ahead into registers, which spares the producer thread two
        // copies per group.  In the tiled layout the pair (column, column + 8) is adjacent.
        // A 128-row item holds SUB quantisation groups (128 / group_size), each with its own scales and zeros.
        const uint8_t *s_gl = a.scales + ((size_t)p * a.G + g0) * (SUB * kItemSBytes) + (16 * u + 2 * g + h) * 2;
        const uint8_t *z_gl = a.qzeros + ((size_t)p * a.G + g0) * (SUB * kItemZBytes) + 8 * u + g;
        auto load_sz = [&](int gg, uint32_t (&sc)[SUB], uint32_t (&zb)[SUB]) {
            // through L2 only: this kernel may start while its predecessor still runs, and the buffers may have been
            // rewritten since an earlier kernel left lines of them in this SM's L1
#pragma unroll
            for (int sub = 0; sub < SUB; ++sub) {
                sc[sub] = __ldcg(reinterpret_cast<const unsigned short *>(s_gl + ((size_t)gg * SUB + sub) * kItemSBytes));
                zb[sub] = __ldcg(z_gl + ((size_t)gg * SUB + sub) * kItemZBytes);
            }
        };
        uint32_t sc_next[SUB], zb_next[SUB];
#pragma unroll
        for (int sub = 0; sub < SUB; ++sub) sc_next[sub] = zb_next[sub] = 0;
        if (2 * set < NB) load_sz(set, sc_next, zb_next);
        // (the format flags are looked at only now, with the first scales and zeros already on their way)
        const uint32_t z_add = flags & kFormatZerosMinusOne;   // stored zero points one too small
        // a layer tiled for the fused gate/up epilogue must be used with it, and only with it (else: nothing is stored)
        layout_ok = ((flags & kFormatGateUp) != 0) == (a.fuse != 0) && ((flags & kFormatBf16) != 0) == BF;
        if (!layout_ok && threadIdx.x == 32 * kFirstDq) atomicMax(&g_device_status, (int)kStatusLayoutMismatch);
        constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u, MAGIC_LO = 0x64006400u, MAGIC_HI = 0x54005400u;
        // set k takes groups k, k + SETS, ...: K64 blocks 2 gg and 2 gg + 1; block b lives in ring refill b / BPS
        int b = 2 * set;
        int s = (b / BPS) % NS, sa = b % NA;
        uint32_t ph = (uint32_t)((b / BPS) / NS) & 1u;
        uint32_t s2[SUB], zlo[SUB], zhi[SUB];
#pragma unroll
        for (int sub = 0; sub < SUB; ++sub) s2[sub] = 0, zlo[sub] = MAGIC_LO, zhi[sub] = MAGIC_HI;
        bool ok = true;
        for (; b < NB && ok; b += ((b & 1) ? 2 * SETS - 1 : 1)) {
            const uint32_t st = ring + s * kStage;
            if ((b % BPS) == 0) {
                // A set skips the other sets' slots, so its parity wait on a slot is only unambiguous once the slot's
                // previous refill is known to have landed: the MMAs of that refill's last block have completed.
                const int c = (b / BPS - NS) * BPS + BPS - 1;
                if (c > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar_done + 8 * (c & (kUmmaDoneRing - 1)), (uint32_t)((c / kUmmaDoneRing) & 1)));
                ok = ok && __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, ph));   // warp-uniform
                if (!ok) break;
            }
            if ((b & 1) == 0) {
#pragma unroll
                for (int sub = 0; sub < SUB; ++sub) {
                    s2[sub] = sc_next[sub] * 0x00010001u;
                    const uint32_t z = (h ? (zb_next[sub] >> 4) : (zb_next[sub] & 15u)) + z_add;   // up to 16: still exact
                    if constexpr (BF) {
                        zero_constants<true>(z, zlo[sub], zhi[sub]);
                    } else {
                        zlo[sub] = (z * 0x00010001u) | MAGIC_LO;
                        zhi[sub] = (z * 0x00100010u) | MAGIC_HI;
                    }
                }
                if (b + 2 * SETS < NB) load_sz((b >> 1) + SETS, sc_next, zb_next);   // this set's next item
            }
            const uint32_t wb = st + (b % BPS) * kUmmaWBlockBytes;
            uint2 wv[4];
#pragma unroll
            for (int t4 = 0; t4 < 4; ++t4) wv[t4] = lds64(wb + w_rd[t4]);
            // constants of the two 32-row halves of this block: the item's group (SUB = 1), the block's (2) or the
            // half's own (4); picked with selects so that the arrays stay in registers
            uint32_t s2_b[2], zlo_b[2], zhi_b[2];
            const bool odd = (b & 1) != 0;
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                constexpr int kLast = SUB - 1;
                const int lo = SUB == 4 ? jj : 0, hi = SUB == 4 ? 2 + jj : kLast;   // even / odd block of the item
                s2_b[jj] = odd ? s2[hi] : s2[lo];
                zlo_b[jj] = odd ? zlo[hi] : zlo[lo];
                zhi_b[jj] = odd ? zhi[hi] : zhi[lo];
            }
            uint32_t r[32];
#pragma unroll
            for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                for (int t4 = 0; t4 < 4; ++t4) {
                    uint32_t w = jj ? wv[t4].y : wv[t4].x;       // rows 32 jj + 8 t4 + (0..7), TMEM columns 16 jj + 4 t4 + (0..3)
                    uint32_t *o = r + 16 * jj + 4 * t4;
                    if constexpr (BF) {
                        // bfloat16: exact q - z, then one rounding in the product with the scale
                        uint32_t d[4];
                        nibble_pairs_minus_zero<true>(w, zlo_b[jj], zhi_b[jj], d);
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[e] = bmul2_u32(d[e], s2_b[jj]);
                        continue;
                    }
                    o[0] = hmul2_u32(hsub2_u32(lop3_and_or(w, LO, MAGIC_LO), zlo_b[jj]), s2_b[jj]);
                    o[1] = hmul2_u32(hsub2_u32(lop3_and_or(w, HI, MAGIC_HI), zhi_b[jj]), s2_b[jj]);
                    w >>= 8;
                    o[2] = hmul2_u32(hsub2_u32(lop3_and_or(w, LO, MAGIC_LO), zlo_b[jj]), s2_b[jj]);
                    o[3] = hmul2_u32(hsub2_u32(lop3_and_or(w, HI, MAGIC_HI), zhi_b[jj]), s2_b[jj]);
                }
            if (b >= NA) {     // the stage's previous block b - NA must have been multiplied
                ok = __all_sync(0xffffffffu, mbar_wait(bar_done + 8 * ((b - NA) & (kUmmaDoneRing - 1)), (uint32_t)(((b - NA) / kUmmaDoneRing) & 1)));
                if (!ok) break;
                tc_fence_after_sync();
            }
            tmem_st_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + kAcol + (j * NA + sa) * 32, r);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_afull + 8 * (j * NA + sa));
            const int step = (b & 1) ? 2 * SETS - 1 : 1;   // to this set's next block
            // and to that block's ring slot
            s += (b + step) / BPS - b / BPS;
            while (s >= NS) { s -= NS; ph ^= 1u; }
            sa += step;
            while (sa >= NA) sa -= NA;
        }
        // ---- epilogue: lane n of the accumulator holds y[m0 .. m0+TOK, 128 p + n]
        pdl_wait();
        ok = __all_sync(0xffffffffu, ok && mbar_wait(bar_dfull, 0));
        if (ok) tc_fence_after_sync();
        ok = ok && layout_ok;
        // 32 tokens (from c0) of this lane's column: the sum of the issuers' accumulators (an issuer without blocks,
        // possible when this CTA has a single K group, left its columns unwritten)
        auto load_acc = [&](int c0, uint32_t (&r)[32]) {
            tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + (j * ISS) * TOK + c0, r);
            tmem_wait_ld();
            if (ISS > 1 && NB > 2) {
                uint32_t r2[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + (j * ISS + 1) * TOK + c0, r2);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) + __uint_as_float(r2[i]));
            }
        };
        if (S == 1) {
            // The accumulator holds a column of y per TMEM lane, so a thread's 32 values of a chunk belong to 32
            // different rows of y.  The four warps of a set turn their 32-token x 128-column chunk around through
            // the (now idle) ring: fp16 rows of 256 bytes in shared memory, then 16 bytes per thread to y - whole
            // 128-byte lines instead of 2-byte stores.  Every warp takes part in the named barriers, also
            // after a wait that gave up (it then moves no data; the status word tells the host).
            const uint32_t stg = ring + (uint32_t)((j * SETS + set) * (32 * kPanel * 2));
            const int bar_id = 1 + j * SETS + set;
            const int tq = 32 * q + lane;           // thread within the set
#pragma unroll 1
            for (int c0 = 0; c0 < TOK; c0 += 32) {
                if (m0 + c0 >= a.M) break;
                if (SETS > 1 && ((c0 >> 5) % SETS) != set) continue;   // the warp sets share the token chunks
                if (ok) {
                    uint32_t r[32];
                    load_acc(c0, r);
                    if (a.bias || a.residual) {
                        // bias[column] + residual[token][column] join the fp32 sum before the one rounding; the 32 lanes
                        // of a warp read 32 neighbouring columns of one token row per load
                        const size_t ncol = (size_t)p * kPanel + n;
                        const float bv = a.bias ? __half2float(a.bias[ncol]) : 0.f;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const int m = m0 + c0 + i;
                            float v = __uint_as_float(r[i]) + bv;
                            if (a.residual && m < a.M) v += __half2float(a.residual[(size_t)m * a.N + ncol]);
                            r[i] = __float_as_uint(v);
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if constexpr (BF) sts_b16(stg + (uint32_t)(i * (kPanel * 2) + n * 2), float_to_out16<true>(__uint_as_float(r[i])));
                        else sts_f16(stg + (uint32_t)(i * (kPanel * 2) + n * 2), __float2half_rn(__uint_as_float(r[i])));
                }
                named_bar_sync(bar_id, 128);
                if (ok && !a.fuse) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int piece = tq + 128 * t, row = piece >> 4, c16 = piece & 15;   // 16 pieces per row
                        const int m = m0 + c0 + row;
                        if (m < a.M && c0 + row < TOK) {
                            const uint4 v = lds128(stg + (uint32_t)piece * 16u);
                            *reinterpret_cast<uint4 *>(a.y + (size_t)m * a.N + (size_t)p * kPanel + c16 * 8) = v;
                        }
                    }
                } else if (ok) {
                    // fused gate/up epilogue: the first 64 staged columns of a row are gate, the last 64 the matching up
                    // columns (both already rounded to fp16); eight outputs (16 bytes of the N / 2 wide row) per piece
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const int piece = tq + 128 * t, row = piece >> 3, c8 = piece & 7;     // 8 output pieces per row
                        const int m = m0 + c0 + row;
                        if (m < a.M && c0 + row < TOK) {
                            const uint4 gv = lds128(stg + (uint32_t)(row * 256 + c8 * 16));
                            const uint4 uv = lds128(stg + (uint32_t)(row * 256 + 128 + c8 * 16));
                            const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, uw[4] = {uv.x, uv.y, uv.z, uv.w};
                            uint32_t ow[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 gf = __half22float2(*reinterpret_cast<const __half2 *>(&gw[e]));
                                const float2 uf = __half22float2(*reinterpret_cast<const __half2 *>(&uw[e]));
                                const __half2 o = __floats2half2_rn(silu_mul(gf.x, uf.x), silu_mul(gf.y, uf.y));
                                ow[e] = *reinterpret_cast<const uint32_t *>(&o);
                            }
                            __half *orow = a.y + (size_t)m * (a.N / 2);
                            const int oc = p * 64 + c8 * 8;
                            if (a.out_index == nullptr) {
                                *reinterpret_cast<uint4 *>(orow + oc) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                            } else {
                                // scattered columns: eight destinations (two 16-byte index loads), eight 2-byte stores
                                const int4 ia = *reinterpret_cast<const int4 *>(a.out_index + oc);
                                const int4 ib = *reinterpret_cast<const int4 *>(a.out_index + oc + 4);
                                const int dst[8] = {ia.x, ia.y, ia.z, ia.w, ib.x, ib.y, ib.z, ib.w};
#pragma unroll
                                for (int e = 0; e < 8; ++e)
                                    orow[dst[e]] = __ushort_as_half((unsigned short)(ow[e >> 1] >> (16 * (e & 1))));
                            }
                        }
                    }
                }
                named_bar_sync(bar_id, 128);   // the next chunk overwrites the staging rows
            }
        } else if (S == 2) {
            // two CTAs: each parks its tile and reads the other's half through distributed shared memory (pushing, as
            // below, measured 2-4 % slower here: half of the data would go to the CTA itself)
            if (ok) {
#pragma unroll 1
                for (int c0 = 0; c0 < TOK; c0 += 32) {
                    if (m0 + c0 >= a.M) break;
                    if (SETS > 1 && ((c0 >> 5) % SETS) != set) continue;
                    uint32_t r[32];
                    load_acc(c0, r);
                    // split-K: park the fp32 partial tile [token][column] at the start of the (idle) ring
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < TOK) sts_f32(ring + (uint32_t)((c0 + i) * kPanel + n) * 4u, __uint_as_float(r[i]));
                }
            }
        } else {
            // split-K over four or eight CTAs.  Every CTA of the cluster is past its main loop once this barrier is
            // through: the rings are idle and the receive barriers armed.  Then each CTA pushes its partial sums to
            // the owners of the columns (st.async, counted by the owner's barrier) and the owner sums what arrived from
            // its own shared memory: about 1 us less per launch than reading the peers' tiles (o M = 64: 9.8 against
            // 11.4 us, down 16.4 against 18.0).
            __syncwarp();
            cluster_arrive_release();
            cluster_wait_acquire();
            if (ok) {
                const int sh = S == 2 ? 6 : S == 4 ? 5 : 4;                 // log2(128 / S)
                const int W = kPanel / S;
                // owner and own-column index of this lane's tile column n
                int owner, lc;
                if (!a.fuse) {
                    owner = n >> sh, lc = n & (W - 1);
                } else {
                    const int hw = W >> 1, c = n & 63;
                    owner = c / hw, lc = (n >> 6) * hw + c - owner * hw;
                }
                const uint32_t dst = map_to_cluster_rank(ring, (uint32_t)owner), dbar = map_to_cluster_rank(bar_recv, (uint32_t)owner);
#pragma unroll 1
                for (int c0 = 0; c0 < TOK; c0 += 32) {
                    if (m0 + c0 >= a.M) break;
                    if (SETS > 1 && ((c0 >> 5) % SETS) != set) continue;
                    uint32_t r[32];
                    load_acc(c0, r);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        st_async_f32(dst + (uint32_t)((rank * TOK + c0 + i) * W + lc) * 4u, __uint_as_float(r[i]), dbar);
                }
            }
            if (layout_ok && mbar_wait_cluster(bar_recv, 0) && ok) {    // (a refused layer: nobody pushes, nobody waits)
            const int p = p0;   // split-K runs with one panel per CTA (NP == 1)
            const int rows = (a.M - m0) < TOK ? (a.M - m0) : TOK;
            // four columns of token row m, starting at tile column cc, summed over the cluster in rank order
            // receive buffer at the start of the (idle) ring: [sender rank][token][own column] floats
            const int W = kPanel / S;
            auto sum4 = [&](int m, int cc) {
                // own column index of tile column cc: plain order, or (fused) gate columns first, then the up columns
                const int lc = !a.fuse ? cc - rank * W : (cc < 64 ? cc - rank * (W >> 1) : (W >> 1) + cc - 64 - rank * (W >> 1));
                float4 v[8];
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    if (qq < S) {
                        const uint4 u = lds128(ring + (uint32_t)((qq * TOK + m) * W + lc) * 4u);
                        v[qq] = make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w));
                    } else {
                        v[qq] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    sum.x += v[qq].x;
                    sum.y += v[qq].y;
                    sum.z += v[qq].z;
                    sum.w += v[qq].w;
                }
                return sum;
            };
            auto store4 = [&](__half *dst, float4 v) {
                uint2 out;
                if constexpr (BF) {
                    out.x = (uint32_t)float_to_out16<true>(v.x) | ((uint32_t)float_to_out16<true>(v.y) << 16);
                    out.y = (uint32_t)float_to_out16<true>(v.z) | ((uint32_t)float_to_out16<true>(v.w) << 16);
                } else {
                    const __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
                    out.x = *reinterpret_cast<const uint32_t *>(&lo);
                    out.y = *reinterpret_cast<const uint32_t *>(&hi);
                }
                *reinterpret_cast<uint2 *>(dst) = out;
            };
            const int c_lo = rank * kPanel / S, width = (rank + 1) * kPanel / S - c_lo;   // width is 16, 32 or 64
            if (!a.fuse) {
                const int w4 = width >> 2;      // four columns (16 bytes) per thread and step
                for (int idx = threadIdx.x - 32 * kFirstDq; idx < rows * w4; idx += 128 * NP * SETS) {
                    const int m = idx / w4, cc = c_lo + 4 * (idx - m * w4);
                    const size_t at = (size_t)(m0 + m) * a.N + (size_t)p * kPanel + cc;
                    float4 v = sum4(m, cc);
                    if (a.bias) {
                        const uint2 b = *reinterpret_cast<const uint2 *>(a.bias + (size_t)p * kPanel + cc);
                        const float2 b0 = __half22float2(*reinterpret_cast<const __half2 *>(&b.x));
                        const float2 b1 = __half22float2(*reinterpret_cast<const __half2 *>(&b.y));
                        v.x += b0.x, v.y += b0.y, v.z += b1.x, v.w += b1.y;
                    }
                    if (a.residual) {
                        const uint2 q = *reinterpret_cast<const uint2 *>(a.residual + at);
                        const float2 q0 = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
                        const float2 q1 = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
                        v.x += q0.x, v.y += q0.y, v.z += q1.x, v.w += q1.y;
                    }
                    store4(a.y + at, v);
                }
            } else {
                // this CTA finishes gate columns [rank width / 2, ...) of the tile and the matching up columns 64 further
                const int half_w = width >> 1, w4 = half_w >> 2;
                for (int idx = threadIdx.x - 32 * kFirstDq; idx < rows * w4; idx += 128 * NP * SETS) {
                    const int m = idx / w4, cc = rank * half_w + 4 * (idx - m * w4);
                    const float4 gsum = sum4(m, cc), usum = sum4(m, 64 + cc);
                    const float4 ov = make_float4(silu_mul(gsum.x, usum.x), silu_mul(gsum.y, usum.y), silu_mul(gsum.z, usum.z),
                                                  silu_mul(gsum.w, usum.w));
                    __half *orow = a.y + (size_t)(m0 + m) * (a.N / 2);
                    const int oc = p * 64 + cc;
                    if (a.out_index == nullptr) {
                        store4(orow + oc, ov);
                    } else {
                        const int4 ia = *reinterpret_cast<const int4 *>(a.out_index + oc);
                        orow[ia.x] = __float2half_rn(ov.x);
                        orow[ia.y] = __float2half_rn(ov.y);
                        orow[ia.z] = __float2half_rn(ov.z);
                        orow[ia.w] = __float2half_rn(ov.w);
                    }
                }
            }
            }
        }
    }
    if (S == 2) {
        // both CTAs have parked their tiles; CTA `rank` finishes columns [c_lo, c_lo + width)
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
        if (warp >= kFirstDq && layout_ok) {
            const int p = p0;   // split-K runs with one panel per CTA (NP == 1)
            const int rows = (a.M - m0) < TOK ? (a.M - m0) : TOK;
            // four columns of token row m, starting at tile column cc, summed over the cluster in rank order
            auto sum4 = [&](int m, int cc) {
                const uint32_t local = ring + (uint32_t)(m * kPanel + cc) * 4u;
                float4 v[8];
#pragma unroll
                for (int qq = 0; qq < 8; ++qq)
                    v[qq] = qq < S ? ld_cluster_f32x4(map_to_cluster_rank(local, (uint32_t)qq)) : make_float4(0.f, 0.f, 0.f, 0.f);
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int qq = 0; qq < 8; ++qq) {
                    sum.x += v[qq].x;
                    sum.y += v[qq].y;
                    sum.z += v[qq].z;
                    sum.w += v[qq].w;
                }
                return sum;
            };
            auto store4 = [&](__half *dst, float4 v) {
                uint2 out;
                if constexpr (BF) {
                    out.x = (uint32_t)float_to_out16<true>(v.x) | ((uint32_t)float_to_out16<true>(v.y) << 16);
                    out.y = (uint32_t)float_to_out16<true>(v.z) | ((uint32_t)float_to_out16<true>(v.w) << 16);
                } else {
                    const __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
                    out.x = *reinterpret_cast<const uint32_t *>(&lo);
                    out.y = *reinterpret_cast<const uint32_t *>(&hi);
                }
                *reinterpret_cast<uint2 *>(dst) = out;
            };
            const int c_lo = rank * kPanel / S, width = (rank + 1) * kPanel / S - c_lo;   // width is 16, 32 or 64
            if (!a.fuse) {
                const int w4 = width >> 2;      // four columns (16 bytes) per thread and step
                for (int idx = threadIdx.x - 32 * kFirstDq; idx < rows * w4; idx += 128 * NP * SETS) {
                    const int m = idx / w4, cc = c_lo + 4 * (idx - m * w4);
                    const size_t at = (size_t)(m0 + m) * a.N + (size_t)p * kPanel + cc;
                    float4 v = sum4(m, cc);
                    if (a.bias) {
                        const uint2 b = *reinterpret_cast<const uint2 *>(a.bias + (size_t)p * kPanel + cc);
                        const float2 b0 = __half22float2(*reinterpret_cast<const __half2 *>(&b.x));
                        const float2 b1 = __half22float2(*reinterpret_cast<const __half2 *>(&b.y));
                        v.x += b0.x, v.y += b0.y, v.z += b1.x, v.w += b1.y;
                    }
                    if (a.residual) {
                        const uint2 q = *reinterpret_cast<const uint2 *>(a.residual + at);
                        const float2 q0 = __half22float2(*reinterpret_cast<const __half2 *>(&q.x));
                        const float2 q1 = __half22float2(*reinterpret_cast<const __half2 *>(&q.y));
                        v.x += q0.x, v.y += q0.y, v.z += q1.x, v.w += q1.y;
                    }
                    store4(a.y + at, v);
                }
            } else {
                // this CTA finishes gate columns [rank width / 2, ...) of the tile and the matching up columns 64 further
                const int half_w = width >> 1, w4 = half_w >> 2;
                for (int idx = threadIdx.x - 32 * kFirstDq; idx < rows * w4; idx += 128 * NP * SETS) {
                    const int m = idx / w4, cc = rank * half_w + 4 * (idx - m * w4);
                    const float4 gsum = sum4(m, cc), usum = sum4(m, 64 + cc);
                    const float4 ov = make_float4(silu_mul(gsum.x, usum.x), silu_mul(gsum.y, usum.y), silu_mul(gsum.z, usum.z),
                                                  silu_mul(gsum.w, usum.w));
                    __half *orow = a.y + (size_t)(m0 + m) * (a.N / 2);
                    const int oc = p * 64 + cc;
                    if (a.out_index == nullptr) {
                        store4(orow + oc, ov);
                    } else {
                        const int4 ia = *reinterpret_cast<const int4 *>(a.out_index + oc);
                        orow[ia.x] = __float2half_rn(ov.x);
                        orow[ia.y] = __float2half_rn(ov.y);
                        orow[ia.z] = __float2half_rn(ov.z);
                        orow[ia.w] = __float2half_rn(ov.w);
                    }
                }
            }
        }
        // no CTA may exit (and free its shared memory) while a peer can still read its tile
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
    } else if (S > 2 && warp < kFirstDq) {
        // (the dequant warps pass this barrier in their epilogue)
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) GPTQ_TRACE_MAX(a.trace_slot, last_exit);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kCols);
    }
}

struct UmmaPlan {
    int tok;        // tokens per CTA tile: 16, 32, 64, 128 or 256
    int np;         // 128-column panels per CTA
    int sets;       // dequant warp sets per panel
    int S;          // CTAs per output tile along K (cluster size)
    int stages;
    int ctas;       // grid of the main launch: (tiles - tail_tiles) * S
    int smem_bytes;
    // When the tiles fill the SMs more than once and the last wave would leave most SMs idle, that wave's tiles
    // go to a second launch that splits K over clusters of tail_S CTAs (0 tiles: no second launch).
    int tail_tiles, tail_S, tail_stages;
};

// A-ring depth per panel: with two panels the 512 tensor-memory columns hold exactly 2 x (128 + 4 x 32)
__host__ __device__ constexpr int umma_a_stages(int tok, int np) { return tok >= 64 ? 4 : 3; }
// resident CTAs per SM: tensor memory (512 columns) and shared memory allow this many
__host__ __device__ constexpr int umma_ctas_per_sm(int tok, int np) { return (np > 1 || tok > 128) ? 1 : tok <= 32 ? 3 : 2; }

// Token tile by M (256 tokens from M = 129 up: one dequantised block then feeds twice the MMA work, and even a
// half-empty 256-token tile measured 15-22 % faster than two 128-token tiles on all four 7B shapes);
// cluster size and shared-memory padding by the same rules as the mma.sync kernel.  Two panels per CTA
// (np = 2) halve the x traffic per flop but allow only one CTA per SM and measured slower, so np = 1.
inline UmmaPlan plan_umma(int M, int N, int K, int sm_count)
{
    UmmaPlan pl{};
    const int tok = M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : 256;
    const int panels = N / kPanel;
    const int np = 1;
    const int sets = 2;
    const int G = K / kGroup, tiles = (panels / np) * ((M + tok - 1) / tok);
    const int stage = umma_slot_bytes(tok, np);
    const int cps_max = umma_ctas_per_sm(tok, np);
    int best_S = 1;
    long long best_t = -1;
    for (int pass = 0; pass < 2 && best_t < 0; ++pass) {
        for (int S = 1; S <= 8; S *= 2) {
            if (S > G || (pass == 1 && S > 1)) break;          // nothing fits at once: several waves, no split
            // the exchange of the fp32 partial tiles grows with the tile: with 128 tokens and more an 8-way split measured
            // slower than a 4-way one (o, M = 128: 16.2 vs 11.5 us; down: 24.5 vs 21.3)
            if (tok >= 128 && S > 4) break;
            const long long ctas = (long long)tiles * S, ipc = (G + S - 1) / S;
            const long long on_busiest_sm = (ctas + sm_count - 1) / sm_count;
            if (pass == 0 && on_busiest_sm > cps_max) continue;
            const long long serial = ipc * 45, shared = on_busiest_sm * ipc * 30;
            const long long t = (serial > shared ? serial : shared) + (S > 1 ? 100 : 0);
            if (best_t < 0 || t < best_t) { best_t = t; best_S = S; }
        }
    }
    const int S = best_S;
    const int groups_per_cta = (G + S - 1) / S;
    int per_sm = (tiles * S + sm_count - 1) / sm_count;
    if (per_sm > cps_max) per_sm = cps_max;
    const int smem_cap = (227 * 1024) / per_sm - 1024;
    const int smem_floor = (227 * 1024) / (per_sm + 1) + 512;
    int stages = (smem_cap - 2048) / stage;
    if (stages > 8) stages = 8;
    // fewer blocks in the ring than "block multiplied" barriers (see the kernel)
    if (stages * umma_blocks_per_slot(tok) >= kUmmaDoneRing) stages = (kUmmaDoneRing - 1) / umma_blocks_per_slot(tok);
    const int refills_per_cta = 2 * groups_per_cta / umma_blocks_per_slot(tok);
    if (stages > refills_per_cta) stages = refills_per_cta;
    while (S > 1 && stages * stage < tok * kPanel * 4) ++stages;   // the ring doubles as the fp32 partial tile
    pl.tok = tok;
    pl.np = np;
    pl.sets = sets;
    pl.S = S;
    pl.stages = stages;
    pl.smem_bytes = 2048 + stages * stage;
    if (pl.smem_bytes < smem_floor) pl.smem_bytes = smem_floor;
    pl.tail_tiles = 0;
    pl.tail_S = 1;
    pl.tail_stages = stages;
    const int slots = sm_count * cps_max;              // CTAs resident at once
    if (S == 1 && tiles > slots && tiles % slots != 0) {
        const int r = tiles % slots;
        int ts = 1;
        while (ts * 2 <= (tok >= 128 ? 4 : 8) && ts * 2 <= G && r * ts * 2 <= slots) ts *= 2;
        int tstages = stages;
        const int trefills = 2 * ((G + ts - 1) / ts) / umma_blocks_per_slot(tok);
        if (tstages > trefills) tstages = trefills;
        while (tstages * stage < tok * kPanel * 4) ++tstages;      // the ring doubles as the fp32 partial tile
        if (ts > 1 && 2048 + tstages * stage <= pl.smem_bytes && tstages * umma_blocks_per_slot(tok) < kUmmaDoneRing) {
            pl.tail_tiles = r;
            pl.tail_S = ts;
            pl.tail_stages = tstages;
        }
    }
    pl.ctas = (tiles - pl.tail_tiles) * S;
    return pl;
}

template <int TOK, int NP, int SETS, int SUB, bool BF>
static int launch_umma_sub(const UmmaArgs &args, const CUtensorMap &w_map, const CUtensorMap &x_map,
                           const UmmaPlan &plan, int ctas, cudaStream_t s)
{
    auto kernel = umma_kernel<TOK, umma_a_stages(TOK, NP), NP, SETS, SUB, BF>;
    static int configured_smem[64] = {};
    const int cfg_st = ensure_dynamic_smem((const void *)kernel, configured_smem, plan.smem_bytes);
    if (cfg_st) return cfg_st;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)ctas);
    cfg.blockDim = dim3(umma_threads(TOK, NP, SETS));
    cfg.dynamicSmemBytes = (size_t)plan.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)args.S;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return record_cuda_error(cudaLaunchKernelEx(&cfg, kernel, args, w_map, x_map));
}

template <int TOK, int NP, int SETS>
static int launch_umma_tok(const UmmaArgs &args, const CUtensorMap &w_map, const CUtensorMap &x_map,
                           const UmmaPlan &plan, int ctas, int sub, int bf16, cudaStream_t s)
{
    switch (sub + (bf16 ? 10 : 0)) {
    case 1: return launch_umma_sub<TOK, NP, SETS, 1, false>(args, w_map, x_map, plan, ctas, s);
    case 2: return launch_umma_sub<TOK, NP, SETS, 2, false>(args, w_map, x_map, plan, ctas, s);
    case 4: return launch_umma_sub<TOK, NP, SETS, 4, false>(args, w_map, x_map, plan, ctas, s);
    case 11: return launch_umma_sub<TOK, NP, SETS, 1, true>(args, w_map, x_map, plan, ctas, s);
    case 12: return launch_umma_sub<TOK, NP, SETS, 2, true>(args, w_map, x_map, plan, ctas, s);
    case 14: return launch_umma_sub<TOK, NP, SETS, 4, true>(args, w_map, x_map, plan, ctas, s);
    default: return GPTQ_ERR_UNSUPPORTED;
    }
}

int launch_umma(const __half *x, const void *qweight, const void *qzeros, const void *scales, __half *y, int M, int N,
                int K, int group_size, const UmmaPlan &plan, int fuse, const __half *bias, const __half *residual,
                const int32_t *out_index, int bf16, cudaStream_t s)
{
    UmmaArgs args;
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
    args.trailer = reinterpret_cast<const TiledTrailer *>((const uint8_t *)qzeros + tiled_zero_bytes(N, K, group_size));
    const int sub = kGroup / group_size;
    if (plan.stages < 1 || plan.stages * umma_blocks_per_slot(plan.tok) >= kUmmaDoneRing) return GPTQ_ERR_UNSUPPORTED;
    // packed weights as rows of 64 bytes (16 words); a box is one ring slot's K64 blocks of a panel (64 rows each)
    CUtensorMap w_map, x_map;
    const uint64_t w_rows = (uint64_t)K * N / 2 / 64;
    int st = make_tensor_map_2d(&w_map, CU_TENSOR_MAP_DATA_TYPE_UINT32, qweight, 16, w_rows, 64, 16,
                                (uint32_t)(64 * umma_blocks_per_slot(plan.tok)),
                                CU_TENSOR_MAP_SWIZZLE_64B);
    if (st) return st;
    // x as K / 64 tiles of [M rows, 64 k]; a box is one ring slot's tiles of one token tile
    st = make_tensor_map_ktiles(&x_map, x, (uint64_t)K, (uint64_t)M, (uint32_t)plan.tok,
                                (uint32_t)umma_blocks_per_slot(plan.tok));
    if (st) return st;
    auto launch = [&](const UmmaArgs &la, int ctas) {
        switch (plan.tok) {
        case 32: return launch_umma_tok<32, 1, 2>(la, w_map, x_map, plan, ctas, sub, bf16, s);
        case 64: return launch_umma_tok<64, 1, 2>(la, w_map, x_map, plan, ctas, sub, bf16, s);
        case 128: return launch_umma_tok<128, 1, 2>(la, w_map, x_map, plan, ctas, sub, bf16, s);
        case 256: return launch_umma_tok<256, 1, 2>(la, w_map, x_map, plan, ctas, sub, bf16, s);
        default: return (int)GPTQ_ERR_UNSUPPORTED;
        }
    };
    args.tile0 = 0;
    if (plan.ctas > 0) {
        st = launch(args, plan.ctas);
        if (st) return st;
    }
    if (plan.tail_tiles > 0) {
        // the last, partly filled wave: the same kernel on clusters that split K, starting at the first tile the
        // main launch left out
        UmmaArgs ta = args;
        ta.tile0 = plan.ctas / plan.S;
        ta.S = plan.tail_S;
        ta.stages = plan.tail_stages;
        ta.trace_slot = next_trace_slot();
        st = launch(ta, plan.tail_tiles * plan.tail_S);
    }
    return st;
}

}  // namespace gptq
