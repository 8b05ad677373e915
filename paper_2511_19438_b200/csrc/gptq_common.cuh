// Shared definitions of the gptq_b200 CUDA library: the tiled weight layout, PTX wrappers
// and the device status word.  sm_100a only.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gptq_b200.h"

namespace gptq {

// ----------------------------------------------------------------------------------------
// Tiled layout written by gptq_repack (sizes equal the canonical ones).
//
// Rows are first sorted by group (identity without act-order), so group `grp` owns sorted
// rows 128*grp .. 128*grp+127.  N is cut into 128-column PANELS.  The unit of streaming is an
// ITEM = (panel p, group grp); item index t = p*G + grp.  Item t owns
//     qweight_out bytes [t*8192, +8192)   scales_out bytes [t*256, +256)   qzeros_out [t*64, +64)
// so a CTA that works through consecutive items reads three contiguous byte streams.
//
// Inside an item the 8192 weight bytes are two K64 BLOCKS of 4096 bytes; a block is eight
// 512-byte UNITS (one per 16 columns, u = 0..7); a unit is 32 LANE chunks of 16 bytes.  Lane
// L = 4*g + t4 (g = 0..7, t4 = 0..3) holds four words c = j + 2*h (j, h in {0,1}):
//     word (j,h): column n = 128p + 16u + g + 8h, sorted rows 64*blk + 32*j + 8*t4 + (0..7)
// and row offset e (0..7) sits in nibble (e>>1) + 4*(e&1) of the word, so that
// `w & 0x000f000f` is the half2 pair (rows e=0,1), `w & 0x00f000f0` the pair (e=2,3) and the
// same two masks on `w >> 8` give (e=4,5) and (e=6,7).
//
// This one layout feeds both kernel families conflict-free from shared memory:
//  * mma.sync kernel: lane L of the warp that owns unit u reads its chunk with one 128-bit
//    load and has the A fragments (weights as the 16-row operand) of four m16n8k16 MMAs.
//  * tcgen05 kernel: the thread that owns column n (TMEM lane) reads 8 bytes (h fixed, j=0,1)
//    from each of the four chunks 4g+t4: 64 consecutive rows of its column.
//
// Scales of an item: per quantisation group inside its 128 rows (SUB = 128 / group_size of them: 1, 2 or 4)
// fp16[128] at position 16u + 2g + h  <- column 128p + 16u + g + 8h; the SUB blocks follow each other.
// Zeros of an item: per group 64 bytes, byte 8u + g = z[col g] | z[col g+8] << 4.
// qzeros_out ends with a 16-byte trailer {magic, flags, group_size, 0} (see TiledTrailer): the tiled buffers
// describe themselves, so gptq_gemm needs no format argument.
// ----------------------------------------------------------------------------------------
constexpr int kGroup = 128;          // rows per item (one quantisation group at group_size 128, two at 64, four at 32)
constexpr int kPanel = 128;          // columns per panel
constexpr int kItemWBytes = 8192;    // packed weights of one item
constexpr int kItemSBytes = 256;     // scales of one group of one item
constexpr int kItemZBytes = 64;      // packed zeros of one group of one item
constexpr int kTrailerBytes = 16;
constexpr uint32_t kTrailerMagic = 0x51545047u;   // "GPTQ"
constexpr uint32_t kFormatZerosMinusOne = 1u;     // == GPTQ_FORMAT_ZEROS_MINUS_ONE
constexpr uint32_t kFormatGateUp = 2u;            // == GPTQ_FORMAT_GATE_UP: column halves interleaved per panel
constexpr uint32_t kFormatBf16 = 4u;              // == GPTQ_FORMAT_BF16: the scales are bfloat16 (so are x and y of the matmul)
constexpr uint32_t kFormatMask = 7u;
// With kFormatGateUp a layer's columns are [gate | up] (N / 2 each) and tiled panel p holds gate columns
// 64 p .. 64 p + 63 in its first half and the matching up columns in its second, so that one CTA sees both.
__host__ __device__ inline int gate_up_source_column(int nt, int N)      // tiled column -> checkpoint column
{
    const int p = nt / kPanel, c = nt % kPanel;
    return (c / 64) * (N / 2) + 64 * p + (c % 64);
}
__host__ __device__ inline int gate_up_tiled_column(int n, int N)        // checkpoint column -> tiled column
{
    const int half = n / (N / 2), rem = n % (N / 2);
    return (rem / 64) * kPanel + half * 64 + (rem % 64);
}
struct TiledTrailer {
    uint32_t magic, flags, group_size, reserved;
};
// bytes of the tiled zero points without the trailer
__host__ __device__ inline size_t tiled_zero_bytes(int N, int K, int group_size)
{
    return (size_t)(K / group_size) * (size_t)(N / 2);
}
constexpr int kBlockWBytes = 4096;   // one K64 block of one panel
constexpr int kUnitBytes = 512;

__host__ __device__ inline int nibble_slot(int e) { return (e >> 1) + 4 * (e & 1); }

// Byte offset of the repacked word that holds (sorted row i, column n), and the nibble slot.
__host__ __device__ inline size_t repacked_word_offset(int i, int n, int G, int *slot)
{
    int p = n / kPanel, nn = n % kPanel;
    int u = nn / 16, c16 = nn % 16, g = c16 & 7, h = c16 >> 3;
    int grp = i / kGroup, r = i % kGroup;
    int blk = r / 64, r64 = r % 64, j = r64 / 32, r32 = r64 % 32, t4 = r32 / 8, e = r32 % 8;
    *slot = nibble_slot(e);
    size_t item = (size_t)p * G + grp;
    return item * kItemWBytes + (size_t)blk * kBlockWBytes + u * kUnitBytes + (4 * g + t4) * 16 + (j + 2 * h) * 4;
}
// grp counts quantisation groups (K / group_size of them, `groups` per column panel)
__host__ __device__ inline size_t repacked_scale_index(int grp, int n, int groups)
{
    int p = n / kPanel, nn = n % kPanel;
    int u = nn / 16, c16 = nn % 16, g = c16 & 7, h = c16 >> 3;
    return ((size_t)p * groups + grp) * kPanel + 16 * u + 2 * g + h;
}
// byte index and nibble (0 = low) of the zero point of (grp, n)
__host__ __device__ inline size_t repacked_zero_byte(int grp, int n, int groups, int *hi)
{
    int p = n / kPanel, nn = n % kPanel;
    int u = nn / 16, c16 = nn % 16, g = c16 & 7;
    *hi = c16 >> 3;
    return ((size_t)p * groups + grp) * kItemZBytes + 8 * u + g;
}

// ----------------------------------------------------------------------------------------
// Device status word: kernels never trap; a bounded wait that gives up records a code here.
// ----------------------------------------------------------------------------------------
enum : int { kStatusOk = 0, kStatusWaitTimeout = 1, kStatusLayoutMismatch = 2 };   // g_device_status, recorded with atomicMax
enum : int { kGidxOk = 0, kGidxUnequalGroups = 1, kGidxOutOfRange = 2 };   // g_gidx_status, likewise
// The library is built as one translation unit, so these are the single definitions.  The g_idx
// check of gptq_repack has a word of its own, so that reading and clearing it never drops a
// pending wait timeout of an earlier kernel.
__device__ int g_device_status = 0;
__device__ int g_gidx_status = 0;

#ifdef __CUDACC__
// ----------------------------------------------------------------------------------------
// PTX wrappers
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up about two seconds after it started, records the failure in the status
// word and returns false instead of hanging; the caller carries on without touching the data.
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// ---- launch timeline (compiled in with -DGPTQ_TIMELINE only) -----------------------------------
// Every matmul launch of a timeline build takes the next of kTraceLaunches rows and its CTAs record, with %globaltimer
// and 64-bit atomic min / max, when the grid's first and last CTA started, when the first weight copy was issued, when
// griddepcontrol.wait first and last returned, when the first activation tile had landed and when the last CTA was
// done.  gptq_trace_reset / gptq_trace_read move the rows; in a normal build the macros expand to nothing.
constexpr int kTraceLaunches = 64;
struct TraceRow {
    unsigned long long first_entry, first_weight_issue, first_wait_done, last_wait_done, first_data, last_exit;
    unsigned long long kernel_and_ctas;     // (1 = mma.sync kernel, 2 = tcgen05 kernel) << 32 | grid size
    unsigned long long last_entry;          // when the grid's last CTA started
};
#ifdef GPTQ_TIMELINE
__device__ TraceRow g_trace[kTraceLaunches];
#define GPTQ_TRACE_MIN(slot, field) \
    do { if ((slot) >= 0) atomicMin(&g_trace[(slot)].field, (unsigned long long)global_timer_ns()); } while (0)
#define GPTQ_TRACE_MAX(slot, field) \
    do { if ((slot) >= 0) atomicMax(&g_trace[(slot)].field, (unsigned long long)global_timer_ns()); } while (0)
#define GPTQ_TRACE_SET(slot, field, v) \
    do { if ((slot) >= 0) g_trace[(slot)].field = (unsigned long long)(v); } while (0)
#else
#define GPTQ_TRACE_MIN(slot, field) do { } while (0)
#define GPTQ_TRACE_MAX(slot, field) do { } while (0)
#define GPTQ_TRACE_SET(slot, field, v) do { } while (0)
#endif
// the row the next launch takes (host side; -1 in a normal build)
int next_trace_slot();

constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __noinline__ bool mbar_wait_limited(uint32_t bar, uint32_t parity, uint64_t limit_ns)
{
    const uint64_t start = global_timer_ns();
    for (;;) {
        for (int it = 0; it < 256; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - start > limit_ns) break;
    }
    atomicMax(&g_device_status, (int)kStatusWaitTimeout);
    return false;
}
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity)
{
    return mbar_wait_limited(bar, parity, kWaitLimitNs);
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (int it = 0; it < 64; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity);
}
// 1-D bulk copy global -> shared with an L2 cache-policy hint, completion counted in bytes on an
// mbarrier.  dst, src and bytes must be multiples of 16.  Issue it from a dedicated producer thread:
// issued from lanes of a warp that goes on to run mma.sync, it faulted ("illegal instruction").
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// (a & b) | c in one instruction
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t hsub2_u32(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("sub.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("mul.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bsub2_u32(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("sub.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t bmul2_u32(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("mul.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// The four 16-bit pairs of exact integers q - z held by one packed word (rows e = 0,1 / 2,3 / 4,5 / 6,7 of its column),
// in the 16-bit float format of the matmul.  fp16 (10 fraction bits): the low nibble of a byte becomes 1024 + q and the
// high nibble, left in place, 1024 + 16 q with a second magic exponent (64 + q), so one shift serves four pairs; zlo and
// zhi are the matching constants 1024 + z and 64 + z.  bfloat16 has 7 fraction bits, a nibble in bits 4..7 would run
// into the exponent, so every pair is shifted down first and becomes 128 + q; zlo = 128 + z serves all four.
template <bool BF>
__device__ __forceinline__ void nibble_pairs_minus_zero(uint32_t w, uint32_t zlo, uint32_t zhi, uint32_t (&o)[4])
{
    constexpr uint32_t LO = 0x000f000fu, HI = 0x00f000f0u;
    if constexpr (BF) {
        constexpr uint32_t MAGIC = 0x43004300u;
        o[0] = bsub2_u32(lop3_and_or(w, LO, MAGIC), zlo);
        o[1] = bsub2_u32(lop3_and_or(w >> 4, LO, MAGIC), zlo);
        o[2] = bsub2_u32(lop3_and_or(w >> 8, LO, MAGIC), zlo);
        o[3] = bsub2_u32(lop3_and_or(w >> 12, LO, MAGIC), zlo);
    } else {
        constexpr uint32_t MAGIC_LO = 0x64006400u, MAGIC_HI = 0x54005400u;
        o[0] = hsub2_u32(lop3_and_or(w, LO, MAGIC_LO), zlo);
        o[1] = hsub2_u32(lop3_and_or(w, HI, MAGIC_HI), zhi);
        w >>= 8;
        o[2] = hsub2_u32(lop3_and_or(w, LO, MAGIC_LO), zlo);
        o[3] = hsub2_u32(lop3_and_or(w, HI, MAGIC_HI), zhi);
    }
}
// the constants for zero point z (0..16): both halves of a pair hold the same column
template <bool BF>
__device__ __forceinline__ void zero_constants(uint32_t z, uint32_t &zlo, uint32_t &zhi)
{
    if constexpr (BF) {
        zlo = (z * 0x00010001u) | 0x43004300u;      // 128 + z
        zhi = zlo;
    } else {
        zlo = (z * 0x00010001u) | 0x64006400u;      // 1024 + z
        zhi = (z * 0x00100010u) | 0x54005400u;      // 64 + z
    }
}
// a pair of 16-bit floats of the matmul's format -> two floats
template <bool BF>
__device__ __forceinline__ float2 pair_to_float2(uint32_t v)
{
    if constexpr (BF) return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
    else return __half22float2(*reinterpret_cast<const __half2 *>(&v));
}
// one float -> the 16 bits of the matmul's output format, round to nearest even
template <bool BF>
__device__ __forceinline__ unsigned short float_to_out16(float v)
{
    if constexpr (BF) return __bfloat16_as_ushort(__float2bfloat16_rn(v));
    else return __half_as_ushort(__float2half_rn(v));
}
// stores one element of y (declared as fp16 storage; with BF the 16 bits are a bfloat16)
template <bool BF>
__device__ __forceinline__ void store_out16(__half *p, float v)
{
    if constexpr (BF) *reinterpret_cast<unsigned short *>(p) = float_to_out16<true>(v);
    else *p = __float2half_rn(v);
}
// D(16x8, f32) = A(16x16, bf16, row) * B(16x8, bf16, col) + C
__device__ __forceinline__ void mma_m16n8k16_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1)
{
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D(16x8, f32) = A(16x16, f16, row) * B(16x8, f16, col) + C
__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1)
{
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds8(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
#endif  // __CUDACC__

// ----------------------------------------------------------------------------------------
// Host-side launch plumbing shared by the translation units
// ----------------------------------------------------------------------------------------
int record_cuda_error(cudaError_t e);   // stores e, returns GPTQ_ERR_CUDA (or GPTQ_OK for success)
// Raises a kernel's dynamic shared-memory limit (and asks for the largest carve-out) the first time a launch on
// the current device needs more than before; `configured` is the launcher's per-device record.  Thread-safe.
int ensure_dynamic_smem(const void *kernel, int *configured, int smem_bytes);

struct Workspace {
    void *ptr = nullptr;
    size_t bytes = 0;
};

struct StreamKPlan {
    int m_tile;       // tokens per CTA tile: 8, 16, 32 or 64
    int stages;
    int ctas;
    int items;        // panels * G
    int split_panels;
    int smem_bytes;
    size_t partial_bytes;   // fp32 partial tiles: ctas * 2 * m_rows * 128 * 4
    size_t ticket_bytes;    // one int per panel
};
StreamKPlan plan_streamk(int m_rows, int N, int K, int sm_count);

// launchers (defined next to their kernels); all pointers are device pointers
int launch_unpack_u8(const int32_t *qweight, const int32_t *qzeros, uint8_t *q_out, uint8_t *z_out, int N, int K,
                     int G, cudaStream_t s);
int launch_dequant_f32(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                       float *w_out, int N, int K, int group_size, int act_order, int repacked, int format,
                       cudaStream_t s);
int launch_repack(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                  void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, int N, int K,
                  int group_size, int act_order, int format, cudaStream_t s);
int launch_gather_x(const __half *x, const int32_t *perm, __half *x_out, int M, int K, cudaStream_t s);
int launch_streamk(const __half *x, const void *qweight, const void *qzeros, const void *scales, __half *y,
                   int M, int N, int K, const StreamKPlan &plan, float *partials, int *tickets, cudaStream_t s);

}  // namespace gptq
