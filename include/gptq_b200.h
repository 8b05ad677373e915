/*
 * gptq_b200 - GPTQ 4-bit weight-only quantized matmul for NVIDIA B200 (sm_100a).
 *
 *     y[M,N] = x[M,K] . dequant(W)[K,N]
 *
 * This is the linear-layer product that the Opt4GPTQ paper accelerates (Section 1:
 * 4-bit GPTQ weights inside every linear layer of the served model; Section 4.2: fp16
 * activations and fp16 weights after dequantisation).  The paper's three kernel-level
 * ideas map onto this library as follows: vectorised loads (Section 3.2, Algorithm 2)
 * become 16-byte-granular bulk and tensor-map (TMA) copies of re-tiled weights and of the
 * activation tiles; native packed-half arithmetic (Section 3.3, Algorithm 3) becomes
 * lop3 / sub.f16x2 / mul.f16x2 dequantisation feeding tensor-core MMAs (mma.sync for up to 16
 * token rows, tcgen05 with the dequantised operand in tensor memory above that); block-level
 * pre-reduction with one committing thread (Section 3.1, Algorithm 1) becomes split-K inside a
 * thread-block cluster, reduced through distributed shared memory in a fixed order, with one
 * plain fp16 store and no atomics on the output.
 *
 * Storage format ("canonical", what checkpoints hold):
 *   qweight int32[K/8, N]  nibble i (bits 4i..4i+3, word read as unsigned) of word (r,n)
 *                          is q[8r+i, n] in 0..15
 *   qzeros  int32[G, N/8]  nibble j of word (g,c) is z[g, 8c+j]; the stored nibble IS the
 *                          zero point (no +1 offset);  G = K / group_size
 *   scales  fp16 [G, N]
 *   g_idx   int32[K]       act-order only: row k uses scale/zero row g_idx[k]
 *   w[k,n] = (q[k,n] - z[g(k),n]) * scales[g(k),n],  g(k) = g_idx[k] or k / group_size
 *
 * All pointers are DEVICE pointers unless a parameter name ends in _host.  The caller owns
 * every buffer; the library allocates no device memory.  All launches are asynchronous on
 * the given stream (a cudaStream_t passed as void*; NULL = the default stream).
 * Every function returns a gptq_status (0 = OK, negative = error); nothing throws, aborts
 * or traps.  Arguments are validated on the host before any launch.
 */
#ifndef GPTQ_B200_H
#define GPTQ_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GPTQ_OK = 0,
    GPTQ_ERR_NULL = -1,        /* a required pointer is NULL */
    GPTQ_ERR_SHAPE = -2,       /* M<1, K%8, N%8, K%group_size, group_size<=0 ... */
    GPTQ_ERR_ALIGN = -3,       /* a pointer is not 16-byte aligned */
    GPTQ_ERR_UNSUPPORTED = -4, /* valid GPTQ shape outside the tiled fast path */
    GPTQ_ERR_LAYOUT = -5,      /* bad `which`/flag argument; from gptq_check_status: a layer's tiling does not fit the call */
    GPTQ_ERR_GIDX = -6,        /* g_idx entry out of range, or groups of unequal size (gptq_repack) */
    GPTQ_ERR_WORKSPACE = -7,   /* workspace missing or too small for this call */
    GPTQ_ERR_CUDA = -8,        /* a CUDA runtime call failed (see gptq_last_cuda_error) */
    GPTQ_ERR_TIMEOUT = -9      /* a bounded device-side wait gave up (see gptq_check_status) */
} gptq_status;

/* Static description of a status code. */
const char *gptq_status_string(int status);
/* cudaError_t of the most recent failing runtime call in this process (0 if none). */
int gptq_last_cuda_error(void);

/* ---- bit-exact building blocks on the canonical layout (the format reading) -------- */

/* The nibble unpacking of the paper's Section 1 format ("4-bit quantized weights"), on its own, for bit-exact
 * checks: q_out uint8[K,N] and z_out uint8[G,N] (either may be NULL to skip it).  Any group_size dividing K. */
int gptq_unpack_u8(const int32_t *qweight, const int32_t *qzeros, uint8_t *q_out, uint8_t *z_out,
                   int N, int K, int group_size, void *stream);

/* The dequantisation every kernel of Section 3 performs before its multiply-accumulate (Eq. 14-15 apply it in
 * half precision; here it is written out in fp32 so that there is exactly one right answer):
 * w_out fp32[K,N] = float(q - z) * float(scale), one fp32 multiply (the product is exact).
 * repacked = 0: inputs are canonical; g_idx is the checkpoint's g_idx when act_order != 0.
 * repacked = 1: inputs are the buffers written by gptq_repack and g_idx is its perm_out;
 *               rows are written back in ORIGINAL order, so both modes give identical bits. */
int gptq_dequant_f32(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                     float *w_out, int N, int K, int group_size, int act_order, int repacked,
                     void *stream);

/* Format variants.  The paper (Section 1, Section 4.2) names 4-bit GPTQ without fixing the checkpoint conventions,
 * and checkpoints of the same family differ in two of them:
 *   - group_size: 128 (all of the paper's models), 64 or 32 rows per scale / zero point, or any multiple of 128 that
 *     divides K (256, 512, ... up to K itself: one scale and zero point per output column, "per-channel").  Every tiled
 *     entry point accepts these; the caller passes the checkpoint's group_size to all of them.  Groups coarser than 128
 *     rows are tiled as groups of 128 rows that repeat their group's scale and zero point (the tiled scales and zero
 *     points then take K/128 instead of K/group_size rows: gptq_repack_bytes says how much), so the kernels see a
 *     group-128 layer and the results are those of the checkpoint's own grouping.  gptq_gemm_noalloc and the CTA-pair
 *     switch accept 128 and coarser only.
 *   - the zero point: stored as is (default), or stored minus one (older checkpoints: the kernels add the one
 *     back, so a stored 15 means 16).  Pass GPTQ_FORMAT_ZEROS_MINUS_ONE to the _format entry points below.
 * gptq_repack_format records the flag in a 16-byte trailer behind the tiled zero points (counted in
 * gptq_repack_bytes(1, ...)), so gptq_gemm and gptq_dequant_f32(repacked = 1) need no format argument. */
#define GPTQ_FORMAT_ZEROS_MINUS_ONE 1
/* A third flag concerns the tiled layout only, not the checkpoint: GPTQ_FORMAT_GATE_UP tiles a layer whose N columns
 * are [gate | up] (N / 2 each, the merged first projection of a Llama MLP block - the models of Section 4.1) so that
 * each 128-column panel holds 64 gate columns and the 64 matching up columns; gptq_gemm_silu_mul needs that order and
 * gptq_gemm refuses it.  gptq_dequant_f32(repacked = 1) undoes it: its output is in checkpoint column order. */
#define GPTQ_FORMAT_GATE_UP 2
/* (No counterpart in the paper, whose models run in fp16 - Section 4.1.)  GPTQ_FORMAT_BF16: the scales are bfloat16
 * (1 sign, 8 exponent, 7 fraction bits: the upper half of an fp32) instead of fp16, as in checkpoints served in
 * bfloat16.  The repack moves the 16-bit words unchanged and records the flag; gptq_dequant_f32 then reads the scales
 * as bfloat16 (the fp32 product float(q - z) * s is still exact), and the layer is multiplied with gptq_gemm_bf16, not
 * gptq_gemm.  May be combined with GPTQ_FORMAT_ZEROS_MINUS_ONE; the fused epilogues (and so GPTQ_FORMAT_GATE_UP),
 * gptq_gemm_host and gptq_gemm_noalloc exist for fp16 layers only (gptq_gemm_host_batch_bf16 is the host-resident
 * path). */
#define GPTQ_FORMAT_BF16 4
/* gptq_dequant_f32 with a format for canonical inputs (repacked = 0; GPTQ_FORMAT_GATE_UP is refused there with
 * GPTQ_ERR_LAYOUT); with repacked = 1 the trailer decides and `format` must be 0 or equal to what the layer was
 * repacked with.  Unknown flag bits: GPTQ_ERR_LAYOUT. */
int gptq_dequant_f32_format(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                            float *w_out, int N, int K, int group_size, int act_order, int repacked, int format,
                            void *stream);

/* ---- one-time repack into the tiled layout the matmul kernels stream ---------------- */

/* Byte size of each gptq_repack output: which = 0 qweight_out, 1 qzeros_out, 2 scales_out,
 * 3 perm_out (0 bytes unless act_order).  Sizes equal the canonical ones, plus 16 bytes of format trailer
 * behind the zero points (with group_size > 128: scales and zero points of K/128 groups).  Returns 0 for an invalid
 * argument. */
size_t gptq_repack_bytes(int which, int N, int K, int group_size, int act_order);

/* Re-tiles a canonical layer (what Section 3.2 / Algorithm 2 achieve with wider loads of the original layout is
 * achieved here by storing the weights in the order the kernels stream them).  Fast-path requirements: group_size 32, 64 or a multiple of 128, K % 128 == 0,
 * N % 128 == 0 (else GPTQ_ERR_UNSUPPORTED).  With act_order != 0 the rows are stably sorted
 * by g_idx so that each group's rows are contiguous; perm_out[i] = original index of sorted
 * row i (int32[K]).  g_idx is range-checked on the device and every group must have exactly
 * group_size rows; with act_order this one-time call synchronises the stream and returns GPTQ_ERR_GIDX
 * for either violation (nothing is tiled then).  Outputs must not alias inputs. */
int gptq_repack(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out,
                int N, int K, int group_size, int act_order, void *stream);
/* The same with a format (see above); gptq_repack is format 0. */
int gptq_repack_format(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                       void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out,
                       int N, int K, int group_size, int act_order, int format, void *stream);

/* ---- the matmul ---------------------------------------------------------------------- */

/* Scratch gptq_gemm needs for this problem: with act_order a gathered copy of x (M*K fp16, rounded
 * up to 256 bytes), otherwise 0 (the split-K partial sums stay in shared memory). */
size_t gptq_workspace_bytes(int M, int N, int K, int group_size, int act_order);

/* Registers caller-owned device scratch for later gptq_gemm calls on the current device.  The workspace is
 * shared by all calls: calls that may overlap on the GPU (different streams) must not share one.
 * ptr = NULL unregisters.  ptr must be 16-byte aligned (GPTQ_ERR_ALIGN). */
int gptq_set_workspace(void *ptr, size_t bytes);

/* The GPTQ linear layer of Sections 1 and 3 (the product all three of the paper's optimisations serve; Section
 * 4.4's last paragraph fixes what "the same result" means: equal up to summation order).
 * y fp16[M,N] = x fp16[M,K] . dequant(W).  qweight/qzeros/scales are the REPACKED buffers from
 * gptq_repack; with act_order != 0, g_idx is gptq_repack's perm_out (16-byte aligned like every other pointer, else
 * GPTQ_ERR_ALIGN; without act-order it may be NULL).
 * fp32 accumulation, one round-to-nearest-even conversion to fp16.  Any M >= 1.  Up to 16 rows the
 * weights enter the MMA as exact integers q - z and the scale multiplies fp32 group sums; above
 * that each scaled weight is rounded to fp16 once before the MMA.
 * The kernels begin fetching weights before earlier work on the stream has finished
 * (programmatic dependent launch); x, y and the workspace are only touched afterwards.  The
 * weight buffers must therefore not be written by a kernel launched immediately before this
 * call on the same stream (gptq_repack itself is safe).
 * Thread safety: calls from several host threads are allowed (the library's own host state is locked);
 * GPU work of calls on different streams may overlap unless they share the act-order workspace.
 * Accuracy: the stated bar |y - y_exact| <= 1e-2 sqrt(K/4096) + 1e-2 |y_exact| holds for the Llama shapes
 * (K >= 4096).  Above 16 token rows the fp16 rounding of each scaled weight gives y an error of about
 * 1.4e-3 sqrt(K/4096) rms for unit-variance x; since the bar shrinks with sqrt(K) as fast as that error does
 * but a layer with very few groups (K <= 256) has columns whose few scales are all large, single elements
 * among millions can exceed the bar there (seen: 1 of 5e6 at K = 256, by a factor of 2). */
int gptq_gemm(const void *x, const void *qweight, const void *qzeros, const void *scales,
              const int32_t *g_idx, void *y, int M, int N, int K, int group_size, int act_order,
              void *stream);

/* (No counterpart in the paper: the product of Sections 1 and 3 in the other 16-bit float format.)
 * y bf16[M,N] = x bf16[M,K] . dequant(W)[K,N] for a layer repacked with GPTQ_FORMAT_BF16: x, y and the scales are
 * bfloat16, everything else (arguments, layouts, act_order values, workspace, stream semantics, error codes, kernels
 * chosen by M) as for gptq_gemm.  Up to 16 token rows the exact integers q - z are multiplied with x on the tensor
 * cores (mma.sync, bf16 operands, fp32 sums) and the scale joins the fp32 group sums; above, each weight is rounded
 * once to bfloat16 after scaling (relative error up to 2^-8) and multiplied by tcgen05.mma with bf16 operands; y is rounded
 * once from the fp32 sum.  A layer of the other format (fp16 layer here, bfloat16 layer in gptq_gemm or any other
 * matmul entry point) is refused: nothing is stored and gptq_check_status returns GPTQ_ERR_LAYOUT.
 * Accuracy: the bar of gptq_gemm, |y - y_exact| <= 1e-2 sqrt(K/4096) + 1e-2 |y_exact|, holds with the same caveat; the
 * output rounding alone is up to 2^-8 |y|. */
int gptq_gemm_bf16(const void *x, const void *qweight, const void *qzeros, const void *scales,
                   const int32_t *g_idx, void *y, int M, int N, int K, int group_size, int act_order,
                   void *stream);

/* act_order argument of the matmul entry points: 0 = groups are consecutive rows; 1 = act-order, the call first
 * gathers x into the sorted row order with g_idx (= gptq_repack's perm_out); GPTQ_ACT_ORDER_PRESORTED = act-order, but
 * x already is in the sorted row order (its producer wrote it that way, see gptq_gemm_silu_mul_scatter): no gather,
 * no workspace, g_idx is ignored and may be NULL.  gptq_gemm_noalloc takes 0 and 1 only. */
#define GPTQ_ACT_ORDER_PRESORTED 2

/* (No counterpart in the paper: additions fused into the epilogue of the product of Sections 1 and 3.)
 * y fp16[M,N] = x . dequant(W) + bias[n] + residual[m][n]: the bias of a projection (fp16 [N]) and the residual add
 * that follows the o and down projections of a Llama block (fp16 [M,N]), joined to the fp32 sums before the one
 * rounding to fp16.  Either pointer may be NULL (adds nothing); both NULL is gptq_gemm.  residual may be y itself
 * (h += proj(x)): each element is read and then written by the same thread.  Both must be 16-byte aligned and are
 * read after earlier work on the stream has finished.  Other arguments, layouts, accuracy and errors as for
 * gptq_gemm; a layer tiled with GPTQ_FORMAT_GATE_UP is refused the same way.  The CTA-pair switch does not apply. */
int gptq_gemm_bias_residual(const void *x, const void *qweight, const void *qzeros, const void *scales,
                            const int32_t *g_idx, const void *bias, const void *residual, void *y,
                            int M, int N, int K, int group_size, int act_order, void *stream);

/* (No counterpart in the paper: an epilogue fused into the product of Sections 1 and 3.)
 * out fp16[M, N / 2] = silu(y[:, :N/2]) * y[:, N/2:], silu(g) = g / (1 + exp(-g)), for y = x . dequant(W) of a layer
 * repacked with GPTQ_FORMAT_GATE_UP: the activation of a Llama MLP block applied before the product leaves the chip,
 * so y itself is never written.  Other arguments as for gptq_gemm; N counts both halves.  Up to 16 token rows the
 * two factors are the fp32 sums; above that each is rounded to fp16 first unless the K range was split across CTAs;
 * silu and the product are evaluated in fp32 (fast exponential, relative error ~1e-6), then rounded to fp16 once.
 * A layer repacked without the flag (or a flagged layer given to gptq_gemm / gptq_gemm_noalloc) stores nothing and
 * makes the next gptq_check_status return GPTQ_ERR_LAYOUT.  The CTA-pair switch below does not apply to it. */
int gptq_gemm_silu_mul(const void *x, const void *qweight, const void *qzeros, const void *scales,
                       const int32_t *g_idx, void *out, int M, int N, int K, int group_size, int act_order,
                       void *stream);

/* (No counterpart in the paper.)  gptq_gemm_silu_mul whose output column i is stored at column out_index[i] of `out`
 * (int32 [N / 2], device, 16-byte aligned, a permutation of 0 .. N/2 - 1): with out_index = the inverse of the sort
 * permutation of an act-order layer that consumes `out` (gptq_invert_perm of that layer's perm_out), `out` is written in
 * that layer's sorted row order and its matmul can run with GPTQ_ACT_ORDER_PRESORTED - the separate gather launch of
 * act-order and its round trip through memory disappear.  Meant for decode-sized M: the stores are 2 bytes each. */
int gptq_gemm_silu_mul_scatter(const void *x, const void *qweight, const void *qzeros, const void *scales,
                               const int32_t *g_idx, const int32_t *out_index, void *out, int M, int N, int K,
                               int group_size, int act_order, void *stream);
/* inverse[perm[i]] = i for i < K (perm a permutation of 0 .. K-1, e.g. gptq_repack's perm_out; entries out of range are
 * skipped). */
int gptq_invert_perm(const int32_t *perm, int32_t *inverse, int K, void *stream);

/* ---- 2- and 3-bit weights (no counterpart in the paper, which treats 4-bit GPTQ only - Section 1) -----------------
 * Checkpoint layout: the values of a column (weights, along K) or of a group's row (zero points, along N) form one bit
 * stream, value i in bits [bits * i, bits * i + bits) of the little-endian concatenation of that column's / row's
 * 32-bit words: qweight int32[K * bits / 32, N], qzeros int32[G, N * bits / 32] (2 bits: 16 values per word; 3 bits: 32
 * values per three words).  K and N must be multiples of 32 (GPTQ_ERR_SHAPE).  gptq_repack_bits widens every field to a
 * nibble and writes an ordinary tiled 4-bit layer - same output sizes as gptq_repack (gptq_repack_bytes), same perm_out,
 * to be used with gptq_gemm and the other 4-bit entry points with act_order as given here.  The tiled layer streams the
 * bytes of a 4-bit layer: these widths are supported, not accelerated.  bits other than 2 or 3: GPTQ_ERR_UNSUPPORTED.
 * format: 0 or GPTQ_FORMAT_ZEROS_MINUS_ONE (the one is added during the repack; the tiled layer stores zero points as
 * they are).  scratch: device, 256-byte aligned, gptq_repack_bits_scratch_bytes (about K * N / 2); GPTQ_ERR_WORKSPACE if
 * smaller; free once the stream has passed the call.  Other arguments and errors as for gptq_repack. */
size_t gptq_repack_bits_scratch_bytes(int bits, int N, int K, int group_size);
int gptq_repack_bits(int bits, const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                     void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, void *scratch,
                     size_t scratch_bytes, int N, int K, int group_size, int act_order, int format, void *stream);
/* fp32 w[K, N] of a canonical 2- or 3-bit layer, bit-exact (for the repacked layer use gptq_dequant_f32, repacked = 1). */
int gptq_dequant_f32_bits(int bits, const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                          float *w_out, int N, int K, int group_size, int act_order, int format, void *stream);

/* ---- 8-bit weights (no counterpart in the paper, which treats 4-bit GPTQ only - Section 1) ------------------------
 * The checkpoint conventions at twice the field width: qweight int32[K/4, N], byte i of a word = row 4 r + i (least
 * significant first); qzeros int32[G, N/4], byte j of a word = column 4 c + j; scales fp16[G, N]; g_idx int32[K].
 * w[k,n] = (q - z) * s with q, z in 0..255 (GPTQ_FORMAT_ZEROS_MINUS_ONE: the stored byte is z - 1; a stored 255 under
 * that convention, z = 256, is refused with GPTQ_ERR_UNSUPPORTED).
 * An 8-bit weight is two nibbles, (q - z) s = (hi - zh) (16 s) + (lo - zl) s: gptq_repack_w8 stores the layer as a 4-bit
 * layer of 2 K rows (rows 0..K-1 the high nibbles with scales 16 s, rows K..2K-1 the low nibbles) in the usual tiled
 * layout, and gptq_gemm_w8 gathers x into [x | x] in that layer's row order and runs the 4-bit kernels on 2 K rows.  One
 * byte per weight is streamed, as the format requires; scales and zero points take twice their canonical bytes.
 * Requirements: as gptq_repack (group_size 32, 64 or a multiple of 128; K % 128 == 0; N % 128 == 0), scales < 4096. */

/* Bytes of each output of gptq_repack_w8: which = 0 qweight_out, 1 qzeros_out, 2 scales_out, 3 perm_out (int32[2 K],
 * always needed).  0 for an invalid argument. */
size_t gptq_repack_w8_bytes(int which, int N, int K, int group_size);
/* Bytes of the device scratch buffer gptq_repack_w8 needs (about K * N: the two planes in canonical 4-bit form). */
size_t gptq_repack_w8_scratch_bytes(int N, int K, int group_size);
/* One-time repack of a canonical 8-bit layer.  All pointers are device pointers; outputs 16-byte aligned, scratch
 * 256-byte aligned and of at least gptq_repack_w8_scratch_bytes (GPTQ_ERR_WORKSPACE otherwise); it may be freed once the
 * stream has passed the call.  g_idx may be NULL when act_order is 0.  perm_out[i] (i < 2 K) is the column of x that row i
 * of the stacked layer multiplies.  The call synchronises the stream (it reads back the validation results: GPTQ_ERR_GIDX
 * as for gptq_repack, GPTQ_ERR_UNSUPPORTED for a zero point of 256).  format: 0 or GPTQ_FORMAT_ZEROS_MINUS_ONE. */
int gptq_repack_w8(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                   void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, void *scratch,
                   size_t scratch_bytes, int N, int K, int group_size, int act_order, int format, void *stream);
/* fp32 w[K, N] of an 8-bit layer, bit-exact (the product float(q - z) * float(s) is exact): repacked = 0 reads the
 * canonical buffers (g_idx used when act_order != 0, format as above); repacked = 1 reads gptq_repack_w8's outputs,
 * g_idx = its perm_out (required), and recombines the two planes. */
int gptq_dequant_f32_w8(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx, float *w_out,
                        int N, int K, int group_size, int act_order, int repacked, int format, void *stream);
/* y fp16[M, N] = x fp16[M, K] . dequant(W8)[K, N] for the outputs of gptq_repack_w8 (perm = its perm_out, 16-byte
 * aligned).  Needs the registered workspace: gptq_workspace_bytes(M, N, 2 * K, group_size, 1) bytes, for the gathered
 * activations.  K and group_size are the checkpoint's.  Stream semantics, kernels by M, accuracy bar and error codes as
 * for gptq_gemm with act_order = 1; up to 16 token rows the integers are exact and the scales join in fp32, above that
 * each plane's scaled weight is rounded to fp16 once. */
int gptq_gemm_w8(const void *x, const void *qweight, const void *qzeros, const void *scales, const int32_t *perm,
                 void *y, int M, int N, int K, int group_size, void *stream);

/* Process-wide switch: with enable != 0, gptq_gemm runs problems with M >= 256 and an even number
 * of 128-column panels on CTA pairs (tcgen05.mma.cta_group::2: two SMs share one 256 x 256 x 16 MMA and
 * each loads half of the x tile).  Same arithmetic and tolerance as the default kernel; it halves the
 * L2 traffic per flop but measured slower on the Llama shapes, so it is off by default. */
int gptq_set_cta_pairs(int enable);

/* The same product for callers whose activations live in host memory: copies x_host (pinned
 * for true asynchrony) to x_stage, runs gptq_gemm, copies y_stage to y_host, all on `stream`.
 * x_stage (M*K fp16) and y_stage (M*N fp16) are caller-owned device buffers. */
int gptq_gemm_host(const void *x_host, const void *qweight, const void *qzeros, const void *scales,
                   const int32_t *g_idx, void *y_host, void *x_stage, void *y_stage,
                   int M, int N, int K, int group_size, int act_order, void *stream);

/* (No counterpart in the paper: a packaging variant of gptq_gemm.)
 * The same product as gptq_gemm for callers that cannot hand the library a workspace because
 * they cannot allocate device memory at all: code hosted inside a serving process whose device
 * memory was partitioned at start-up and where a later cudaMalloc is forbidden or would stall
 * the whole device (cudaMalloc/cudaFree synchronise it), such as a decode loop with a latency
 * budget.  The split-K partial tiles, their tickets and (act-order) the gathered activations
 * live in an 8 MiB array that is part of the library image: every GPU that loads the library
 * holds it until the process exits.  Arguments, layouts and arithmetic are those of gptq_gemm.
 *  - Problems whose scratch need (gptq_plan_noalloc's workspace_bytes) exceeds gptq_noalloc_scratch_bytes()
 *    are refused with GPTQ_ERR_WORKSPACE; nothing is launched.  (All decode shapes of the 7B
 *    and 13B layers fit up to M = 16.)
 *  - The call allocates and frees nothing, on the device or through any library.
 *  - The first call on each device looks up the array's device address (the device must be
 *    current, as for every call); make that first call before any stream capture begins.
 *  - All calls share the one array, which keeps the previous call's contents; each call clears
 *    the tickets it needs on `stream` first.  Calls that can overlap on the GPU (different
 *    streams, several host threads) race on it: serialise them, or use gptq_gemm with
 *    per-stream workspaces. */
int gptq_gemm_noalloc(const void *x, const void *qweight, const void *qzeros, const void *scales,
                      const int32_t *g_idx, void *y, int M, int N, int K, int group_size, int act_order,
                      void *stream);
/* Size in bytes of the built-in scratch array (host-only, no CUDA call). */
size_t gptq_noalloc_scratch_bytes(void);

/* One matmul of a step for gptq_gemm_host_batch: the arguments of gptq_gemm_host. */
typedef struct {
    const void *x_host;      /* fp16 [M, K], host (pinned for true asynchrony) */
    const void *qweight;     /* device, repacked */
    const void *qzeros;      /* device, repacked */
    const void *scales;      /* device, repacked */
    const int32_t *g_idx;    /* device perm_out, or NULL */
    void *y_host;            /* fp16 [M, N], host */
    void *x_stage;           /* device, M*K fp16 */
    void *y_stage;           /* device, M*N fp16 */
    int M, N, K, group_size, act_order;
} gptq_host_problem_t;

/* A step of matmuls whose activations live in host memory (the linears of a decode step, configs of
 * Section 4's serving setting): for each problem in order, on `stream`: copy x to the device, gptq_gemm,
 * copy y back - the same results as `count` gptq_gemm_host calls, but pipelined: the copies run on two
 * internal streams (created on first use) in chunks of consecutive problems (up to 16, up to 2 MiB of activations and
 * results, none sharing a staging buffer with another of the last few chunks; large problems go one by one): the x of a chunk go up, its matmuls run back to back on `stream`, its y come down, and chunk c+1 goes up
 * while chunk c computes and chunk c-1 comes down; the matmuls themselves stay in order on `stream`, and `stream`
 * completes after the last copy.  Staging buffers may be shared between problems (reuse waits for the earlier user;
 * problems that share one never sit in the same chunk).
 * All problems are validated before anything is enqueued; on an invalid problem *bad_index (if not
 * NULL) receives its index and nothing runs.  If a later step fails, `stream` is still joined with the
 * internal streams before the error is returned.  The internal streams and events belong to the device:
 * concurrent calls on one device (several host threads, or several user streams) are serialised by a lock
 * for the duration of the enqueue.  The call is stream-ordered (the internal streams fork from `stream` and join it
 * again), so after one ordinary call - which creates the internal streams and events - it may be captured into a CUDA
 * graph and replayed: every replay copies the host buffers as they are then. */
int gptq_gemm_host_batch(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index);
/* The same pipeline for bfloat16 layers: every problem's x_host / y_host hold bfloat16 and its layer was repacked with
 * GPTQ_FORMAT_BF16; each matmul is a gptq_gemm_bf16.  Arguments, ordering and errors as above. */
int gptq_gemm_host_batch_bf16(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index);
/* The same pipeline for 8-bit layers (gptq_repack_w8): each matmul is a gptq_gemm_w8; a problem's g_idx is the layer's
 * perm_out (required), act_order is ignored, K and group_size are the checkpoint's, and the registered workspace must
 * cover the largest problem (gptq_workspace_bytes(M, N, 2 * K, group_size, 1)). */
int gptq_gemm_host_batch_w8(const gptq_host_problem_t *problems, int count, void *stream, int *bad_index);

/* Synchronises `stream` and returns GPTQ_ERR_LAYOUT if a kernel since the last check met a layer whose tiling does
 * not fit the call (see GPTQ_FORMAT_GATE_UP), GPTQ_ERR_TIMEOUT if a kernel's bounded wait gave up (the flag is
 * cleared either way), GPTQ_ERR_CUDA on a runtime error, else OK. */
int gptq_check_status(void *stream);

/* Self-test of that mechanism (no counterpart in the paper): launches one thread that waits, the way the matmul
 * kernels wait, on a barrier nothing will ever complete, gives up after limit_us microseconds (1 .. 1e6) and
 * returns normally; the next gptq_check_status then reports GPTQ_ERR_TIMEOUT.  Nothing faults or hangs. */
int gptq_selftest_wait_timeout(unsigned int limit_us, void *stream);

/* ---- launch timeline (no counterpart in the paper: a tracing aid) ------------------------ */

/* A library built with -DGPTQ_TIMELINE (GPTQ_NVCC_EXTRA=-DGPTQ_TIMELINE for the Python build) gives every matmul launch
 * the next of 64 rows (round robin) in which its CTAs record %globaltimer times: first and last CTA started, first weight
 * copy issued, griddepcontrol.wait first / last returned, first activation tile landed, last CTA done - what shows
 * whether consecutive launches overlap.  gptq_trace_reset clears the rows (synchronises `stream`); gptq_trace_read
 * synchronises `stream`, copies up to max_rows rows of eight 64-bit values {first_entry, first_weight_issue,
 * first_wait_done, last_wait_done, first_data, last_exit, kernel (1 mma.sync, 2 tcgen05) << 32 | CTAs, last_entry} (times in
 * nanoseconds) to host
 * memory and returns the number of rows.  A row nobody wrote keeps ~0 in its "first" fields.  In a normal build both
 * return GPTQ_ERR_UNSUPPORTED and the kernels carry no tracing code.  `python -m paper_2511_19438_b200.timeline` prints
 * the table for a chain of decode launches. */
int gptq_trace_reset(void *stream);
int gptq_trace_read(unsigned long long *rows_out, int max_rows, void *stream);

/* ---- host-only: how a problem would be launched (no CUDA call; usable without a GPU) -- */

typedef struct {
    char kernel_name[48]; /* the kernel instantiation, e.g. "splitk_kernel<1,1>": a profiler prints the same integers, followed by the
                             bfloat16 flag (false for gptq_gemm, true for gptq_gemm_bf16) */
    int kernel;       /* 1 = cluster split-K mma.sync kernel (gptq_gemm, M <= 16),
                         2 = tcgen05 kernel (gptq_gemm, M >= 17),
                         3 = stream-K mma.sync kernel (gptq_gemm_noalloc) */
    int m_tile;       /* tokens per CTA tile */
    int m_chunks;     /* launches along M */
    int stages;       /* pipeline depth */
    int ctas;         /* grid size of one launch */
    int items;        /* (128-column panel, 128-row group) work items of one launch */
    int split_panels; /* panels whose K range is shared by several CTAs */
    int smem_bytes;   /* dynamic shared memory per CTA */
    size_t workspace_bytes;
    int cluster_size; /* CTAs that share one panel (kernel 1) or one output tile (kernel 2); 1 for kernel 3 */
    int tail_ctas;    /* kernel 2 only: grid of a second launch that takes the tiles of a partly filled last
                         wave and splits K over clusters (`ctas` is then the first launch alone); 0 = none */
    int tail_cluster_size; /* cluster size of that second launch (1 when there is none) */
} gptq_plan_t;

/* How gptq_gemm would launch this problem on a GPU with sm_count SMs. */
int gptq_plan(int M, int N, int K, int group_size, int act_order, int sm_count, gptq_plan_t *out);
/* The same for gptq_gemm_noalloc (stream-K kernel; workspace_bytes is its need of the built-in scratch). */
int gptq_plan_noalloc(int M, int N, int K, int group_size, int act_order, int sm_count, gptq_plan_t *out);

/* For tests only (not needed to use the library): the stream-K partition gptq_gemm_noalloc's kernel uses, from
 * the same arithmetic as the kernel.  CTA `cta` of `ctas` works
 * through items [*first_item, *end_item) of `items`; the K range of panel `panel` (its `groups`
 * consecutive items) is shared by CTAs *first_cta .. *last_cta, whose partial tiles are summed
 * in that order. */
int gptq_plan_cta_range(int items, int ctas, int cta, int *first_item, int *end_item);
int gptq_plan_panel_owners(int items, int ctas, int groups, int panel, int *first_cta, int *last_cta);

#ifdef __cplusplus
}
#endif
#endif /* GPTQ_B200_H */
