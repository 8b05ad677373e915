/*
 * CPU oracle for the GPTQ 4-bit weight-only matmul  y[M,N] = x[M,K] . dequant(W)[K,N].
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or helper
 * with the CUDA path and must never be linked into or called from it.
 *
 * What it follows.  The paper (Opt4GPTQ, Section 1 and Section 4.2) accelerates
 * the 4-bit GPTQ linear layer with fp16 activations and states (Section 4.4,
 * last paragraph) that its kernels equal plain GPTQ up to floating-point
 * summation order.  So the oracle is the plain definition itself:
 *
 *   q[k][n]  = nibble (k mod 8) of qweight[k/8][n]     (LSB first, word as uint32)
 *   z[g][n]  = nibble (n mod 8) of qzeros[g][n/8]
 *   g(k)     = g_idx[k] if act-order else k / group_size
 *   w32[k][n]= float(q[k][n] - z[g(k)][n]) * float(scales[g(k)][n])   one fp32 multiply
 *   y[m][n]  = sum_{k ascending} double(x[m][k]) * double(w32[k][n])  fp64
 *
 * The paper never spells the storage format out; the reading above (LSB-first
 * nibbles, stored zero point used as is, unsigned shifts) is the one the tests
 * pin with hand-packed words.  The fp32 product is exact (|q-z| <= 15 needs 4
 * bits, an fp16 significand 11), so there is one right dequantised value.
 *
 * Parity with numbers printed in the paper: unpinned - the paper prints no value
 * for this computation.  Each function is pinned by the mathematics instead
 * (hand-packed words, brute force, closed forms, special cases); see tests/.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE-754 binary16 -> binary32, written from the format definition:
 * 1 sign, 5 exponent (bias 15), 10 fraction bits. */
float oracle_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t exp = (uint32_t)(h >> 10) & 0x1Fu;
    uint32_t frac = (uint32_t)h & 0x3FFu;
    uint32_t bits;
    if (exp == 0) {
        if (frac == 0) {
            bits = sign << 31;                           /* signed zero */
        } else {                                         /* subnormal: frac * 2^-24 */
            int e = -1;
            do { frac <<= 1; e++; } while ((frac & 0x400u) == 0);
            frac &= 0x3FFu;
            bits = (sign << 31) | ((uint32_t)(127 - 15 - e) << 23) | (frac << 13);
        }
    } else if (exp == 31) {
        bits = (sign << 31) | 0x7F800000u | (frac << 13); /* inf / nan */
    } else {
        bits = (sign << 31) | ((exp + 127 - 15) << 23) | (frac << 13);
    }
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static inline unsigned nibble(int32_t word, int i)
{
    return ((uint32_t)word >> (4 * i)) & 15u;
}

/* Step 1: q[k][n] for all k < K, n < N. */
void oracle_unpack_q(const int32_t *qweight, int K, int N, uint8_t *q_out)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            q_out[(size_t)k * N + n] = (uint8_t)nibble(qweight[(size_t)(k >> 3) * N + n], k & 7);
}

/* Step 2: z[g][n] for all g < G, n < N. */
void oracle_unpack_z(const int32_t *qzeros, int G, int N, uint8_t *z_out)
{
    for (int g = 0; g < G; g++)
        for (int n = 0; n < N; n++)
            z_out[(size_t)g * N + n] = (uint8_t)nibble(qzeros[(size_t)g * (N / 8) + (n >> 3)], n & 7);
}

static inline int group_of(const int32_t *g_idx, int k, int group_size)
{
    return g_idx ? g_idx[k] : k / group_size;
}

static inline float dequant_one(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                                const int32_t *g_idx, int N, int group_size, int k, int n)
{
    int g = group_of(g_idx, k, group_size);
    int q = (int)nibble(qweight[(size_t)(k >> 3) * N + n], k & 7);
    int z = (int)nibble(qzeros[(size_t)g * (N / 8) + (n >> 3)], n & 7);
    float s = oracle_half_to_float(scales[(size_t)g * N + n]);
    return (float)(q - z) * s;
}

/* Steps 3-4: w32[k][n].  g_idx may be NULL (no act-order). */
void oracle_dequant_f32(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                        const int32_t *g_idx, int K, int N, int group_size, float *w_out)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            w_out[(size_t)k * N + n] = dequant_one(qweight, qzeros, scales, g_idx, N, group_size, k, n);
}

/* Step 5: y[m][n] in fp64, k ascending. */
void oracle_gemm_f64(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                     const uint16_t *scales, const int32_t *g_idx,
                     int M, int N, int K, int group_size, double *y_out)
{
    #pragma omp parallel for schedule(static)
    for (int n = 0; n < N; n++) {
        for (int m = 0; m < M; m++) {
            double acc = 0.0;
            for (int k = 0; k < K; k++) {
                float w = dequant_one(qweight, qzeros, scales, g_idx, N, group_size, k, n);
                acc += (double)oracle_half_to_float(x[(size_t)m * K + k]) * (double)w;
            }
            y_out[(size_t)m * N + n] = acc;
        }
    }
}

/* Step 5 on chosen outputs only: y_out[i] = y[rows[i]][cols[i]], the same sum,
 * for spot checks at sizes where the full product would take too long. */
void oracle_gemm_f64_at(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                        const uint16_t *scales, const int32_t *g_idx,
                        int M, int N, int K, int group_size,
                        const int32_t *rows, const int32_t *cols, int count, double *y_out)
{
    (void)M;
    #pragma omp parallel for schedule(static)
    for (int i = 0; i < count; i++) {
        int m = rows[i], n = cols[i];
        double acc = 0.0;
        for (int k = 0; k < K; k++) {
            float w = dequant_one(qweight, qzeros, scales, g_idx, N, group_size, k, n);
            acc += (double)oracle_half_to_float(x[(size_t)m * K + k]) * (double)w;
        }
        y_out[i] = acc;
    }
}

/* ---- format variant: zero points stored minus one -------------------------------------------
 * Older GPTQ checkpoints store z - 1 in the zero-point nibble and the kernels that read them add
 * the one back; the paper (Section 1, Section 4.2) does not say which of the two conventions its
 * checkpoints use, so both are defined.  The functions above take the stored nibble as the zero
 * point; the two below take stored + 1 (1..16), everything else unchanged. */
static inline float dequant_one_v1(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                                   const int32_t *g_idx, int N, int group_size, int k, int n)
{
    int g = group_of(g_idx, k, group_size);
    int q = (int)nibble(qweight[(size_t)(k >> 3) * N + n], k & 7);
    int z = (int)nibble(qzeros[(size_t)g * (N / 8) + (n >> 3)], n & 7) + 1;
    float s = oracle_half_to_float(scales[(size_t)g * N + n]);
    return (float)(q - z) * s;
}

void oracle_dequant_f32_v1(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                           const int32_t *g_idx, int K, int N, int group_size, float *w_out)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            w_out[(size_t)k * N + n] = dequant_one_v1(qweight, qzeros, scales, g_idx, N, group_size, k, n);
}

void oracle_gemm_f64_v1(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                        const uint16_t *scales, const int32_t *g_idx,
                        int M, int N, int K, int group_size, double *y_out)
{
    #pragma omp parallel for schedule(static)
    for (int n = 0; n < N; n++) {
        for (int m = 0; m < M; m++) {
            double acc = 0.0;
            for (int k = 0; k < K; k++) {
                float w = dequant_one_v1(qweight, qzeros, scales, g_idx, N, group_size, k, n);
                acc += (double)oracle_half_to_float(x[(size_t)m * K + k]) * (double)w;
            }
            y_out[(size_t)m * N + n] = acc;
        }
    }
}

/* ---- the gated-MLP neighbour of the gate_up projection ---------------------------------------
 * In the Llama-class models the paper serves (Section 4.1), the columns of the fused gate_up projection are
 * [gate | up] and the next operation is out[m][i] = silu(gate[m][i]) * up[m][i], silu(t) = t / (1 + exp(-t)).
 * The paper's kernels stop at the matmul; the library can fuse this step into the matmul's epilogue, and this
 * is its definition: y is the fp64 matmul result [M, 2 I], out is [M, I]. */
void oracle_silu_mul_f64(const double *y, int M, int I, double *out)
{
    for (int m = 0; m < M; m++)
        for (int i = 0; i < I; i++) {
            double g = y[(size_t)m * 2 * I + i], u = y[(size_t)m * 2 * I + I + i];
            out[(size_t)m * I + i] = g / (1.0 + exp(-g)) * u;
        }
}

/* ---- the additive neighbours of a projection -------------------------------------------------
 * A linear layer of the served models may carry a bias (one fp16 value per output column), and the o and down
 * projections of a Llama-class block (Section 4.1) are followed by the residual add h = h + proj(...).  The paper's
 * kernels stop at the matmul; the library can fuse both additions into the matmul's epilogue, and this is their
 * definition: out[m][n] = y[m][n] + bias[n] + residual[m][n] in fp64, y the fp64 matmul result [M, N]; bias (fp16
 * bits, [N]) and residual (fp16 bits, [M, N]) may each be NULL (then it adds nothing). */
void oracle_add_bias_residual_f64(const double *y, const uint16_t *bias, const uint16_t *residual, int M, int N,
                                  double *out)
{
    for (int m = 0; m < M; m++)
        for (int n = 0; n < N; n++) {
            double v = y[(size_t)m * N + n];
            if (bias) v += (double)oracle_half_to_float(bias[n]);
            if (residual) v += (double)oracle_half_to_float(residual[(size_t)m * N + n]);
            out[(size_t)m * N + n] = v;
        }
}

/* ---- format variant: bfloat16 activations and scales ------------------------------------------
 * The paper's models run in fp16 (Section 4.1); the same checkpoints are also served with bfloat16
 * activations and scales, and the method is unchanged: only the two 16-bit number formats differ.
 * bfloat16 is the upper half of an IEEE-754 binary32 (1 sign, 8 exponent, 7 fraction bits), so its
 * value is the binary32 whose upper 16 bits it is and whose lower 16 bits are zero.  The product
 * float(q - z) * s stays exact in fp32 (4 bits times an 8-bit significand).
 * zeros_plus = 0: the stored nibble is the zero point; 1: it is the zero point minus one. */
float oracle_bfloat16_to_float(uint16_t b)
{
    uint32_t bits = (uint32_t)b << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

static inline float dequant_one_bf16(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                                     const int32_t *g_idx, int N, int group_size, int zeros_plus, int k, int n)
{
    int g = group_of(g_idx, k, group_size);
    int q = (int)nibble(qweight[(size_t)(k >> 3) * N + n], k & 7);
    int z = (int)nibble(qzeros[(size_t)g * (N / 8) + (n >> 3)], n & 7) + zeros_plus;
    float s = oracle_bfloat16_to_float(scales[(size_t)g * N + n]);
    return (float)(q - z) * s;
}

void oracle_dequant_f32_bf16(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                             const int32_t *g_idx, int K, int N, int group_size, int zeros_plus, float *w_out)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            w_out[(size_t)k * N + n] = dequant_one_bf16(qweight, qzeros, scales, g_idx, N, group_size, zeros_plus, k, n);
}

/* y[m][n] in fp64, k ascending; x and scales are bfloat16 bits. */
void oracle_gemm_f64_bf16(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                          const uint16_t *scales, const int32_t *g_idx,
                          int M, int N, int K, int group_size, int zeros_plus, double *y_out)
{
    #pragma omp parallel for schedule(static)
    for (int n = 0; n < N; n++) {
        for (int m = 0; m < M; m++) {
            double acc = 0.0;
            for (int k = 0; k < K; k++) {
                float w = dequant_one_bf16(qweight, qzeros, scales, g_idx, N, group_size, zeros_plus, k, n);
                acc += (double)oracle_bfloat16_to_float(x[(size_t)m * K + k]) * (double)w;
            }
            y_out[(size_t)m * N + n] = acc;
        }
    }
}

/* The same sum on chosen outputs only: y_out[i] = y[rows[i]][cols[i]]. */
void oracle_gemm_f64_bf16_at(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                             const uint16_t *scales, const int32_t *g_idx,
                             int M, int N, int K, int group_size, int zeros_plus,
                             const int32_t *rows, const int32_t *cols, int count, double *y_out)
{
    (void)M;
    #pragma omp parallel for schedule(static)
    for (int i = 0; i < count; i++) {
        int m = rows[i], n = cols[i];
        double acc = 0.0;
        for (int k = 0; k < K; k++) {
            float w = dequant_one_bf16(qweight, qzeros, scales, g_idx, N, group_size, zeros_plus, k, n);
            acc += (double)oracle_bfloat16_to_float(x[(size_t)m * K + k]) * (double)w;
        }
        y_out[i] = acc;
    }
}

/* ---- format variant: 8-bit weights -------------------------------------------------------------
 * The paper treats 4-bit GPTQ only (Section 1); the same checkpoints family also stores 8-bit
 * weights, with the same conventions at twice the field width (this reading is pinned by hand-packed
 * words in the tests, like the 4-bit one):
 *   q[k][n] = byte (k mod 4) of qweight[k/4][n]   (LSB first; qweight is int32[K/4][N])
 *   z[g][n] = byte (n mod 4) of qzeros[g][n/4]    (qzeros is int32[G][N/4]), + zeros_plus (0 or 1)
 *   w32[k][n] = float(q - z) * float(scales[g(k)][n])   exact: |q - z| <= 256 needs 9 bits
 *   y[m][n] = sum_{k ascending} double(x[m][k]) * double(w32[k][n]) */
static inline unsigned byte_of(int32_t word, int i)
{
    return ((uint32_t)word >> (8 * i)) & 255u;
}

void oracle_unpack_q8(const int32_t *qweight, int K, int N, uint8_t *q_out)
{
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            q_out[(size_t)k * N + n] = (uint8_t)byte_of(qweight[(size_t)(k >> 2) * N + n], k & 3);
}

void oracle_unpack_z8(const int32_t *qzeros, int G, int N, uint8_t *z_out)
{
    for (int g = 0; g < G; g++)
        for (int n = 0; n < N; n++)
            z_out[(size_t)g * N + n] = (uint8_t)byte_of(qzeros[(size_t)g * (N / 4) + (n >> 2)], n & 3);
}

static inline float dequant_one_w8(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                                   const int32_t *g_idx, int N, int group_size, int zeros_plus, int k, int n)
{
    int g = group_of(g_idx, k, group_size);
    int q = (int)byte_of(qweight[(size_t)(k >> 2) * N + n], k & 3);
    int z = (int)byte_of(qzeros[(size_t)g * (N / 4) + (n >> 2)], n & 3) + zeros_plus;
    float s = oracle_half_to_float(scales[(size_t)g * N + n]);
    return (float)(q - z) * s;
}

void oracle_dequant_f32_w8(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                           const int32_t *g_idx, int K, int N, int group_size, int zeros_plus, float *w_out)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            w_out[(size_t)k * N + n] = dequant_one_w8(qweight, qzeros, scales, g_idx, N, group_size, zeros_plus, k, n);
}

void oracle_gemm_f64_w8(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                        const uint16_t *scales, const int32_t *g_idx,
                        int M, int N, int K, int group_size, int zeros_plus, double *y_out)
{
    #pragma omp parallel for schedule(static)
    for (int n = 0; n < N; n++) {
        for (int m = 0; m < M; m++) {
            double acc = 0.0;
            for (int k = 0; k < K; k++) {
                float w = dequant_one_w8(qweight, qzeros, scales, g_idx, N, group_size, zeros_plus, k, n);
                acc += (double)oracle_half_to_float(x[(size_t)m * K + k]) * (double)w;
            }
            y_out[(size_t)m * N + n] = acc;
        }
    }
}

void oracle_gemm_f64_w8_at(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                           const uint16_t *scales, const int32_t *g_idx,
                           int M, int N, int K, int group_size, int zeros_plus,
                           const int32_t *rows, const int32_t *cols, int count, double *y_out)
{
    (void)M;
    #pragma omp parallel for schedule(static)
    for (int i = 0; i < count; i++) {
        int m = rows[i], n = cols[i];
        double acc = 0.0;
        for (int k = 0; k < K; k++) {
            float w = dequant_one_w8(qweight, qzeros, scales, g_idx, N, group_size, zeros_plus, k, n);
            acc += (double)oracle_half_to_float(x[(size_t)m * K + k]) * (double)w;
        }
        y_out[i] = acc;
    }
}

/* ---- format variant: 2- and 3-bit weights ------------------------------------------------------
 * The paper treats 4-bit GPTQ only (Section 1); the checkpoint family also has 2- and 3-bit layers.
 * Reading (pinned by hand-packed words in the tests): the values of a column (weights, along K) or
 * of a group's row (zero points, along N) form one bit stream, value i in bits [bits*i, bits*i+bits)
 * of the little-endian concatenation of that column's / row's 32-bit words - for 2 bits, 16 values
 * per word; for 3 bits, 32 values per three words, values 10 and 21 straddling a word boundary.
 *   qweight int32[K*bits/32][N], qzeros int32[G][N*bits/32], scales fp16[G][N]
 *   w32[k][n] = float(q - z) * float(s), z = stored + zeros_plus;  y as in the 4-bit case. */
static inline unsigned stream_field(const int32_t *words, size_t stride, int index, int bits)
{
    int bit = bits * index, w = bit >> 5, sh = bit & 31;
    uint64_t two = (uint32_t)words[(size_t)w * stride];
    if (sh + bits > 32) two |= (uint64_t)(uint32_t)words[(size_t)(w + 1) * stride] << 32;
    return (unsigned)((two >> sh) & ((1u << bits) - 1u));
}

void oracle_unpack_qn(const int32_t *qweight, int K, int N, int bits, uint8_t *q_out)
{
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            q_out[(size_t)k * N + n] = (uint8_t)stream_field(qweight + n, (size_t)N, k, bits);
}

void oracle_unpack_zn(const int32_t *qzeros, int G, int N, int bits, uint8_t *z_out)
{
    for (int g = 0; g < G; g++)
        for (int n = 0; n < N; n++)
            z_out[(size_t)g * N + n] = (uint8_t)stream_field(qzeros + (size_t)g * (N * bits / 32), 1, n, bits);
}

static inline float dequant_one_wn(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                                   const int32_t *g_idx, int N, int group_size, int bits, int zeros_plus, int k, int n)
{
    int g = group_of(g_idx, k, group_size);
    int q = (int)stream_field(qweight + n, (size_t)N, k, bits);
    int z = (int)stream_field(qzeros + (size_t)g * (N * bits / 32), 1, n, bits) + zeros_plus;
    float s = oracle_half_to_float(scales[(size_t)g * N + n]);
    return (float)(q - z) * s;
}

void oracle_dequant_f32_wn(const int32_t *qweight, const int32_t *qzeros, const uint16_t *scales,
                           const int32_t *g_idx, int K, int N, int group_size, int bits, int zeros_plus, float *w_out)
{
    #pragma omp parallel for schedule(static)
    for (int k = 0; k < K; k++)
        for (int n = 0; n < N; n++)
            w_out[(size_t)k * N + n] = dequant_one_wn(qweight, qzeros, scales, g_idx, N, group_size, bits, zeros_plus, k, n);
}

void oracle_gemm_f64_wn(const uint16_t *x, const int32_t *qweight, const int32_t *qzeros,
                        const uint16_t *scales, const int32_t *g_idx,
                        int M, int N, int K, int group_size, int bits, int zeros_plus, double *y_out)
{
    #pragma omp parallel for schedule(static)
    for (int n = 0; n < N; n++) {
        for (int m = 0; m < M; m++) {
            double acc = 0.0;
            for (int k = 0; k < K; k++) {
                float w = dequant_one_wn(qweight, qzeros, scales, g_idx, N, group_size, bits, zeros_plus, k, n);
                acc += (double)oracle_half_to_float(x[(size_t)m * K + k]) * (double)w;
            }
            y_out[(size_t)m * N + n] = acc;
        }
    }
}
