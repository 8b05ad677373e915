// 8-bit GPTQ weights through the 4-bit kernels.
//
// An 8-bit weight is two nibbles, q = 16 hi + lo, and so is its zero point, z = 16 zh + zl:
//     (q - z) s = (hi - zh) (16 s) + (lo - zl) s.
// A layer [K, N] of 8-bit weights is therefore the sum of two 4-bit layers over the same activations: a HIGH plane with
// weights hi, zero points zh and scales 16 s (exact: a power of two) and a LOW plane with lo, zl and s.  The repack
// stacks the planes along K - a 4-bit layer of 2 K rows, rows 0..K-1 the high plane - and tiles that layer as usual;
// the matmul gathers x into [x | x] in the stacked (and, with act-order, sorted) row order and runs the 4-bit kernels
// on 2 K rows.  The bytes streamed are those of the 8-bit layer (one byte per weight; scales and zero points twice),
// and so is the arithmetic: the integers are exact and each plane's scale joins in fp32 (M <= 16), respectively each
// plane's scaled weight is rounded to fp16 once (tcgen05 kernel).
//
// Canonical 8-bit layout (the 4-bit conventions at twice the field width): qweight int32[K/4, N], byte i of a word =
// row 4 r + i; qzeros int32[G, N/4], byte j of a word = column 4 c + j; scales fp16[G, N]; g_idx int32[K].
#pragma once
#include "gptq_common.cuh"
#include "gptq_layout.cuh"

namespace gptq {

__device__ int g_w8_status = 0;   // 1: a zero point of 256 (stored 255 under the minus-one convention) was met

// One thread per (8 rows, column): two 8-bit words in, one word of each plane out (nibble i of a 4-bit word = row 8 r + i).
__global__ void w8_split_weights_kernel(const int32_t *__restrict__ qweight8, int32_t *__restrict__ q4, int N, int K)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)(K / 8) * N) return;
    const size_t r = idx / N, n = idx % N;
    const uint32_t w0 = (uint32_t)qweight8[(2 * r) * N + n], w1 = (uint32_t)qweight8[(2 * r + 1) * N + n];
    uint32_t hi = 0, lo = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t b0 = (w0 >> (8 * i)) & 255u, b1 = (w1 >> (8 * i)) & 255u;
        lo |= (b0 & 15u) << (4 * i) | (b1 & 15u) << (4 * (i + 4));
        hi |= (b0 >> 4) << (4 * i) | (b1 >> 4) << (4 * (i + 4));
    }
    q4[r * N + n] = (int32_t)hi;
    q4[((size_t)(K / 8) + r) * N + n] = (int32_t)lo;
}

// Zero points, scales and group indices of the stacked layer: groups 0..G-1 belong to the high plane, G..2G-1 to the low.
__global__ void w8_split_meta_kernel(const int32_t *__restrict__ qzeros8, const __half *__restrict__ scales,
                                     const int32_t *__restrict__ g_idx, int32_t *__restrict__ z4,
                                     __half *__restrict__ s4, int32_t *__restrict__ g4, int N, int K, int G,
                                     int group_size, int z_plus)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < (size_t)G * (N / 8)) {           // eight columns: two 8-bit words in, one word per plane out
        const size_t g = idx / (N / 8), c = idx % (N / 8);
        const uint32_t a = (uint32_t)qzeros8[g * (N / 4) + 2 * c], b = (uint32_t)qzeros8[g * (N / 4) + 2 * c + 1];
        uint32_t zh = 0, zl = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t z = (((j < 4 ? a : b) >> (8 * (j & 3))) & 255u) + (uint32_t)z_plus;
            if (z > 255u) {                      // 256 has no nibble pair: refused by the caller
                atomicMax(&g_w8_status, 1);
                z = 255u;
            }
            zh |= (z >> 4) << (4 * j);
            zl |= (z & 15u) << (4 * j);
        }
        z4[g * (N / 8) + c] = (int32_t)zh;
        z4[((size_t)G + g) * (N / 8) + c] = (int32_t)zl;
    }
    if (idx < (size_t)G * N) {
        const __half sc = scales[idx];
        s4[idx] = __float2half_rn(16.f * __half2float(sc));    // exact unless it overflows (scale >= 4096)
        s4[(size_t)G * N + idx] = sc;
    }
    if (idx < (size_t)K) {
        const int g = g_idx ? g_idx[idx] : (int)(idx / group_size);
        // an index outside 0..G-1 stays outside 0..2G-1 in both planes, so the sort's range check still sees it
        const bool bad = g < 0 || g >= G;
        g4[idx] = bad ? -1 : g;
        g4[(size_t)K + idx] = bad ? -1 : G + g;
    }
}

// perm of the stacked layer -> index into x: row K + k of the low plane multiplies x[k] as well
__global__ void w8_fold_perm_kernel(int32_t *__restrict__ perm, int K)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < 2 * K && perm[i] >= K) perm[i] -= K;
}

// x_out[m][i] = x[m][perm[i]] for the 2 K rows of the stacked layer (x has K columns, x_out 2 K).
__global__ void w8_gather_x_kernel(const __half *__restrict__ x, const int32_t *__restrict__ perm,
                                   __half *__restrict__ x_out, int M, int K)
{
    pdl_launch_dependents();   // the matmul that follows may start fetching weights now
    pdl_wait();                // x may come from the kernel just before this one
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 2 * K) return;
    const int src = perm[i];
    for (int m = blockIdx.y; m < M; m += gridDim.y) x_out[(size_t)m * 2 * K + i] = x[(size_t)m * K + src];
}

int launch_w8_gather_x(const __half *x, const int32_t *perm, __half *x_out, int M, int K, cudaStream_t s)
{
    const int T = 256;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((2 * K + T - 1) / T, (unsigned)min(M, 64));
    cfg.blockDim = dim3(T);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return record_cuda_error(cudaLaunchKernelEx(&cfg, w8_gather_x_kernel, x, perm, x_out, M, K));
}

// ------------------------------------------------------------------------------ dequant fp32 (bit-exact checks)
// Canonical layout: one thread per (k, n); float(q - z) * float(s) is exact (9 bits times 11).
__global__ void w8_dequant_canonical_kernel(const int32_t *__restrict__ qweight, const int32_t *__restrict__ qzeros,
                                            const __half *__restrict__ scales, const int32_t *__restrict__ g_idx,
                                            float *__restrict__ w_out, int N, int K, int group_size, int z_plus)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)K * N) return;
    const int k = (int)(idx / N), n = (int)(idx % N);
    const int g = g_idx ? g_idx[k] : k / group_size;
    const int q = (int)(((uint32_t)qweight[(size_t)(k >> 2) * N + n] >> (8 * (k & 3))) & 255u);
    const int z = (int)(((uint32_t)qzeros[(size_t)g * (N / 4) + (n >> 2)] >> (8 * (n & 3))) & 255u) + z_plus;
    w_out[idx] = __fmul_rn((float)(q - z), __half2float(scales[(size_t)g * N + n]));
}

// Tiled (stacked) layout: thread per (sorted row i < K, column n).  Row i of the high plane and row K + i of the low
// plane belong to the same checkpoint row perm[i]; the integer 16 (hi - zh) + (lo - zl) is q - z, and the low plane's
// scale is the checkpoint's.
__global__ void w8_dequant_tiled_kernel(const uint8_t *__restrict__ qweight, const uint8_t *__restrict__ qzeros,
                                        const __half *__restrict__ scales, const int32_t *__restrict__ perm,
                                        float *__restrict__ w_out, int N, int K, int group_size)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)K * N) return;
    const int i = (int)(idx / N), n = (int)(idx % N);
    const int K2 = 2 * K, groups = K2 / group_size;
    int nib[2], zp[2];
#pragma unroll
    for (int plane = 0; plane < 2; ++plane) {
        const int row = plane * K + i, grp = row / group_size;
        int slot, hi;
        const size_t off = repacked_word_offset(row, n, K2 / kGroup, &slot);
        nib[plane] = (int)((*reinterpret_cast<const uint32_t *>(qweight + off) >> (4 * slot)) & 15u);
        const uint8_t zb = qzeros[repacked_zero_byte(grp, n, groups, &hi)];
        zp[plane] = hi ? (zb >> 4) : (zb & 15);
    }
    const float s = __half2float(scales[repacked_scale_index((K + i) / group_size, n, groups)]);
    w_out[(size_t)perm[i] * N + n] = __fmul_rn((float)(16 * (nib[0] - zp[0]) + (nib[1] - zp[1])), s);
}

int launch_w8_dequant_f32(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                          float *w_out, int N, int K, int group_size, int repacked, int z_plus, cudaStream_t s)
{
    const int T = 256;
    const unsigned blocks = (unsigned)(((size_t)K * N + T - 1) / T);
    if (repacked)
        w8_dequant_tiled_kernel<<<blocks, T, 0, s>>>((const uint8_t *)qweight, (const uint8_t *)qzeros,
                                                     (const __half *)scales, g_idx, w_out, N, K, group_size);
    else
        w8_dequant_canonical_kernel<<<blocks, T, 0, s>>>((const int32_t *)qweight, (const int32_t *)qzeros,
                                                         (const __half *)scales, g_idx, w_out, N, K, group_size, z_plus);
    return record_cuda_error(cudaGetLastError());
}

// ------------------------------------------------------------------------------ repack
// Byte offsets of the four parts of the scratch buffer (stacked canonical 4-bit layer), each 256-byte aligned.
struct W8Scratch {
    size_t q4, z4, s4, g4, total;
};
inline W8Scratch w8_scratch_layout(int N, int K, int group_size)
{
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t G = (size_t)(K / group_size);
    W8Scratch w;
    w.q4 = 0;
    w.z4 = up((size_t)K * N);                       // 2 K / 8 words of 4 bytes per column
    w.s4 = w.z4 + up(2 * G * (N / 8) * 4);
    w.g4 = w.s4 + up(2 * G * N * 2);
    w.total = w.g4 + up((size_t)2 * K * 4);
    return w;
}

// group_size is the checkpoint's; returns GPTQ_ERR_UNSUPPORTED for a zero point of 256, GPTQ_ERR_GIDX as launch_repack
int launch_w8_repack(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                     void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, void *scratch, int N,
                     int K, int group_size, int z_plus, cudaStream_t s)
{
    const W8Scratch lay = w8_scratch_layout(N, K, group_size);
    uint8_t *base = (uint8_t *)scratch;
    int32_t *q4 = (int32_t *)(base + lay.q4), *z4 = (int32_t *)(base + lay.z4), *g4 = (int32_t *)(base + lay.g4);
    __half *s4 = (__half *)(base + lay.s4);
    const int T = 256, G = K / group_size;
    const size_t words = (size_t)(K / 8) * N;
    w8_split_weights_kernel<<<(unsigned)((words + T - 1) / T), T, 0, s>>>(qweight, q4, N, K);
    size_t meta = (size_t)G * N;
    if (meta < (size_t)K) meta = (size_t)K;
    w8_split_meta_kernel<<<(unsigned)((meta + T - 1) / T), T, 0, s>>>(qzeros, (const __half *)scales, g_idx, z4, s4, g4, N,
                                                                      K, G, group_size, z_plus);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error(e);
    int status = 0;
    e = cudaMemcpyFromSymbolAsync(&status, g_w8_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return record_cuda_error(e);
    if (status != 0) {
        const int zero = 0;
        e = cudaMemcpyToSymbolAsync(g_w8_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return record_cuda_error(e);
        return GPTQ_ERR_UNSUPPORTED;
    }
    // the stacked layer always goes through the sort: without act-order its group indices are already ascending and
    // the permutation comes out as the identity
    const int st = launch_repack(q4, z4, s4, g4, qweight_out, qzeros_out, scales_out, perm_out, N, 2 * K, group_size, 1, 0, s);
    if (st) return st;
    w8_fold_perm_kernel<<<(2 * K + T - 1) / T, T, 0, s>>>(perm_out, K);
    repack_fence_kernel<<<1, 32, 0, s>>>();
    return record_cuda_error(cudaGetLastError());
}

}  // namespace gptq
