// 2- and 3-bit GPTQ weights: expanded to 4-bit nibbles by the one-time repack.
//
// Canonical layout: the values of a column (weights) or of a group's row (zero points) form one bit stream, value i in
// bits [bits * i, bits * i + bits) of the little-endian concatenation of that column's / row's 32-bit words; qweight
// int32[K * bits / 32, N], qzeros int32[G, N * bits / 32].  The repack widens every field to a nibble (zero points with
// the older minus-one convention get their one added here, they stay below 16) and tiles the resulting 4-bit layer as
// usual; it is then multiplied by gptq_gemm like any other.  The tiled layer takes the bytes of a 4-bit layer, i.e. the
// matmul streams 2 x (2-bit) or 1.33 x (3-bit) the bytes the checkpoint holds: these widths are supported, not sped up.
#pragma once
#include "gptq_common.cuh"
#include "gptq_layout.cuh"

namespace gptq {

__device__ __forceinline__ uint32_t stream_field(const int32_t *words, size_t stride, int index, int bits)
{
    const int bit = bits * index, w = bit >> 5, sh = bit & 31;
    unsigned long long two = (uint32_t)words[(size_t)w * stride];
    if (sh + bits > 32) two |= (unsigned long long)(uint32_t)words[(size_t)(w + 1) * stride] << 32;
    return (uint32_t)((two >> sh) & ((1u << bits) - 1u));
}

// One thread per (8 rows, column): nibble i of the 4-bit word = row 8 r + i.
__global__ void wn_expand_weights_kernel(const int32_t *__restrict__ qweight, int32_t *__restrict__ q4, int N, int K, int bits)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)(K / 8) * N) return;
    const int r = (int)(idx / N), n = (int)(idx % N);
    uint32_t out = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) out |= stream_field(qweight + n, (size_t)N, 8 * r + i, bits) << (4 * i);
    q4[idx] = (int32_t)out;
}

// One thread per (group, 8 columns): nibble j of the 4-bit word = column 8 c + j.
__global__ void wn_expand_zeros_kernel(const int32_t *__restrict__ qzeros, int32_t *__restrict__ z4, int N, int G, int bits, int z_plus)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)G * (N / 8)) return;
    const int g = (int)(idx / (N / 8)), c = (int)(idx % (N / 8));
    const int32_t *row = qzeros + (size_t)g * (N * bits / 32);
    uint32_t out = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) out |= (stream_field(row, 1, 8 * c + j, bits) + (uint32_t)z_plus) << (4 * j);
    z4[idx] = (int32_t)out;
}

// Canonical layout, one thread per (k, n): float(q - z) * float(s), exact.
__global__ void wn_dequant_canonical_kernel(const int32_t *__restrict__ qweight, const int32_t *__restrict__ qzeros,
                                            const __half *__restrict__ scales, const int32_t *__restrict__ g_idx,
                                            float *__restrict__ w_out, int N, int K, int group_size, int bits, int z_plus)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)K * N) return;
    const int k = (int)(idx / N), n = (int)(idx % N);
    const int g = g_idx ? g_idx[k] : k / group_size;
    const int q = (int)stream_field(qweight + n, (size_t)N, k, bits);
    const int z = (int)stream_field(qzeros + (size_t)g * (N * bits / 32), 1, n, bits) + z_plus;
    w_out[idx] = __fmul_rn((float)(q - z), __half2float(scales[(size_t)g * N + n]));
}

int launch_wn_dequant_f32(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                          float *w_out, int N, int K, int group_size, int bits, int z_plus, cudaStream_t s)
{
    const int T = 256;
    wn_dequant_canonical_kernel<<<(unsigned)(((size_t)K * N + T - 1) / T), T, 0, s>>>(
        (const int32_t *)qweight, (const int32_t *)qzeros, (const __half *)scales, g_idx, w_out, N, K, group_size, bits, z_plus);
    return record_cuda_error(cudaGetLastError());
}

// scratch: the expanded canonical 4-bit weights (K * N / 2 bytes, rounded up to 256) followed by the expanded zero points
inline size_t wn_scratch_bytes(int N, int K, int group_size)
{
    const size_t q4 = (((size_t)K * N / 2) + 255) & ~(size_t)255;
    return q4 + ((((size_t)(K / group_size) * (N / 8) * 4) + 255) & ~(size_t)255);
}

int launch_wn_repack(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                     void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, void *scratch, int N,
                     int K, int group_size, int bits, int act_order, int z_plus, cudaStream_t s)
{
    int32_t *q4 = (int32_t *)scratch;
    int32_t *z4 = (int32_t *)((uint8_t *)scratch + ((((size_t)K * N / 2) + 255) & ~(size_t)255));
    const int T = 256, G = K / group_size;
    const size_t words = (size_t)(K / 8) * N, zwords = (size_t)G * (N / 8);
    wn_expand_weights_kernel<<<(unsigned)((words + T - 1) / T), T, 0, s>>>(qweight, q4, N, K, bits);
    wn_expand_zeros_kernel<<<(unsigned)((zwords + T - 1) / T), T, 0, s>>>(qzeros, z4, N, G, bits, z_plus);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error(e);
    // the zero points now hold their final values: the tiled layer uses the stored-as-is convention
    return launch_repack(q4, z4, scales, g_idx, qweight_out, qzeros_out, scales_out, perm_out, N, K, group_size, act_order, 0, s);
}

}  // namespace gptq
