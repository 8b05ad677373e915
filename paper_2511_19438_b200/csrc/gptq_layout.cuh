// Format kernels: nibble unpack, fp32 dequantisation (canonical and tiled layouts), the
// one-time repack into the tiled layout, and the activation gather used with act-order.
// All of them are plain element-per-thread kernels; none is on the per-token path except
// gather_x (act-order only).
#pragma once
#include "gptq_common.cuh"

namespace gptq {

// ------------------------------------------------------------------------------ unpack
__global__ void unpack_q_kernel(const int32_t *__restrict__ qweight, uint8_t *__restrict__ q_out, int N, int K)
{
    // one thread per packed word: writes its 8 rows of one column
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t words = (size_t)(K / 8) * N;
    if (idx >= words) return;
    int r = (int)(idx / N), n = (int)(idx % N);
    uint32_t w = (uint32_t)qweight[idx];
#pragma unroll
    for (int i = 0; i < 8; ++i) q_out[(size_t)(8 * r + i) * N + n] = (uint8_t)((w >> (4 * i)) & 15u);
}

__global__ void unpack_z_kernel(const int32_t *__restrict__ qzeros, uint8_t *__restrict__ z_out, int N, int G)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t words = (size_t)G * (N / 8);
    if (idx >= words) return;
    uint32_t w = (uint32_t)qzeros[idx];
#pragma unroll
    for (int j = 0; j < 8; ++j) z_out[idx * 8 + j] = (uint8_t)((w >> (4 * j)) & 15u);
}

int launch_unpack_u8(const int32_t *qweight, const int32_t *qzeros, uint8_t *q_out, uint8_t *z_out, int N, int K,
                     int G, cudaStream_t s)
{
    const int T = 256;
    if (q_out) {
        size_t words = (size_t)(K / 8) * N;
        unpack_q_kernel<<<(unsigned)((words + T - 1) / T), T, 0, s>>>(qweight, q_out, N, K);
    }
    if (z_out) {
        size_t words = (size_t)G * (N / 8);
        unpack_z_kernel<<<(unsigned)((words + T - 1) / T), T, 0, s>>>(qzeros, z_out, N, G);
    }
    return record_cuda_error(cudaGetLastError());
}

// ------------------------------------------------------------------------------ dequant fp32
// One thread per (k, n).  float(q - z) * float(s): a single fp32 multiply whose result is exact.
// A scale is 16 bits of fp16 or, with the bfloat16 format flag, of bfloat16 (the upper half of an fp32).
__device__ __forceinline__ float scale_to_float(const __half *p, bool bf16)
{
    return bf16 ? __uint_as_float((uint32_t)__half_as_ushort(*p) << 16) : __half2float(*p);
}
__global__ void dequant_canonical_kernel(const int32_t *__restrict__ qweight, const int32_t *__restrict__ qzeros,
                                         const __half *__restrict__ scales, const int32_t *__restrict__ g_idx,
                                         float *__restrict__ w_out, int N, int K, int group_size, int z_add, int bf16)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)K * N) return;
    int k = (int)(idx / N), n = (int)(idx % N);
    int g = g_idx ? g_idx[k] : k / group_size;
    int q = (int)(((uint32_t)qweight[(size_t)(k >> 3) * N + n] >> (4 * (k & 7))) & 15u);
    int z = (int)(((uint32_t)qzeros[(size_t)g * (N / 8) + (n >> 3)] >> (4 * (n & 7))) & 15u) + z_add;
    w_out[idx] = __fmul_rn((float)(q - z), scale_to_float(scales + (size_t)g * N + n, bf16 != 0));
}

// Tiled layout: thread per (sorted row i, column n); the row goes back to its original index.
__global__ void dequant_tiled_kernel(const uint8_t *__restrict__ qweight, const uint8_t *__restrict__ qzeros,
                                     const __half *__restrict__ scales, const int32_t *__restrict__ perm,
                                     float *__restrict__ w_out, int N, int K, int group_size)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)K * N) return;
    int i = (int)(idx / N), n = (int)(idx % N);
    int groups = K / group_size, grp = i / group_size;
    int slot, hi;
    // the trailer says whether the stored zero points are one too small and whether the column halves are interleaved
    const TiledTrailer *tr = reinterpret_cast<const TiledTrailer *>(qzeros + tiled_zero_bytes(N, K, group_size));
    const int nt = (tr->flags & kFormatGateUp) ? gate_up_tiled_column(n, N) : n;
    size_t off = repacked_word_offset(i, nt, K / kGroup, &slot);
    uint32_t word = *reinterpret_cast<const uint32_t *>(qweight + off);
    int q = (int)((word >> (4 * slot)) & 15u);
    uint8_t zb = qzeros[repacked_zero_byte(grp, nt, groups, &hi)];
    int z = (hi ? (zb >> 4) : (zb & 15)) + (int)(tr->flags & kFormatZerosMinusOne);
    float s = scale_to_float(scales + repacked_scale_index(grp, nt, groups), (tr->flags & kFormatBf16) != 0);
    int k = perm ? perm[i] : i;
    w_out[(size_t)k * N + n] = __fmul_rn((float)(q - z), s);
}

int launch_dequant_f32(const void *qweight, const void *qzeros, const void *scales, const int32_t *g_idx,
                       float *w_out, int N, int K, int group_size, int act_order, int repacked, int format,
                       cudaStream_t s)
{
    const int T = 256;
    size_t total = (size_t)K * N;
    unsigned blocks = (unsigned)((total + T - 1) / T);
    if (repacked)
        dequant_tiled_kernel<<<blocks, T, 0, s>>>((const uint8_t *)qweight, (const uint8_t *)qzeros,
                                                  (const __half *)scales, act_order ? g_idx : nullptr, w_out, N, K,
                                                  group_size);
    else
        dequant_canonical_kernel<<<blocks, T, 0, s>>>((const int32_t *)qweight, (const int32_t *)qzeros,
                                                      (const __half *)scales, act_order ? g_idx : nullptr, w_out,
                                                      N, K, group_size, (format & (int)kFormatZerosMinusOne) ? 1 : 0,
                                                      (format & (int)kFormatBf16) ? 1 : 0);
    return record_cuda_error(cudaGetLastError());
}

// ------------------------------------------------------------------------------ act-order sort
// perm = stable argsort(g_idx).  Thread k counts the keys that sort before its own:
// rank(k) = #{k' : g[k'] < g[k]} + #{k' < k : g[k'] == g[k]}.  O(K^2) compares, one-time, K <= ~16k.
// Also checks 0 <= g[k] < G and that every group has exactly group_size rows.
__global__ void argsort_gidx_kernel(const int32_t *__restrict__ g_idx, int32_t *__restrict__ perm, int K, int G,
                                    int group_size)
{
    extern __shared__ int32_t tile[];
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    int mine = (k < K) ? g_idx[k] : 0;
    bool bad = (k < K) && (mine < 0 || mine >= G);
    int below = 0, same_before = 0, same_total = 0;
    for (int base = 0; base < K; base += blockDim.x) {
        int kk = base + threadIdx.x;
        tile[threadIdx.x] = (kk < K) ? g_idx[kk] : -1;
        __syncthreads();
        int lim = min((int)blockDim.x, K - base);
        for (int j = 0; j < lim; ++j) {
            int other = tile[j];
            below += (other < mine);
            same_total += (other == mine);
            same_before += (other == mine) && (base + j < k);
        }
        __syncthreads();
    }
    if (k >= K) return;
    if (bad) {
        atomicMax(&g_gidx_status, (int)kGidxOutOfRange);
        return;
    }
    if (same_total != group_size) atomicMax(&g_gidx_status, (int)kGidxUnequalGroups);
    int rank = below + same_before;
    if (rank >= 0 && rank < K) perm[rank] = k;
}

// ------------------------------------------------------------------------------ repack
// One thread per output word of the tiled layout.
__global__ void repack_weights_kernel(const int32_t *__restrict__ qweight, const int32_t *__restrict__ perm,
                                      uint32_t *__restrict__ out, int N, int K, int gate_up)
{
    size_t o = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t words = (size_t)(K / 8) * N;
    if (o >= words) return;
    int G = K / kGroup;
    // decode the output word index: [item][blk(2)][unit(8)][lane(32)][c(4)]
    int c = (int)(o & 3), lane = (int)((o >> 2) & 31), u = (int)((o >> 7) & 7), blk = (int)((o >> 10) & 1);
    size_t item = o >> 11;
    int p = (int)(item / G), grp = (int)(item % G);
    int g = lane >> 2, t4 = lane & 3, j = c & 1, h = c >> 1;
    int n = p * kPanel + 16 * u + g + 8 * h;
    if (gate_up) n = gate_up_source_column(n, N);
    int i0 = grp * kGroup + blk * 64 + j * 32 + t4 * 8;
    uint32_t word = 0;
    if (perm == nullptr) {
        uint32_t src = (uint32_t)qweight[(size_t)(i0 >> 3) * N + n];
#pragma unroll
        for (int e = 0; e < 8; ++e) word |= ((src >> (4 * e)) & 15u) << (4 * nibble_slot(e));
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            int k = perm[i0 + e];
            uint32_t q = ((uint32_t)qweight[(size_t)(k >> 3) * N + n] >> (4 * (k & 7))) & 15u;
            word |= q << (4 * nibble_slot(e));
        }
    }
    out[o] = word;
}

// One thread per (group, column): scale to its tiled position; thread with h == 0 also writes the
// zero byte of its column pair.  Thread 0 writes the trailer behind the zero points.
__global__ void repack_meta_kernel(const int32_t *__restrict__ qzeros, const __half *__restrict__ scales,
                                   uint8_t *__restrict__ z_out, __half *__restrict__ s_out, int N, int G,
                                   int group_size, int repeat, uint32_t flags)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx == 0) {
        TiledTrailer tr{kTrailerMagic, flags, (uint32_t)group_size, 0u};
        *reinterpret_cast<TiledTrailer *>(z_out + (size_t)G * (N / 2)) = tr;
    }
    if (idx >= (size_t)G * N) return;
    // one thread per (tiled group, tiled column nt); its values come from checkpoint column n of checkpoint group
    // grp / repeat (repeat > 1: the checkpoint's groups span `repeat` tiled groups of 128 rows)
    int grp = (int)(idx / N), nt = (int)(idx % N);
    const int src = grp / repeat;
    const bool gate_up = (flags & kFormatGateUp) != 0;
    int n = gate_up ? gate_up_source_column(nt, N) : nt;
    s_out[repacked_scale_index(grp, nt, G)] = scales[(size_t)src * N + n];
    if (((nt % 16) >> 3) == 0) {
        const int32_t *zrow = qzeros + (size_t)src * (N / 8);
        uint32_t za = ((uint32_t)zrow[n >> 3] >> (4 * (n & 7))) & 15u;
        int nb = n + 8;     // the partner column: eight further in both numberings (halves are multiples of 64)
        uint32_t zb = ((uint32_t)zrow[nb >> 3] >> (4 * (nb & 7))) & 15u;
        int hi;
        z_out[repacked_zero_byte(grp, nt, G, &hi)] = (uint8_t)(za | (zb << 4));
    }
}

// Ends the repack with an ordinary (fully stream-ordered) kernel boundary, so that a matmul
// launched right after it with programmatic dependent launch cannot fetch weights early.
__global__ void repack_fence_kernel() {}

int launch_repack(const int32_t *qweight, const int32_t *qzeros, const void *scales, const int32_t *g_idx,
                  void *qweight_out, void *qzeros_out, void *scales_out, int32_t *perm_out, int N, int K,
                  int source_group_size, int act_order, int format, cudaStream_t s)
{
    // source_group_size: rows per group in the checkpoint; group_size: rows per group of the tiled layer (the same, or
    // 128 when the checkpoint's groups are a multiple of 128 rows: the tiled groups then repeat their group's values)
    const int group_size = source_group_size > kGroup ? kGroup : source_group_size;
    const int T = 256;
    int G = K / group_size;
    if (act_order) {
        int blocks = (K + T - 1) / T;
        argsort_gidx_kernel<<<blocks, T, T * sizeof(int32_t), s>>>(g_idx, perm_out, K, K / source_group_size, source_group_size);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return record_cuda_error(e);
        // one-time call: read the validation result before tiling with a possibly invalid perm
        int status = 0;
        e = cudaMemcpyFromSymbolAsync(&status, g_gidx_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (status != kGidxOk) {
            int zero = 0;
            e = cudaMemcpyToSymbolAsync(g_gidx_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
            if (e == cudaSuccess) e = cudaStreamSynchronize(s);
            if (e != cudaSuccess) return record_cuda_error(e);
            return GPTQ_ERR_GIDX;   // out of range, or groups of unequal size
        }
    }
    size_t words = (size_t)(K / 8) * N;
    repack_weights_kernel<<<(unsigned)((words + T - 1) / T), T, 0, s>>>(qweight, act_order ? perm_out : nullptr,
                                                                        (uint32_t *)qweight_out, N, K,
                                                                        (format & (int)kFormatGateUp) ? 1 : 0);
    size_t meta = (size_t)G * N;
    repack_meta_kernel<<<(unsigned)((meta + T - 1) / T), T, 0, s>>>(qzeros, (const __half *)scales,
                                                                    (uint8_t *)qzeros_out, (__half *)scales_out, N, G,
                                                                    group_size, source_group_size / group_size, (uint32_t)format);
    repack_fence_kernel<<<1, 32, 0, s>>>();
    return record_cuda_error(cudaGetLastError());
}

// ------------------------------------------------------------------------------ gather x
// x_out[m][i] = x[m][perm[i]]: puts the activations in the sorted row order of the tiled weights.
__global__ void gather_x_kernel(const __half *__restrict__ x, const int32_t *__restrict__ perm,
                                __half *__restrict__ x_out, int M, int K)
{
    pdl_launch_dependents();   // the matmul that follows may start fetching weights now
    pdl_wait();                // x may come from the kernel just before this one
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    int src = perm[i];
    for (int m = blockIdx.y; m < M; m += gridDim.y) x_out[(size_t)m * K + i] = x[(size_t)m * K + src];
}

// The same for many token rows: a block stages kGatherRows whole rows of x in shared memory with coalesced 16-byte
// loads, then every thread picks eight permuted elements per row from there and writes them with one 16-byte store.
// (The element-per-thread kernel above reads 2 bytes per 32-byte sector; with thousands of rows that costs several
// times the copy itself.)
constexpr int kGatherRows = 4;
__global__ void __launch_bounds__(256)
gather_x_rows_kernel(const __half *__restrict__ x, const int32_t *__restrict__ perm, __half *__restrict__ x_out, int M, int K)
{
    extern __shared__ uint4 gather_rows[];     // kGatherRows x K halves
    pdl_launch_dependents();
    pdl_wait();
    const int m0 = blockIdx.x * kGatherRows;
    const int nrows = (M - m0) < kGatherRows ? (M - m0) : kGatherRows;
    const int chunks = K / 8;                  // 16-byte chunks per row
    const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)m0 * K);   // the rows are adjacent in memory
    for (int i = threadIdx.x; i < nrows * chunks; i += blockDim.x) gather_rows[i] = src[i];
    __syncthreads();
    const __half *rows = reinterpret_cast<const __half *>(gather_rows);
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        const int4 pa = reinterpret_cast<const int4 *>(perm)[2 * c], pb = reinterpret_cast<const int4 *>(perm)[2 * c + 1];
        const int idx[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
        for (int r = 0; r < nrows; ++r) {
            __align__(16) __half v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = rows[(size_t)r * K + idx[e]];
            *reinterpret_cast<uint4 *>(x_out + (size_t)(m0 + r) * K + 8 * c) = *reinterpret_cast<const uint4 *>(v);
        }
    }
}

int launch_gather_x(const __half *x, const int32_t *perm, __half *x_out, int M, int K, cudaStream_t s)
{
    const size_t rows_smem = (size_t)kGatherRows * K * sizeof(__half);
    // measured on the 7B shapes: pays from about a thousand rows on (M = 4096: 17-57 us instead of 48-250), from 512
    // rows on the long-K layers; below that its few blocks leave most SMs idle and the element-per-thread kernel wins
    if ((M >= 1024 || (M >= 512 && K >= 8192)) && K % 8 == 0 && rows_smem <= 200 * 1024) {
        static int configured_smem[64] = {};
        const int cfg_st = ensure_dynamic_smem((const void *)gather_x_rows_kernel, configured_smem, (int)rows_smem);
        if (cfg_st) return cfg_st;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)((M + kGatherRows - 1) / kGatherRows));
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = rows_smem;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return record_cuda_error(cudaLaunchKernelEx(&cfg, gather_x_rows_kernel, x, perm, x_out, M, K));
    }
    const int T = 256;
    // launched as a programmatic dependent of the kernel before it: its CTAs become resident while that kernel still
    // runs, and griddepcontrol.wait holds the copy back until that kernel (which may write x, and may still be reading
    // the previous contents of x_out) has completed
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((K + T - 1) / T, (unsigned)min(M, 64));
    cfg.blockDim = dim3(T);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return record_cuda_error(cudaLaunchKernelEx(&cfg, gather_x_kernel, x, perm, x_out, M, K));
}

// inverse[perm[i]] = i: where an element that sits at original position c goes in the sorted order
__global__ void invert_perm_kernel(const int32_t *__restrict__ perm, int32_t *__restrict__ inverse, int K)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const int c = perm[i];
    if (c >= 0 && c < K) inverse[c] = i;
}

int launch_invert_perm(const int32_t *perm, int32_t *inverse, int K, cudaStream_t s)
{
    invert_perm_kernel<<<(K + 255) / 256, 256, 0, s>>>(perm, inverse, K);
    return record_cuda_error(cudaGetLastError());
}

}  // namespace gptq
