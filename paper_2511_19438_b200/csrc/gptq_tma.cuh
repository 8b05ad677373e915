// Tensor-map (TMA) plumbing: host-side encoding through the driver entry point (looked up at run
// time, so the library does not link libcuda) and the device-side tiled load.
#pragma once
#include <cuda.h>

#include "gptq_common.cuh"

namespace gptq {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline int get_encode_tiled(EncodeTiledFn *out)
{
    static EncodeTiledFn cached = nullptr;
    if (cached == nullptr) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (q != cudaDriverEntryPointSuccess || fn == nullptr) return GPTQ_ERR_CUDA;
        cached = (EncodeTiledFn)fn;
    }
    *out = cached;
    return GPTQ_OK;
}

// 2-D row-major tensor of 16-bit or 32-bit elements: `inner` elements per row, `rows` rows, row pitch
// `pitch_bytes` (multiple of 16).  Box = box_inner x box_rows.  Out-of-range elements read as zero.
inline int make_tensor_map_2d(CUtensorMap *map, CUtensorMapDataType dtype, const void *base, uint64_t inner,
                              uint64_t rows, uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows,
                              CUtensorMapSwizzle swizzle)
{
    EncodeTiledFn encode;
    int st = get_encode_tiled(&encode);
    if (st) return st;
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, dtype, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
    return GPTQ_OK;
}

// x[rows, K] (fp16, row-major) seen as K / 64 tiles of [rows, 64]: dimensions (64, rows, K / 64) with strides
// (row pitch, 128 bytes).  A box of (64, box_rows, box_tiles) then lands as box_tiles consecutive 128-byte-swizzled
// [box_rows x 64] tiles - one copy where the 2-D view (whose swizzled inner extent is limited to 128 bytes) needs one
// per tile.  Rows beyond `rows` read as zero.
inline int make_tensor_map_ktiles(CUtensorMap *map, const void *base, uint64_t K, uint64_t rows, uint32_t box_rows,
                                  uint32_t box_tiles)
{
    EncodeTiledFn encode;
    int st = get_encode_tiled(&encode);
    if (st) return st;
    cuuint64_t dims[3] = {64, rows, K / 64};
    cuuint64_t strides[2] = {K * 2, 128};
    cuuint32_t box[3] = {64, box_rows, box_tiles};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
    return GPTQ_OK;
}

#ifdef __CUDACC__
// Tiled 3-D load global -> shared; c0 (innermost) * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
// Tiled 2-D load global -> shared; c0 is the innermost coordinate (c0 * element size must be a
// multiple of 16 bytes).  Completion is counted in bytes (the full box) on the mbarrier.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar,
                                                 uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_prefetch_descriptor(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
#endif

}  // namespace gptq
