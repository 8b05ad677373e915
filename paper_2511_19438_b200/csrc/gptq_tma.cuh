// Tensor-map (TMA) plumbing: host-side encoding through the driver entry point (looked up at run
// time, so the library does not link libcuda) and the device-side tiled load.
#pragma once
#include <cuda.h>

#include <atomic>
#include <mutex>

#include "gptq_common.cuh"

namespace gptq {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline int get_encode_tiled(EncodeTiledFn *out)
{
    static std::atomic<EncodeTiledFn> cached{nullptr};
    EncodeTiledFn fnp = cached.load(std::memory_order_acquire);
    if (fnp == nullptr) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return record_cuda_error(e);
        if (q != cudaDriverEntryPointSuccess || fn == nullptr) return GPTQ_ERR_CUDA;
        fnp = (EncodeTiledFn)fn;
        cached.store(fnp, std::memory_order_release);   // every thread looks up the same pointer
    }
    *out = fnp;
    return GPTQ_OK;
}

// Encoding a tensor map costs the host a microsecond or two, and a decode step encodes hundreds: the maps are
// cached by everything that defines them (device, base pointer, extents, box, swizzle).  A map describes
// addresses and shapes only, never contents, so a cached entry stays valid for as long as the key matches.
struct TensorMapKey {
    int dev, kind;
    const void *base;
    uint64_t d0, d1, pitch;
    uint32_t b0, b1, b2, swizzle;
    bool operator==(const TensorMapKey &o) const
    {
        return dev == o.dev && kind == o.kind && base == o.base && d0 == o.d0 && d1 == o.d1 && pitch == o.pitch &&
               b0 == o.b0 && b1 == o.b1 && b2 == o.b2 && swizzle == o.swizzle;
    }
};
struct TensorMapCache {
    static constexpr int kSlots = 512;   // direct-mapped
    std::mutex mu;
    TensorMapKey keys[kSlots];
    CUtensorMap maps[kSlots];
    bool used[kSlots] = {};
    static size_t slot_of(const TensorMapKey &k)
    {
        uint64_t h = (uint64_t)(uintptr_t)k.base * 0x9E3779B97F4A7C15ull;
        h ^= (k.d0 * 31 + k.d1) * 0xC2B2AE3D27D4EB4Full + k.b1 * 131 + k.b2 * 17 + (uint64_t)k.kind * 7 + (uint64_t)k.dev;
        return (size_t)((h >> 20) % kSlots);
    }
    bool lookup(const TensorMapKey &k, CUtensorMap *out)
    {
        std::lock_guard<std::mutex> lock(mu);
        const size_t s = slot_of(k);
        if (!used[s] || !(keys[s] == k)) return false;
        *out = maps[s];
        return true;
    }
    void store(const TensorMapKey &k, const CUtensorMap &m)
    {
        std::lock_guard<std::mutex> lock(mu);
        const size_t s = slot_of(k);
        keys[s] = k;
        maps[s] = m;
        used[s] = true;
    }
};
inline TensorMapCache &tensor_map_cache()
{
    static TensorMapCache cache;
    return cache;
}
inline int current_device_or_error(int *dev)
{
    cudaError_t e = cudaGetDevice(dev);
    return e == cudaSuccess ? GPTQ_OK : record_cuda_error(e);
}

// 2-D row-major tensor of 16-bit or 32-bit elements: `inner` elements per row, `rows` rows, row pitch
// `pitch_bytes` (multiple of 16).  Box = box_inner x box_rows.  Out-of-range elements read as zero.
inline int make_tensor_map_2d(CUtensorMap *map, CUtensorMapDataType dtype, const void *base, uint64_t inner,
                              uint64_t rows, uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows,
                              CUtensorMapSwizzle swizzle)
{
    TensorMapKey key{0, (int)dtype, base, inner, rows, pitch_bytes, box_inner, box_rows, 0, (uint32_t)swizzle};
    int st = current_device_or_error(&key.dev);
    if (st) return st;
    if (tensor_map_cache().lookup(key, map)) return GPTQ_OK;
    EncodeTiledFn encode;
    st = get_encode_tiled(&encode);
    if (st) return st;
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, dtype, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
    tensor_map_cache().store(key, *map);
    return GPTQ_OK;
}

// x[rows, K] (fp16, row-major) seen as K / 64 tiles of [rows, 64]: dimensions (64, rows, K / 64) with strides
// (row pitch, 128 bytes).  A box of (64, box_rows, box_tiles) then lands as box_tiles consecutive 128-byte-swizzled
// [box_rows x 64] tiles - one copy where the 2-D view (whose swizzled inner extent is limited to 128 bytes) needs one
// per tile.  Rows beyond `rows` read as zero.
inline int make_tensor_map_ktiles(CUtensorMap *map, const void *base, uint64_t K, uint64_t rows, uint32_t box_rows,
                                  uint32_t box_tiles)
{
    TensorMapKey key{0, 1000, base, K, rows, 0, 64, box_rows, box_tiles, 0};
    int st = current_device_or_error(&key.dev);
    if (st) return st;
    if (tensor_map_cache().lookup(key, map)) return GPTQ_OK;
    EncodeTiledFn encode;
    st = get_encode_tiled(&encode);
    if (st) return st;
    cuuint64_t dims[3] = {64, rows, K / 64};
    cuuint64_t strides[2] = {K * 2, 128};
    cuuint32_t box[3] = {64, box_rows, box_tiles};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
    tensor_map_cache().store(key, *map);
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
__device__ __forceinline__ void tma_prefetch_descriptor(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
#endif

}  // namespace gptq
