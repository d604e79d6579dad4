// Host helpers of the tensor-core GEMM: TMA descriptor encoding and device queries.
#pragma once
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace peak {
namespace umma {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    });
    return fn;
}

// Tensor map over a stack of `batch` row-major 2-D arrays `batch_stride` elements apart: `inner` contiguous
// elements per row, `outer` rows, `pitch` elements between rows; box = box_inner x box_outer x 1, 128-byte
// swizzle, zero fill.  batch <= 1 gives a two-dimensional map of the one matrix.
// `swizzle_bytes`: 128 (the tensor-core tiles), 64, or 0 for a dense box.
inline bool encode_map(CUtensorMap *tm, Elem e, const void *base, int64_t inner, int64_t outer, int64_t pitch,
                       int box_inner, int box_outer, int64_t batch, int64_t batch_stride, int swizzle_bytes = 128) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const CUtensorMapDataType dt = e == Elem::F16    ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                   : e == Elem::BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                   : is_fp8(e)       ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                                     : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    const cuuint64_t eb = (cuuint64_t)elem_bytes(e);
    const cuuint32_t rank = batch > 1 ? 3 : 2;  // a single matrix gets a two-dimensional descriptor
    cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)(batch < 1 ? 1 : batch)};
    cuuint64_t strides[2] = {(cuuint64_t)pitch * eb, (cuuint64_t)batch_stride * eb};
    cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapSwizzle sw = swizzle_bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
                                  : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                        : CU_TENSOR_MAP_SWIZZLE_NONE;
    CUresult r = fn(tm, dt, rank, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Descriptor cache.  A tensor map is a pure function of the arguments above (it holds an address and a
// shape, no reference to the memory), so a call that repeats a (pointer, shape, pitch, box) combination --
// the same weights every step, a buffer reused across layers -- takes the 128-byte descriptor from a small
// direct-mapped table instead of encoding it again.  The table is per host thread: no lock, no sharing.
struct MapKey {
    const void *base;
    int64_t inner, outer, pitch, batch, batch_stride;
    int elem, box_inner, box_outer, swizzle;
    bool operator==(const MapKey &o) const {
        return base == o.base && inner == o.inner && outer == o.outer && pitch == o.pitch && batch == o.batch &&
               batch_stride == o.batch_stride && elem == o.elem && box_inner == o.box_inner &&
               box_outer == o.box_outer && swizzle == o.swizzle;
    }
};
constexpr int kMapCacheSlots = 64;
struct MapCache {
    MapKey key[kMapCacheSlots];
    CUtensorMap map[kMapCacheSlots];
    bool used[kMapCacheSlots];
    uint64_t hits, misses;
};
inline MapCache &map_cache() {
    thread_local MapCache c{};
    return c;
}
inline bool make_map(CUtensorMap *tm, Elem e, const void *base, int64_t inner, int64_t outer, int64_t pitch, int box_inner,
                     int box_outer, int64_t batch = 1, int64_t batch_stride = 0, int swizzle_bytes = 128) {
    const MapKey k{base, inner, outer, pitch, batch, batch_stride, (int)e, box_inner, box_outer, swizzle_bytes};
    uint64_t h = (uint64_t)reinterpret_cast<uintptr_t>(base) >> 4;
    h ^= (uint64_t)inner * 0x9E3779B97F4A7C15ull;
    h ^= ((uint64_t)outer + 0x7F4A7C15ull) * 0xC2B2AE3D27D4EB4Full;
    h ^= (uint64_t)(box_outer * 131 + box_inner + swizzle_bytes * 7919) * 0x165667B19E3779F9ull;
    h ^= h >> 29;
    MapCache &c = map_cache();
    const int slot = (int)(h % kMapCacheSlots);
    if (c.used[slot] && c.key[slot] == k) {
        *tm = c.map[slot];
        ++c.hits;
        return true;
    }
    if (!encode_map(tm, e, base, inner, outer, pitch, box_inner, box_outer, batch, batch_stride, swizzle_bytes)) return false;
    c.key[slot] = k;
    c.map[slot] = *tm;
    c.used[slot] = true;
    ++c.misses;
    return true;
}

inline int sm_count() {
    static int sms[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return 148;
    if (sms[dev] == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        sms[dev] = n > 0 ? n : 148;
    }
    return sms[dev];
}


}  // namespace umma
}  // namespace peak
