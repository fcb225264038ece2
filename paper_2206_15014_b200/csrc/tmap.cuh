// Tensor maps (cuTensorMapEncodeTiled through the runtime's driver entry point) shared by the kernels that move
// tiles with TMA.
#pragma once
#include "common.cuh"
#include <cuda.h>
#include <cuda_runtime.h>
#include <mutex>

namespace nm {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        (void)cudaGetLastError();
    });
    return fn;
}

// The encoding is a pure function of its arguments (base address, shape, box, swizzle, element type), and layers are
// launched again and again on the same buffers: the last few maps are kept, so that a repeated launch does not pay
// the driver's encoding again (three maps per GEMM call; it shows in the latency of small problems).
struct TensorMapCache {
    struct Key {
        const void* base; uint64_t d0, d1; uint32_t b0, b1, swz, dtype, esize, kind;
        bool operator==(const Key& o) const {
            return base == o.base && d0 == o.d0 && d1 == o.d1 && b0 == o.b0 && b1 == o.b1 && swz == o.swz &&
                   dtype == o.dtype && esize == o.esize && kind == o.kind;
        }
    };
    static constexpr int kEntries = 32;
    Key keys[kEntries];
    CUtensorMap maps[kEntries];
    bool used[kEntries] = {};
    unsigned next = 0;
    std::mutex mu;
    bool find(const Key& k, CUtensorMap* out) {
        std::lock_guard<std::mutex> lock(mu);
        for (int i = 0; i < kEntries; ++i)
            if (used[i] && keys[i] == k) { *out = maps[i]; return true; }
        return false;
    }
    void put(const Key& k, const CUtensorMap& m) {
        std::lock_guard<std::mutex> lock(mu);
        const int i = (int)(next++ % kEntries);
        keys[i] = k; maps[i] = m; used[i] = true;
    }
};
inline TensorMapCache& tensor_map_cache() {
    static TensorMapCache cache;
    return cache;
}

// 2-D matrix [rows, row_elems] of `esize`-byte elements (dense pitch), box = [box_rows, box_elems].
inline int make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_elems,
                    uint32_t box_rows, uint32_t box_elems, CUtensorMapSwizzle swz,
                    CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_UINT8, uint32_t esize = 1) {
    const TensorMapCache::Key key{base, rows, row_elems, box_rows, box_elems, (uint32_t)swz, (uint32_t)dtype, esize, 2u};
    if (tensor_map_cache().find(key, map)) return NM_OK;
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return record_text_error("cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[2] = {row_elems, rows};
    cuuint64_t strides[1] = {row_elems * esize};
    cuuint32_t box[2] = {box_elems, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dtype, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_text_error("cuTensorMapEncodeTiled failed");
    tensor_map_cache().put(key, *map);
    return NM_OK;
}

// X viewed as [k-slice][token][128 bytes] so that one box covers several 128-byte-wide slices of a token tile.
inline int make_map_x3(CUtensorMap* map, const void* base, uint64_t tokens, uint64_t k_bytes, uint32_t box_rows, uint32_t box_slices) {
    const TensorMapCache::Key key{base, tokens, k_bytes, box_rows, box_slices, 0u, 0u, 1u, 3u};
    if (tensor_map_cache().find(key, map)) return NM_OK;
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return record_text_error("cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {128, tokens, k_bytes / 128};
    cuuint64_t strides[2] = {k_bytes, 128};
    cuuint32_t box[3] = {128, box_rows, box_slices};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_text_error("cuTensorMapEncodeTiled failed for the 3-D view of X");
    tensor_map_cache().put(key, *map);
    return NM_OK;
}

}  // namespace nm
