// Host-side helpers of the tensor-core path: TMA tensor-map encoding through the driver entry
// point (looked up at run time, so the library has no link-time dependency on libcuda).
#ifndef PF_TC_HOST_H_
#define PF_TC_HOST_H_

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace pf {
namespace tc {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return static_cast<EncodeTiledFn>(nullptr);
        return reinterpret_cast<EncodeTiledFn>(ptr);
    }();
    return fn;
}

// 2-D bf16 tensor map over a row-major [rows, cols] matrix with row pitch ld (elements); boxes are
// 64 columns (128 bytes, the swizzle span) by box_rows rows; out-of-range elements read as zero.
inline bool make_map_2d(CUtensorMap* map, const void* p, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
    const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(p), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Encoding a tensor map costs a driver call of about a microsecond, and a training step issues the
// same few maps over and over, so encoded maps are kept in a small direct-mapped cache keyed by
// everything the encoding depends on (the map holds no data, only addresses and shapes).
struct MapKey {
    const void* p;
    int64_t rows, cols, ld;
    int box_rows;
    bool operator==(const MapKey& o) const {
        return p == o.p && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows;
    }
};
inline bool cached_map_2d(CUtensorMap* map, const void* p, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    constexpr int kSlots = 512;
    struct Slot { MapKey key; CUtensorMap map; bool used; };
    static Slot slots[kSlots];
    static std::mutex mu;
    const MapKey key{p, rows, cols, ld, box_rows};
    uint64_t h = reinterpret_cast<uintptr_t>(p) * 0x9E3779B97F4A7C15ull;
    h ^= static_cast<uint64_t>(rows) * 0xC2B2AE3D27D4EB4Full + static_cast<uint64_t>(cols) * 0x165667B19E3779F9ull +
         static_cast<uint64_t>(ld) * 31 + static_cast<uint64_t>(box_rows);
    Slot& s = slots[(h >> 20) % kSlots];
    std::lock_guard<std::mutex> lock(mu);
    if (s.used && s.key == key) { *map = s.map; return true; }
    if (!make_map_2d(map, p, rows, cols, ld, box_rows)) return false;
    s.key = key; s.map = *map; s.used = true;
    return true;
}

inline bool tma_ok(const void* p, int64_t ld) {
    return (reinterpret_cast<uintptr_t>(p) & 15) == 0 && (ld % 8) == 0 && ld * 2 < (1LL << 40);
}


}  // namespace tc
}  // namespace pf
#endif
