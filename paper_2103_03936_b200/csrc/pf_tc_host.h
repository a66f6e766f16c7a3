// Host-side helpers of the tensor-core path: TMA tensor-map encoding through the driver entry
// point (looked up at run time, so the library has no link-time dependency on libcuda).
#ifndef PF_TC_HOST_H_
#define PF_TC_HOST_H_

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <utility>

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

// 4-D bf16 tensor map over an NHWC image [N, H, W, C]: boxes are 64 channels x box_w x box_h pixels
// of one image (box_w * box_h rows of 128 bytes in shared memory, pixel-major); coordinates may
// start outside the image (zero padding of the convolution), out-of-range pixels read as zero.
inline bool cached_map_nhwc(CUtensorMap* map, const void* p, int64_t N, int64_t H, int64_t W, int64_t C,
                            int box_w, int box_h) {
    constexpr int kSlots = 64;
    struct Slot { MapKey key; CUtensorMap map; bool used; };
    static Slot slots[kSlots];
    static std::mutex mu;
    const MapKey key{p, N * 100003 + H, C, W, -(box_h * 1024 + box_w)};
    const uint64_t h = reinterpret_cast<uintptr_t>(p) * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(key.rows) * 31 +
                       static_cast<uint64_t>(C) * 131 + static_cast<uint64_t>(W) * 1031 + static_cast<uint64_t>(-key.box_rows);
    Slot& s = slots[(h >> 20) % kSlots];
    std::lock_guard<std::mutex> lock(mu);
    if (s.used && s.key == key) { *map = s.map; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W), static_cast<cuuint64_t>(H),
                                static_cast<cuuint64_t>(N)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(C) * 2, static_cast<cuuint64_t>(W) * C * 2,
                                   static_cast<cuuint64_t>(H) * W * C * 2};
    const cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(box_w), static_cast<cuuint32_t>(box_h), 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(p), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    s.key = key; s.map = *map; s.used = true;
    return true;
}

// 3-D view of a contiguous row-major [tiles * rows_tile, cols] matrix as [tiles][rows_tile][cols]:
// a store box of box_rows rows that starts inside a tile is clipped at the end of that tile, which
// is how partially filled 128-row MMA tiles (image rows that do not pack into 128 pixels) are
// written without touching the next tile's pixels.
inline bool cached_map_tiled_rows(CUtensorMap* map, const void* p, int64_t tiles, int rows_tile, int64_t cols,
                                  int box_rows) {
    constexpr int kSlots = 64;
    struct Slot { MapKey key; CUtensorMap map; bool used; };
    static Slot slots[kSlots];
    static std::mutex mu;
    const MapKey key{p, tiles, cols, rows_tile, -(1 << 24) - box_rows};
    const uint64_t h = reinterpret_cast<uintptr_t>(p) * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(tiles) * 31 +
                       static_cast<uint64_t>(cols) * 131 + static_cast<uint64_t>(rows_tile) * 1031 + box_rows;
    Slot& s = slots[(h >> 20) % kSlots];
    std::lock_guard<std::mutex> lock(mu);
    if (s.used && s.key == key) { *map = s.map; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows_tile),
                                static_cast<cuuint64_t>(tiles)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(cols) * 2, static_cast<cuuint64_t>(rows_tile) * cols * 2};
    const cuuint32_t box[3] = {64u, static_cast<cuuint32_t>(box_rows), 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(p), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    s.key = key; s.map = *map; s.used = true;
    return true;
}

// Launch with programmatic stream serialization: the kernel's prologue (barrier set-up, TMEM
// allocation, descriptor prefetch) overlaps the tail of the previous kernel in the stream; the
// kernel itself calls griddepcontrol.wait before it touches global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

inline bool tma_ok(const void* p, int64_t ld) {
    return (reinterpret_cast<uintptr_t>(p) & 15) == 0 && (ld % 8) == 0 && ld * 2 < (1LL << 40);
}


}  // namespace tc
}  // namespace pf
#endif
