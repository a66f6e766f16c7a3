// Flat gradient buffer (Pufferfish Section 4.1): every factor gradient is copied, in list
// order and tightly, into one contiguous buffer so that one all-reduce per iteration suffices.
//
// The copy is pure HBM streaming.  Tight packing means a tensor's destination is only
// element-aligned (2 bytes for bf16 after an odd-sized tensor), so source and destination
// are in general not co-aligned.  Each destination tensor is split into
//   head  : bytes up to the first 16-byte boundary of the destination   (element copies)
//   body  : whole 16-byte destination vectors; each is assembled from the two aligned 16-byte
//           source vectors that cover it, with a funnel shift, so both sides move 16 bytes
//           per access whatever the relative alignment
//   tail  : the bytes after the last whole vector                        (element copies)
// Work is cut into fixed-size chunks of destination vectors; a block finds its tensor by
// binary search in a prefix table passed by value in the kernel parameters (no device-side
// table, hence no workspace and no host-to-device copy).
#include "pf_internal.h"

namespace pf {
namespace {

constexpr int kPackBatch = 512;         // tensors per launch (the table travels in the kernel parameters: 14 KB of the 32 KB limit)
constexpr int kVecPerChunk = 512;       // 8 KB of destination per block-chunk
constexpr int kPackThreads = 256;

struct PackBatch {
    const unsigned char* src[kPackBatch];
    unsigned char* dst[kPackBatch];  // where each tensor's bytes go
    int64_t bytes[kPackBatch];
    int chunk_prefix[kPackBatch + 1];
    int count;
    int elem_bytes;
};

template <int Q>
__device__ __forceinline__ uint4 combine(const uint4 lo, const uint4 hi, unsigned bit_shift) {
    // bytes [4Q + bit_shift/8, +16) of the 32-byte window lo:hi
    const unsigned w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    uint4 o;
    o.x = __funnelshift_r(w[Q + 0], w[Q + 1], bit_shift);
    o.y = __funnelshift_r(w[Q + 1], w[Q + 2], bit_shift);
    o.z = __funnelshift_r(w[Q + 2], w[Q + 3], bit_shift);
    o.w = __funnelshift_r(w[Q + 3], w[Q + 4], bit_shift);
    return o;
}

__global__ void __launch_bounds__(kPackThreads)
pack_kernel(const PackBatch pb) {
    // which tensor does this chunk belong to?
    const int chunk = blockIdx.x;
    int lo = 0, hi = pb.count;  // invariant: prefix[lo] <= chunk < prefix[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pb.chunk_prefix[mid] <= chunk) lo = mid; else hi = mid;
    }
    const int t = lo;
    const int local_chunk = chunk - pb.chunk_prefix[t];
    // Launched with programmatic stream serialization: the table search above (kernel parameters
    // only) overlaps the tail of the kernel that produces the gradients; nothing in global memory
    // is touched before that kernel has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned char* src = pb.src[t];
    const int64_t bytes = pb.bytes[t];
    unsigned char* dst = pb.dst[t];
    const int es = pb.elem_bytes;

    // destination split
    const uintptr_t d0 = reinterpret_cast<uintptr_t>(dst);
    int64_t head = static_cast<int64_t>((16 - (d0 & 15)) & 15);
    if (head > bytes) head = bytes;
    const int64_t nvec = (bytes - head) / 16;
    const int64_t tail_beg = head + nvec * 16;

    if (local_chunk == 0) {
        // head and tail: element-granular copies by the first chunk's block
        for (int64_t b = threadIdx.x * es; b < head; b += kPackThreads * es) {
            if (es == 2) *reinterpret_cast<unsigned short*>(dst + b) = *reinterpret_cast<const unsigned short*>(src + b);
            else         *reinterpret_cast<unsigned int*>(dst + b) = *reinterpret_cast<const unsigned int*>(src + b);
        }
        for (int64_t b = tail_beg + threadIdx.x * es; b < bytes; b += kPackThreads * es) {
            if (es == 2) *reinterpret_cast<unsigned short*>(dst + b) = *reinterpret_cast<const unsigned short*>(src + b);
            else         *reinterpret_cast<unsigned int*>(dst + b) = *reinterpret_cast<const unsigned int*>(src + b);
        }
    }

    const int64_t v_beg = static_cast<int64_t>(local_chunk) * kVecPerChunk;
    int64_t v_end = v_beg + kVecPerChunk;
    if (v_end > nvec) v_end = nvec;
    const unsigned char* sbody = src + head;               // source byte matching dst vector 0
    const unsigned sh = static_cast<unsigned>(reinterpret_cast<uintptr_t>(sbody) & 15);
    const uint4* sal = reinterpret_cast<const uint4*>(sbody - sh);   // aligned-down source
    uint4* dvec = reinterpret_cast<uint4*>(dst + head);
    if (sh == 0) {
#pragma unroll 4
        for (int64_t v = v_beg + threadIdx.x; v < v_end; v += kPackThreads) dvec[v] = __ldg(sal + v);
    } else {
        const unsigned q = sh >> 2, bit = (sh & 3) * 8;
#pragma unroll 2
        for (int64_t v = v_beg + threadIdx.x; v < v_end; v += kPackThreads) {
            // Both aligned source vectors contain at least one byte of this tensor: the first
            // holds source byte 16v (valid), the second holds byte 16v+15 (valid because vector v
            // is a whole destination vector).
            const uint4 a = __ldg(sal + v), b = __ldg(sal + v + 1);
            uint4 o;
            switch (q) {
                case 0: o = combine<0>(a, b, bit); break;
                case 1: o = combine<1>(a, b, bit); break;
                case 2: o = combine<2>(a, b, bit); break;
                default: o = combine<3>(a, b, bit); break;
            }
            dvec[v] = o;
        }
    }
}

}  // namespace

// One launch per kPackBatch tensors: tensor i moves numels[i] elements from src(i) to dst(i).
template <typename SrcOf, typename DstOf>
static cudaError_t copy_list(const int64_t* numels, int count, int elem_bytes, SrcOf src_of, DstOf dst_of,
                             cudaStream_t stream) {
    int i = 0;
    while (i < count) {
        PackBatch pb;
        pb.count = 0;
        pb.elem_bytes = elem_bytes;
        pb.chunk_prefix[0] = 0;
        while (i < count && pb.count < kPackBatch) {
            if (numels[i] > 0) {
                const int64_t bytes = numels[i] * elem_bytes;
                const int64_t chunks = ceil_div(ceil_div(bytes, 16), kVecPerChunk);
                if (pb.chunk_prefix[pb.count] + chunks > 0x7fffffff) return cudaErrorInvalidValue;
                pb.src[pb.count] = src_of(i);
                pb.dst[pb.count] = dst_of(i);
                pb.bytes[pb.count] = bytes;
                pb.chunk_prefix[pb.count + 1] = pb.chunk_prefix[pb.count] + static_cast<int>(chunks);
                ++pb.count;
            }
            ++i;
        }
        if (pb.count == 0) continue;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(pb.chunk_prefix[pb.count]));
        cfg.blockDim = dim3(kPackThreads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, pack_kernel, pb);
        if (e != cudaSuccess) return e;
        count_launch();
    }
    return cudaSuccess;
}

cudaError_t pack_launch(const void* const* grads, const int64_t* numels, const int64_t* offsets,
                        int count, int elem_bytes, void* flat, cudaStream_t stream) {
    unsigned char* f = static_cast<unsigned char*>(flat);
    return copy_list(numels, count, elem_bytes,
                     [&](int i) { return static_cast<const unsigned char*>(grads[i]); },
                     [&](int i) { return f + offsets[i] * elem_bytes; }, stream);
}

// The inverse: tensor i receives flat[offsets[i] .. offsets[i] + numels[i]).  The same kernel with
// the roles swapped (the flat buffer is now the side that is only element-aligned).
cudaError_t unpack_launch(const void* flat, void* const* grads, const int64_t* numels, const int64_t* offsets,
                          int count, int elem_bytes, cudaStream_t stream) {
    const unsigned char* f = static_cast<const unsigned char*>(flat);
    return copy_list(numels, count, elem_bytes,
                     [&](int i) { return f + offsets[i] * elem_bytes; },
                     [&](int i) { return static_cast<unsigned char*>(grads[i]); }, stream);
}

}  // namespace pf
