// pf_lowrank_linear_fwd_static: the factorized linear forward for callers that cannot allocate
// device memory.  The scratch that pf_lowrank_linear_fwd takes as a caller-provided workspace
// lives here in a fixed device array that is part of the library image.
#include <mutex>

#include "pf.h"
#include "pf_internal.h"

namespace {

// Every GPU that loads this library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = PF_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code the array's name is only a handle for the runtime, not a device address: the
// address a kernel can use must be asked for, per device, with that device current.
std::mutex g_setup_mutex;
void* g_scratch_ptr[64] = {};

int static_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return PF_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return PF_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return PF_OK;
}

}  // namespace

extern "C" int pf_lowrank_linear_fwd_static(const void* x, int64_t ldx, const void* U, int64_t ldu,
                                            const void* V, int64_t ldv, void* y, int64_t ldy,
                                            void* T_stash, int64_t ldt,
                                            int64_t m, int64_t k, int64_t n, int64_t r, int dtype,
                                            void* cuda_stream) {
    if ((dtype != PF_F32 && dtype != PF_BF16) || m < 0 || k < 1 || n < 1 || r < 1)
        return PF_ERR_INVALID_ARG;
    void* scratch = nullptr;
    const int st = static_scratch(&scratch);
    if (st != PF_OK) return st;
    // The bound is what this call will really use, not the public workspace query (which reserves for
    // every path a call of these sizes could take): the fused kernel keeps x U on chip and needs at
    // most one m x r copy of it, the unfused paths add re-pitched operand copies and fp32 slices.  A
    // problem that needs more than the array is refused here, before anything is launched.
    // Nothing in the forward reads scratch before writing it (the intermediate x U and the
    // re-pitched operand copies are fully rewritten, pad columns included), so the previous
    // call's contents need no clearing.
    return pf::linear_fwd_impl(x, ldx, U, ldu, V, ldv, y, ldy, T_stash, ldt, m, k, n, r, dtype, scratch,
                               kStaticScratchBytes, cuda_stream, true);
}

extern "C" size_t pf_static_scratch_bytes(void) { return kStaticScratchBytes; }
