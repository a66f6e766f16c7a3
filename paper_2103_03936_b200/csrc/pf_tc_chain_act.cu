// The fused chain kernel (pf_tc_chain_kernel.cuh) with the bias / activation output epilogue, both the
// single-tile and the persistent form, compiled in a translation unit of its own so that the plain
// forms keep their code and placement.
#include <cuda.h>

#include "pf_tc.h"
#include "pf_tc_host.h"
#include "pf_tc_chain_kernel.cuh"

namespace pf {
namespace tc {

int chain_launch_act(bool persistent, dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& ta,
                     const CUtensorMap& tb1, const CUtensorMap& tb2, const CUtensorMap& to, const CUtensorMap& tt,
                     const ChainParams& p) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_chain_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess ||
            cudaFuncSetAttribute(tc_chain_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    const cudaError_t e =
        persistent ? launch_overlapped(tc_chain_kernel<true, true>, grid, dim3(kChainThreads), smem, stream, ta, tb1, tb2, to, tt, p)
                   : launch_overlapped(tc_chain_kernel<false, true>, grid, dim3(kChainThreads), smem, stream, ta, tb1, tb2, to, tt, p);
    if (e != cudaSuccess) return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

}  // namespace tc
}  // namespace pf
