// The persistent form of the fused chain kernel (pf_tc_chain_kernel.cuh), compiled in a translation
// unit of its own: with both forms in one module the single-tile form, which the one-wave layers run,
// measurably slowed down inside a training step although the persistent form was never launched there.
#include <cuda.h>

#include "pf_tc.h"
#include "pf_tc_host.h"
#include "pf_tc_chain_kernel.cuh"
#include "pf_tc_chain_pipe.cuh"

namespace pf {
namespace tc {

int chain_launch_multi(dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& ta, const CUtensorMap& tb1,
                       const CUtensorMap& tb2, const CUtensorMap& to, const CUtensorMap& tt, const ChainParams& p) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_chain_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    if (launch_overlapped(tc_chain_kernel<true>, grid, dim3(kChainThreads), smem, stream, ta, tb1, tb2, to, tt, p) !=
        cudaSuccess)
        return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

// The software-pipelined persistent form (pf_tc_chain_pipe.cuh), r <= 128.
int chain_launch_pipe(dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& ta, const CUtensorMap& tb1,
                      const CUtensorMap& tb2, const CUtensorMap& to, const CUtensorMap& tt, const ChainParams& p) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(tc_chain_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return PF_ERR_CUDA;
        configured[dev] = true;
    }
    if (launch_overlapped(tc_chain_pipe_kernel, grid, dim3(kChainThreads), smem, stream, ta, tb1, tb2, to, tt, p) != cudaSuccess)
        return PF_ERR_CUDA;
    count_launch();
    return PF_OK;
}

}  // namespace tc
}  // namespace pf
