// Instantiations of the GEMM kernel for one container and problem kind (a translation unit of its own so that the
// instantiations compile in parallel).
#include "hq_gemm_kernel.cuh"

namespace hq {
namespace gemm {

cudaError_t launch_i8_gemm(int mode, int grid, size_t smem, cudaStream_t st, const CUtensorMap& tmA,
                           const CUtensorMap& tmB, const CUtensorMap& tmY, const GemmParams& p) {
    return dispatch<false, false>(mode, grid, smem, st, tmA, tmB, tmY, p);
}

}  // namespace gemm
}  // namespace hq
