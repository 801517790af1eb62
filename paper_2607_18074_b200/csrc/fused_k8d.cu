// Instantiation of the fused kernels for 8 radial components per stage (directional state).
#include "fused_impl.cuh"

namespace sobek {

cudaError_t fused_launch_k8_dual(int D, const CUtensorMap& th, const CUtensorMap& tl, const void* args, int grid, size_t sh,
                     cudaStream_t s) {
    return launch_fused_d<8, true>(D, th, tl, *(const FusedArgs*)args, grid, sh, s);
}

}  // namespace sobek
