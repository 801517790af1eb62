// Instantiation of the edge-stream kernels for K-chunk 16 (directional state of the double backward).
#include "edge_stream_impl.cuh"

namespace sobek {

cudaError_t stream_launch_k16_dual(const void* args, int cls, int t_begin, int t_count, cudaStream_t s) {
    return launch_class<16, true>(cls, *(const StreamArgs*)args, t_begin, t_count, s);
}

}  // namespace sobek
