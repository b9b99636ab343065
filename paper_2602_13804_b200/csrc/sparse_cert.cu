// Fused sparse pass with the routing certificate: the register variants of the fused kernel.
#include "sparse_kernel.cuh"

namespace vsa {

cudaError_t launch_sparse_cert(const SparseArgs& a, int threads)
{
    if (threads == 128) return launch_threads<128, 0, true>(a);
    return threads == 512 ? launch_threads<512, 0, true>(a) : launch_threads<256, 0, true>(a);
}

}  // namespace vsa
