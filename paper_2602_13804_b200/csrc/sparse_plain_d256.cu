// Fused sparse pass, closed-form weights, head dimension 256.
#include "sparse_kernel.cuh"

namespace vsa {

cudaError_t launch_sparse_plain_d256(const SparseArgs& a, int threads)
{
    if (threads == 128) return launch_threads_128<256>(a);
    return threads == 512 ? launch_threads<512, 0, false, 256>(a) : launch_threads<256, 0, false, 256>(a);
}

}  // namespace vsa
