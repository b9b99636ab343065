// Fused sparse pass, closed-form weights: the kernel variants without iterative solve or certificate.
#include "sparse_kernel.cuh"

namespace vsa {

cudaError_t launch_sparse_plain(const SparseArgs& a, int threads)
{
    if (threads == 128) return launch_threads_128<>(a);
    return threads == 512 ? launch_threads<512, 0, false>(a) : launch_threads<256, 0, false>(a);
}

}  // namespace vsa
