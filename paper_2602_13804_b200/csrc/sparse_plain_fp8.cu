// Fused sparse pass, closed-form weights, fp8 (e4m3) KV cache.
#include "sparse_kernel.cuh"

namespace vsa {

cudaError_t launch_sparse_plain_fp8(const SparseArgs& a, int threads)
{
    if (threads == 128) return launch_threads_128<kHeadDim, true>(a);
    return threads == 512 ? launch_threads<512, 0, false, kHeadDim, true>(a)
                          : launch_threads<256, 0, false, kHeadDim, true>(a);
}

}  // namespace vsa
