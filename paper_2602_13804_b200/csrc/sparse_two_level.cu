// Fused sparse pass with the two-level routing front end (closed-form weights): the unit selects its
// super-pages, scores the pages inside them and routes the best of those in the same kernel.
#include "sparse_kernel.cuh"

namespace vsa {

cudaError_t launch_sparse_two_level(const SparseArgs& a, int threads)
{
    if (threads == 128) return launch_tok<128, -2, 0, false>(a);
    return threads == 512 ? launch_tok<512, -2, 0, false>(a) : launch_tok<256, -2, 0, false>(a);
}

}  // namespace vsa
