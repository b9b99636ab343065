// Fused sparse pass with an iterative solve on the candidate set: entropic mirror descent (kind 1) and
// Frank-Wolfe (kind 2) variants of the kernel, 256 threads.
#include "sparse_kernel.cuh"

namespace vsa {

cudaError_t launch_sparse_solve(const SparseArgs& a)
{
    return a.solver_kind == 2 ? launch_threads<256, 2, false>(a) : launch_threads<256, 1, false>(a);
}

}  // namespace vsa
