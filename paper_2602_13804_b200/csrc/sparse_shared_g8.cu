// Group-shared sparse pass (sparse_shared.cuh): instances for groups of eight query heads.
#include "sparse_shared.cuh"

namespace vsa {

cudaError_t launch_sparse_shared_g8(const GroupSharedArgs& a) { return launch_shared_tok<8>(a); }

}  // namespace vsa
