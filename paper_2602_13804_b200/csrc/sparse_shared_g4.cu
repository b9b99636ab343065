// Group-shared sparse pass (sparse_shared.cuh): instances for groups of four query heads.
#include "sparse_shared.cuh"

namespace vsa {

cudaError_t launch_sparse_shared_g4(const GroupSharedArgs& a) { return launch_shared_tok<4>(a); }

}  // namespace vsa
