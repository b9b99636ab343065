// Group-shared sparse pass (sparse_shared.cuh): instances for groups of one and two query heads, and the
// dispatch over the group size.
#include "sparse_shared.cuh"

namespace vsa {

cudaError_t launch_sparse_shared_g4(const GroupSharedArgs& a);
cudaError_t launch_sparse_shared_g8(const GroupSharedArgs& a);

bool sparse_shared_supported(const Geometry& g, int P)
{
    if (g.page_size != kPageSize) return false;   // 16-token pages only
    if (g.token_stride != kHeadDim || g.head_stride != (long long)kPageSize * kHeadDim) return false;
    if (g.group != 1 && g.group != 2 && g.group != 4 && g.group != 8) return false;
    return (size_t)shared_layout(g.group, P).total * 4 <= (size_t)227 * 1024;
}

cudaError_t launch_sparse_shared(const GroupSharedArgs& a)
{
    switch (a.g.group) {
        case 1: return launch_shared_tok<1>(a);
        case 2: return launch_shared_tok<2>(a);
        case 4: return launch_sparse_shared_g4(a);
        case 8: return launch_sparse_shared_g8(a);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace vsa
