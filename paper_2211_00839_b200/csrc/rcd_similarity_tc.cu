// Tensor-core similarity kernel (placeholder until the tcgen05 path lands).
#include "rcd_internal.h"

namespace rcd {

rcd_status launch_similarity_tc(rcd_ctx *ctx, const void *Xs, rcd_feat_dtype dtype, int64_t Ntot, int64_t d,
                                const SimClasses &cls, void *S, cudaStream_t st, bool *handled)
{
    (void)ctx; (void)Xs; (void)dtype; (void)Ntot; (void)d; (void)cls; (void)S; (void)st;
    *handled = false;
    return RCD_OK;
}

}  // namespace rcd
