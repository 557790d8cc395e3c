// Tensor-core forward kernel (placeholder until the tcgen05 path lands).
#include "tlin_internal.h"
namespace tlin {
int launch_fwd_tc(const void*, const void*, const void*, void*, float*, int, int, int, int, int, int,
                  const tlin_fwd_plan&, float*, cudaStream_t) {
    return TLIN_ERR_UNSUPPORTED;
}
}  // namespace tlin
