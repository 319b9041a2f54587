// Layer-output metric: Y = X W^T against its quantised counterparts (Section 3.2, layer analysis).
#include "mofq_internal.h"

namespace mofq {

size_t layer_metric_ws_bytes(const mofq_layer *, int, const mofq_config *) { return 0; }

int layer_metric_run(const mofq_layer &, const mofq_config *, mofq_result *, float *, float *, void *, size_t, cudaStream_t)
{
    return MOFQ_ERR_UNSUPPORTED;
}

}  // namespace mofq
