// Tensor-core (tcgen05) scoring kernels.  Placeholder until the kernels land: reports "unsupported" so that every
// configuration runs on the CUDA-core kernels.
#include "aif_internal.h"

namespace aif {

bool tc_supported(const aif_config &) { return false; }
cudaError_t tc_prepare_weights(aif_ctx *, const aif_weights *, cudaStream_t) { return cudaSuccess; }
cudaError_t launch_score_tc(const aif_ctx *, const ScoreLaunch &, int64_t, cudaStream_t) { return cudaErrorNotSupported; }
int tc_tiles_for(const aif_ctx *, int) { return 0; }

}  // namespace aif
