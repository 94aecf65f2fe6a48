// Lazy ratio (Eq. 1), tensor-core path.  Placeholder until the MMA kernel lands:
// reports "unsupported" so that every shape takes the CUDA-core path.
#include "lt_internal.h"

namespace lt {

bool scores_mma_supported(const lt_shape&, int) { return false; }

cudaError_t launch_scores_mma(const ScoreArgs&, const LayerTable&, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace lt
