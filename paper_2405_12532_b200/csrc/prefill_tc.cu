// tcgen05 path placeholder: not yet available, the dispatcher uses the CUDA-core kernels.
#include "pyr_internal.h"

namespace pyr {
bool prefill_tc_supported(const PrefillArgs&) { return false; }
cudaError_t launch_prefill_tc(const PrefillArgs&, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_score_tc(const PrefillArgs&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace pyr
