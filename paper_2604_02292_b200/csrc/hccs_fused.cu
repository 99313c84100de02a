// Fused int8 attention (placeholder translation unit until the tcgen05 kernel lands).
#include "hccs_internal.h"

namespace hccs {
bool fused_shape_supported(int32_t, int32_t) { return false; }
cudaError_t launch_fused(const FusedArgs &, cudaStream_t, uint64_t *) { return cudaErrorNotSupported; }
}  // namespace hccs
