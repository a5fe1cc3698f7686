// Tensor-core latent attention (placeholder until the tcgen05 kernel lands).
#include "nm_mla.cuh"

namespace nm {
int attention_partial_tc(const void *, const void *, AttnPartials, AttnPlan, int, float, cudaStream_t) { return NM_ERR_UNSUPPORTED; }
}  // namespace nm
