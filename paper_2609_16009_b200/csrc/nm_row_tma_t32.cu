// Explicit instantiations of the TMA-ring row-major kernel, 32 threads per weight row.
#include "nm_row_tma.cuh"

namespace nm {
NM_INSTANTIATE_TMA(32, bf16_t)
NM_INSTANTIATE_TMA(32, float)
}  // namespace nm
