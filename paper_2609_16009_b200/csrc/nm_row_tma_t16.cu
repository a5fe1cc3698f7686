// Explicit instantiations of the TMA-ring row-major kernel, 16 threads per weight row.
#include "nm_row_tma.cuh"

namespace nm {
NM_INSTANTIATE_TMA(16, bf16_t)
NM_INSTANTIATE_TMA(16, float)
}  // namespace nm
