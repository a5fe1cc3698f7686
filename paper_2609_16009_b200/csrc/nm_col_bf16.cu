// Explicit instantiations of the column-major narrow-product kernels for bf16 inputs.
#include "nm_matmul_kernels.cuh"

namespace nm {
NM_INSTANTIATE(col, bf16_t, bf16_t)
NM_INSTANTIATE(col, bf16_t, float)
}  // namespace nm
