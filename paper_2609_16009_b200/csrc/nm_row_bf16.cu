// Explicit instantiations of the row-major narrow-product kernels for bf16 inputs.
#include "nm_matmul_kernels.cuh"

namespace nm {
NM_INSTANTIATE(row, bf16_t, bf16_t)
NM_INSTANTIATE(row, bf16_t, float)
}  // namespace nm
