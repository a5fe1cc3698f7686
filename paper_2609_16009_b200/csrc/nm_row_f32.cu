// Explicit instantiations of the row-major narrow-product kernels for f32 inputs.
#include "nm_matmul_kernels.cuh"

namespace nm {
NM_INSTANTIATE(row, float, float)
}  // namespace nm
