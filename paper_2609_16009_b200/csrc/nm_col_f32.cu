// Explicit instantiations of the column-major narrow-product kernels for f32 inputs.
#include "nm_matmul_kernels.cuh"

namespace nm {
NM_INSTANTIATE(col, float, float)
}  // namespace nm
