// Explicit instantiations of the column-major narrow-product kernels for fp16 inputs (the optional element type).
#include "nm_matmul_kernels.cuh"

namespace nm {
NM_INSTANTIATE(col, f16_t, f16_t)
}  // namespace nm
