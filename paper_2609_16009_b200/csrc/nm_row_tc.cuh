// Swap-AB tensor-core narrow product (bf16 B, row- or column-major): launch interface.
#pragma once

#include <cuda.h>

#include "nm_matmul_kernels.cuh"

namespace nm {

constexpr int kTcTN = 128;      // columns of C per CTA (the MMA's M)
constexpr int kTcKT = 64;       // k-rows per stage

// Token columns of the accumulator for M tokens: 16, 32 or 64.
int row_tc_tokens(int M);
size_t row_tc_smem_bytes(int nstage, size_t slot_bytes = 0, int tokens = 16);
// Clusters of `cluster_size` CTAs (split-K inside a cluster, M tokens) the GPU holds at once; 0 without a device.
int row_tc_max_clusters(int cluster_size, int nstage, int M, bool col_major, bool f32_out);
// map_b: row-major B as bf16 [H][K][N], boxes {64, 64, 1}; column-major B as bf16 [H][N][K], boxes {64, 128, 1}; both with
// 128-byte swizzle; map_a: A as bf16 [H][M][K], boxes {64, 16, 1}, 128-byte swizzle.  ta.base.tn must be kTcTN and
// ta.base.kr a multiple of kTcKT.
template <typename TO>
cudaError_t launch_row_tc(const CUtensorMap &map_b, const CUtensorMap &map_a, const TmaArgs &ta, cudaStream_t s, bool col_major);

}  // namespace nm
