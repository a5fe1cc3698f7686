// Shared declarations of the MLA decode-step kernels.
#pragma once

#include "nm_common.cuh"

namespace nm {

constexpr int kAttnTileRows = 64;        // cache rows per attention tile
constexpr int kMaxAttnSplits = 128;      // upper bound on sequence splits (sizes the workspace)
constexpr int kAttnCluster = 4;          // splits merged on chip by the tensor-core kernel (cluster size)

// Per split s and head h: ml[(s*H+h)*2] = running max of the scaled scores, [..+1] = sum of
// exp(score - max); O[(s*H+h)*dc + c] = sum_j exp(score_j - max) * cache[j][c]  (not normalised).
struct AttnPartials {
    float *ml;
    float *O;
};

struct AttnPlan {
    int nsplit;
    int rows_per_split;                  // multiple of kAttnTileRows
    int tensor_core;                     // 1: tcgen05 kernel (partials merged per cluster), 0: CUDA-core kernel
    int npartial;                        // partial results the final merge has to read
};

AttnPlan plan_attention(const void *Q, const void *cache, int H, int n_rows, int kv_lora);

// Tensor-core (tcgen05 / TMEM) pass over the rows of each split.  Returns NM_ERR_UNSUPPORTED when
// the shape is not one it takes (the caller then uses the CUDA-core kernel).
int attention_partial_tc(const void *Q, const void *cache, AttnPartials part, AttnPlan plan, int n_rows,
                         float scale, cudaStream_t stream, bool programmatic_launch);

// Tuning aid: 12 phase timestamps (ns) of CTA (0,0) of the tensor-core kernel go to `p` when non-null.
void set_attention_trace(unsigned long long *p);

}  // namespace nm
