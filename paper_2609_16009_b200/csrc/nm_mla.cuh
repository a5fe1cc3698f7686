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
    int rows_per_split;                  // multiple of kAttnTileRows (of tile_rows for the wide-tile kernel)
    int tensor_core;                     // 0: CUDA-core kernel; tcgen05 kernels: 1 = 128 heads per CTA, 32-row tiles; 2 = 64 heads per CTA;
                                         // 3 = 128 heads per CTA, wide tiles (nm_attn_wide.cu)
    int npartial;                        // partial results the final merge has to read
    int tile_rows, cluster;              // wide-tile kernel: cache rows per tile (64, 128, 256) and row runs merged on chip (1, 2, 4)
};

AttnPlan plan_attention(const void *Q, const void *cache, int H, int n_rows, int kv_lora);

// Tensor-core (tcgen05 / TMEM) pass over the rows of each split.  Returns NM_ERR_UNSUPPORTED when
// the shape is not one it takes (the caller then uses the CUDA-core kernel).
// Weight bytes pulled into L2 while the tensor cores work (by the merge kernel's idle prologue, or by a warp of
// the attention kernel): one
// contiguous block plus `nranges` ranges of `range_bytes`, `range_stride` apart (all may be empty).
struct L2Prefetch {
    const char *block;
    long block_bytes;
    const char *base;
    long range_stride;
    int nranges;
    long range_bytes;
};

int attention_partial_tc(const void *Q, const void *cache, AttnPartials part, AttnPlan plan, int n_rows,
                         float scale, cudaStream_t stream, bool programmatic_launch, L2Prefetch prefetch);

// The same pass over several independent sequences in one launch (small-batch decode): sequence t has its own
// cache rows, row count and split plan; its queries are rows [128 t, 128 t + 128) of Q, its partials start
// slot_stride slots after those of sequence t - 1.  All sequences use the same number of splits.
constexpr int kMaxBatch = 16;
int attention_partial_tc_batch(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split,
                               int nsplit, AttnPartials part, int slot_stride, float scale, cudaStream_t stream,
                               bool programmatic_launch, L2Prefetch prefetch = L2Prefetch{});

// Fused per-head stages of the decode step (nm_head_kernels.cu); they take nope = 128, kv_lora = 512, v = 128.
bool head_kernels_apply(int H, int nope, int rope, int dc, int dv);
bool down_finish_applies(int q_lora, int dc, int rope);
int launch_down_finish(const void *x, const void *gamma_q, const void *gamma_kv, const float *cos_sin, void *c_qn, void *cache_row,
                       int q_lora, int dc, int rope, float eps, cudaStream_t s, bool pdl);
// Consumers of the KV part of the down-projection (RMSNorm of the latent, RoPE of the key part, the cache-row
// write) for one extra CTA of the per-head query kernel: they are not needed before the attention merge, so they
// ride along there instead of ending the down-projection.
struct KvFinish {
    int enabled;
    const uint16_t *ckr;                   // [dc + rope] raw outputs of h * (W_DKV | W_KR)
    const uint16_t *gamma;
    const float *cos_sin;
    uint16_t *cache_row;
    int dc, rope;
    float eps;
};
int launch_q_finish(const void *q, const void *W_UK, const float *cos_sin, void *q_full, int H, int rope, cudaStream_t s, bool pdl,
                    KvFinish kv = KvFinish{});
int launch_uv_merge(const void *Q, const void *cache, AttnPartials part, int npart, long extra_row, int rope, float scale,
                    const void *W_UV, void *o_lat_bf16, float *o_lat_f32, void *o, int H, cudaStream_t s, bool pdl,
                    L2Prefetch prefetch = L2Prefetch{});

// The pass with 64 heads per CTA (nm_attn_tc64.cu): four CTAs per split, 64-row cache stages.  rows_per_split must be
// multiples of 64.  Same partial layout as the 128-head kernel.
int attention_tc64_max_clusters(int cluster);      // clusters of that many CTAs of the kernel resident at once
int attention_partial_tc64(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split, int nsplit,
                           int cluster /* splits merged on chip: 4, 2 or 1 */, AttnPartials part, int slot_stride, float scale, cudaStream_t stream, bool programmatic_launch,
                           L2Prefetch prefetch);

// The pass with wide score tiles (nm_attn_wide.cu): all 128 heads per CTA, tile_rows (64, 128 or 256) cache rows per
// scores MMA, two CTAs (column halves) per row run; rows_per_split must be multiples of tile_rows.  Same partial layout.
int attention_partial_wide(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split, int nsplit,
                           int tile_rows, int cluster /* row runs merged on chip: 4, 2 or 1 */, AttnPartials part, int slot_stride, float scale,
                           cudaStream_t stream, bool programmatic_launch, L2Prefetch prefetch);

// Small-batch decode (nm_batch_kernels.cu): per-sequence rows and partial counts of one launch.
struct BatchRows {
    long new_row[kMaxBatch];             // element offset, from the cache base, of the row each sequence's step writes
    int npart[kMaxBatch];                // attention partials to merge for each sequence
    int slot_stride;                     // partial slots between consecutive sequences
};
int launch_down_finish_batch(const void *x, const void *gamma_q, const void *gamma_kv, const float *cos_sin, void *c_qn, void *cache,
                             const BatchRows &rows, int T, int q_lora, int dc, int rope, float eps, cudaStream_t s, bool pdl);
int launch_q_finish_batch(const void *q, const void *W_UK, const float *cos_sin, void *q_full, int H, int rope, int T, cudaStream_t s, bool pdl);
int launch_uv_merge_batch(const void *Q, const void *cache, AttnPartials part, const BatchRows &rows, int T, int rope, float scale,
                          const void *W_UV, void *o_lat_bf16, void *o, int H, cudaStream_t s, bool pdl);

// The same stages without the per-head products (those then run as batched products on the tensor cores).
int launch_rope_batch(const void *q, const float *cos_sin, void *q_full, int H, int nope, int dc, int rope, int T, cudaStream_t s, bool pdl);
int launch_attn_merge_batch(const void *Q, const void *cache, AttnPartials part, const BatchRows &rows, int T, int rope, float scale,
                            void *o_lat_bf16, int H, cudaStream_t s, bool pdl);

// Tuning aid: phase timestamps (ns) of the tensor-core kernel go to `p` when non-null: 32 slots for CTA (0,0),
// then four per CTA (start, Q landed, last P*V done, end); 32 + 4 * 256 values at most.
void set_attention_trace(unsigned long long *p);
unsigned long long *attention_trace();

}  // namespace nm
