/*
 * nm - narrow matrix multiplication and single-token MLA decode for NVIDIA B200 (sm_100a).
 *
 * C-ABI boundary.  Every pointer is a DEVICE pointer unless a parameter is documented as
 * "host".  The caller owns every buffer and every stream; calls enqueue work on the given
 * stream and return without synchronising.  The library never allocates device memory: kernels
 * that need scratch (split-K partial sums, split-KV partial outputs) take it from a workspace
 * the caller provides.  On any error nothing is enqueued and a negative code is returned.
 *
 * Conventions
 *   A  row-major M x K, element (m,k) at m*K + k           (the token rows, 1 <= M <= 16)
 *   B  K x N weights; NM_ROW_MAJOR: element (k,n) at k*N + n
 *                     NM_COL_MAJOR: element (k,n) at n*K + k  (an [out,in] weight such as
 *                     W^{DKV} in R^{d_c x d}, MLA Operator Optimization section)
 *   C  row-major M x N, element (m,n) at m*N + n
 *   The other narrow case of the Narrow Dimension condition, N = 1, is served by transposition:
 *   C^T[1 x M] = B^T[1 x K] * A^T[K x M], i.e. pass the row-major A as a column-major B.
 *   Arithmetic: inputs are widened exactly to fp32, products accumulate in fp32, partial sums
 *   stay fp32, and the result is rounded once (round-to-nearest-even) to the output type
 *   (Data Type Issue section; Algorithm 2, gather stage and output cast).
 */
#ifndef NM_H
#define NM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *nm_stream;          /* a cudaStream_t */

typedef enum {
    NM_F32 = 0,                   /* fp32 in, fp32 out */
    NM_BF16 = 1,                  /* bf16 in, fp32 accumulate, bf16 out */
    NM_BF16_F32OUT = 2,           /* bf16 in, fp32 accumulate, fp32 out (unrounded sums) */
    NM_F16 = 3                    /* fp16 (IEEE binary16) in, fp32 accumulate, fp16 out.  Not a type the paper computes in (its
                                   * data is bf16; Data Type Issue section) - an optional element type of the same product.
                                   * Row- and column-major B: the swap-AB tensor-core kernel (weights of 8 MB and more,
                                   * operands it can address; also 17..NM_MAX_M_TENSOR rows) or the CUDA-core row / column
                                   * kernels; NM_FRACTAL_NZ returns NM_ERR_UNSUPPORTED. */
} nm_dtype;

/* Storage of B (K x N).  NM_FRACTAL_NZ: the tiling the paper's weight matrices have in memory (MLA Operator
 * Optimization section, figure of the special formats) - 16 x 16 fractals, the fractals ordered by columns (those of
 * the first 16 columns from top to bottom, then the next 16 columns), the elements of a fractal by rows: element
 * (k, n) at ((n/16)*(K/16) + k/16)*256 + (k%16)*16 + n%16.  bf16 only, K and N multiples of 16, M <= 16; read in
 * place by tiled TMA copies, no transposition pass.  NM_ERR_UNSUPPORTED otherwise. */
typedef enum { NM_ROW_MAJOR = 0, NM_COL_MAJOR = 1, NM_FRACTAL_NZ = 2 } nm_layout;

enum {
    NM_OK = 0,
    NM_ERR_INVALID_ARG = -1,      /* null pointer, M outside 1..16, N or K < 1, bad stride */
    NM_ERR_UNSUPPORTED = -2,      /* dtype / layout / dimension combination not built */
    NM_ERR_ALIGNMENT = -3,        /* a pointer is not aligned to its element size */
    NM_ERR_WORKSPACE = -4,        /* workspace missing or too small */
    NM_ERR_CUDA = -5,             /* a CUDA call failed; see nm_last_cuda_error() */
    NM_ERR_TIMEOUT = -6,          /* a bounded device-side wait expired (nm_check_status) */
    NM_ERR_TOO_LARGE = -7,        /* problem needs more scratch than nm_matmul_static has built in */
    NM_ERR_BOUNDS = -8            /* debug build (libnm_check.so) only: a kernel's access outside the operand it belongs to
                                   * was caught and skipped; reported by nm_check_status */
};

#define NM_MAX_M 16
/* More tokens than the narrow range proper (the paper's outlook: remainder rows, larger tokens): up to 64 rows are
 * taken in one pass over B by the tensor-core kernel when the operands qualify for it (bf16, 16-byte aligned A and B
 * with rows / columns that stay aligned); NM_ERR_UNSUPPORTED otherwise. */
#define NM_MAX_M_TENSOR 64

/* ---- misc ------------------------------------------------------------------------------- */

int nm_version(void);
const char *nm_status_string(int status);
/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char *nm_last_cuda_error(void);

/*
 * Synchronises `stream`, then reads and clears the device status word.  Returns NM_ERR_TIMEOUT
 * if a kernel gave up on a bounded wait (its output is then invalid), NM_OK otherwise.  Every
 * device-side wait in this library (on an mbarrier fed by a TMA copy or a tensor-core commit) is
 * limited to about a second, after which the kernel flags the error and runs to its end.
 */
int nm_check_status(nm_stream stream);

/* ---- workspace --------------------------------------------------------------------------- */

/*
 * Bytes of scratch nm_matmul / nm_matmul_batched may need for this problem: split-K partial
 * sums (fp32) plus arrival counters (Algorithm 1, "Partial Sum Buffer" tmpBuf and gather
 * stage).  H = 1 for the unbatched call.  The size does not depend on tuning overrides.
 */
size_t nm_matmul_workspace_bytes(int M, int N, int K, int H, nm_dtype dtype, nm_layout layout_B);

/*
 * Clear a workspace (enqueues one memset of `bytes` on `stream`); what matters are the arrival
 * counters in it.  Must be done once before first use; the kernels leave the counters at zero
 * afterwards, so no clearing is needed between calls.  `bytes` must be at least
 * NM_WS_COUNTER_BYTES.
 */
#define NM_WS_COUNTER_BYTES 65536
int nm_workspace_init(void *workspace, size_t bytes, nm_stream stream);

/*
 * Register a process-wide default workspace for nm_matmul and nm_matmul_batched (the calls
 * that follow the paper's problem statement and therefore carry no workspace argument).  The
 * memory stays owned by the caller and must outlive its use.  The call clears the counters with
 * a synchronous memset.  Two calls that use the default workspace must not overlap on the GPU
 * (use the _ws variants with distinct workspaces on concurrent streams).
 */
int nm_set_workspace(void *workspace, size_t bytes);

/* ---- narrow matrix product ------------------------------------------------------------------ */

/*
 * C[M x N] = A[M x K] * B[K x N], 1 <= M <= 16  (Narrow Dimension condition; Eq. 4 for
 * M = 1, K = 7168, N = 576; Algorithm 1 for the split-K / gather structure).
 * Any N, K >= 1 is accepted; the vectorised path needs 16-byte aligned A, B and N (row-major)
 * or K (column-major) a multiple of 16 bytes' worth of elements, otherwise a scalar kernel runs.
 * Uses the default workspace when the chosen tiling splits K; returns NM_ERR_WORKSPACE if none
 * is registered or it is too small.  17 <= M <= NM_MAX_M_TENSOR: see NM_MAX_M_TENSOR above.
 */
int nm_matmul(const void *A, const void *B, void *C, int M, int N, int K,
              nm_dtype dtype, nm_layout layout_B, nm_stream stream);

/* Same product with an explicit workspace (counters cleared once by nm_workspace_init). */
int nm_matmul_ws(const void *A, const void *B, void *C, int M, int N, int K,
                 nm_dtype dtype, nm_layout layout_B, void *workspace, size_t workspace_bytes,
                 nm_stream stream);

/*
 * H independent narrow products (per-head absorbed-MLA projections):
 *   C(m,h,:) = A(m,h,:) * B_h,   A(m,h,k) at m*lda + h*strideA + k,
 *   B_h dense K x N in layout_B at B + h*strideB,   C(m,h,n) at m*ldc + h*strideC + n
 * (all strides in elements).  q_nope can thus be read in place from q[T][H][nope+rope]
 * with lda = H*(nope+rope), strideA = nope+rope.
 */
int nm_matmul_batched(const void *A, const void *B, void *C, int M, int N, int K, int H,
                      long lda, long strideA, long strideB, long ldc, long strideC,
                      nm_dtype dtype, nm_layout layout_B, nm_stream stream);

int nm_matmul_batched_ws(const void *A, const void *B, void *C, int M, int N, int K, int H,
                         long lda, long strideA, long strideB, long ldc, long strideC,
                         nm_dtype dtype, nm_layout layout_B, void *workspace,
                         size_t workspace_bytes, nm_stream stream);

/*
 * End-to-end form with HOST operands: A_host (M x K) and C_host (M x N) are host buffers
 * (pinned for asynchronous copies), B stays on the device (the resident weight).  A is copied
 * through `A_staging` and C through `C_staging` (device buffers of M*K and M*N elements).
 * Enqueues copy-in, the product (explicit workspace) and copy-out on `stream`.
 */
int nm_matmul_host(const void *A_host, const void *B, void *C_host, void *A_staging,
                   void *C_staging, int M, int N, int K, nm_dtype dtype, nm_layout layout_B,
                   void *workspace, size_t workspace_bytes, nm_stream stream);

/*
 * The same product for callers that must not allocate.  (The paper has no counterpart: this is
 * an addition for embedding the library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits or cannot succeed - a plugin inside
 * a serving runtime whose memory pool was sized up front and has claimed the whole GPU, a latency
 * critical loop that may not take the device-wide synchronisation an allocation implies, or a
 * host that simply has no allocator to lend (a thin C program that only maps its inputs and
 * outputs).  Such a caller passes A, B and C as usual and nothing else: the split-K partial sums
 * and arrival counters go into a fixed NM_STATIC_SCRATCH_BYTES array that is part of the library's
 * device image (every GPU that loads the library holds it until the process exits).  The call
 * itself uses no cudaMalloc, cudaFree or any other allocating routine.
 *
 * Limits and rules:
 *  - a problem whose tiling needs more scratch than the array holds is refused with
 *    NM_ERR_TOO_LARGE and nothing is enqueued (the products of the MLA decode step at M <= 16 fit);
 *  - the first call on each device looks up the array's device address and enqueues one 64 KB
 *    memset of the counters on `stream`; make that first call before starting any stream capture;
 *  - all calls on a GPU share the one array, which keeps whatever the last call left in it; the
 *    kernels restore the counters themselves, but two calls that overlap on the GPU (different
 *    streams, or programmatic launch) race on the partial sums - issue them on one stream.
 */
#define NM_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)
int nm_matmul_static(const void *A, const void *B, void *C, int M, int N, int K,
                     nm_dtype dtype, nm_layout layout_B, nm_stream stream);

/* ---- single-token MLA decode step ------------------------------------------------------------------ */

/*
 * Vector-side stages that consume the narrow products (MLA Operator Optimization section: "RMS,
 * RoPE and caching normalization" start right after MatMul 2).  All tensors bf16.
 *   nm_rmsnorm:  y[i] = x[i] * rsqrt(mean(x^2) + eps) * gamma[i],  i < n  (n <= 16384), rounded to bf16
 *   nm_rope:     n_vec vectors of `dim` elements (vector v at x + v*x_stride, written to
 *                y + v*y_stride, strides in elements); interleaved pairs (x[2i], x[2i+1]) turn by the
 *                angle whose (cos, sin) is cos_sin[2i], cos_sin[2i+1] (fp32, one table row)
 *   nm_rope_table: fills table[(p - pos_begin)*dim + 2i + {0,1}] = (cos, sin)(p * base^(-2i/dim))
 *                for pos_begin <= p < pos_begin + n_pos, computed in fp64 on the device
 */
int nm_rmsnorm(const void *x, const void *gamma, void *y, int n, float eps, nm_stream stream);
int nm_rope(const void *x, void *y, int n_vec, int dim, long x_stride, long y_stride,
            const float *cos_sin, nm_stream stream);
int nm_rope_table(float *table, long pos_begin, int n_pos, int dim, double base, nm_stream stream);

/*
 * Absorbed latent attention for all heads of one token over cache rows [0, n_rows):
 *   s[h,j] = scale * <Q[h,:], cache[j,:]>,  p = softmax_j(s),  o[h,:] = sum_j p[h,j] * cache[j,:kv_lora]
 * Q is [H][kv_lora+rope] bf16 (per head q_lat | q_rope), cache is [>= n_rows][kv_lora+rope] bf16.
 * If `extra_row` >= 0 that cache row is attended as well (the row the step has just written; it is
 * merged in the combine so that the pass over the old rows need not wait for it).  Outputs:
 * o_bf16 [H][kv_lora] (may be NULL) and o_f32 [H][kv_lora] unrounded (may be NULL).
 * Supported: H = 128, kv_lora = 512, rope = 64 on the tensor-core path.  Workspace: see
 * nm_mla_attention_workspace_bytes.  The pass over the rows is a tcgen05 kernel split over the
 * sequence; a second kernel merges the splits with their log-sum-exp weights.
 */
size_t nm_mla_attention_workspace_bytes(int H, int n_rows, int kv_lora);
int nm_mla_attention(const void *Q, const void *kv_cache, void *o_bf16, float *o_f32, int H,
                     int n_rows, long extra_row, int kv_lora, int rope, float scale,
                     void *workspace, size_t workspace_bytes, nm_stream stream);
/* Two-phase form used by the decode step: the split pass, then the merge. */
int nm_mla_attention_partial(const void *Q, const void *kv_cache, int H, int n_rows, int kv_lora,
                             int rope, float scale, void *workspace, size_t workspace_bytes,
                             nm_stream stream);
int nm_mla_attention_combine(const void *Q, const void *kv_cache, void *o_bf16, float *o_f32, int H,
                             int n_rows, long extra_row, int kv_lora, int rope, float scale,
                             void *workspace, size_t workspace_bytes, nm_stream stream);

/*
 * One decode step for one token (DeepSeek-V3-style MLA, absorbed form).  Stages, each rounded to
 * bf16 as the paper rounds MatMul 2's output before RoPE / RMSNorm (Algorithm 2, output cast):
 *   c_q = h*W_DQ; c_qn = RMSNorm(c_q; gamma_q); q = c_qn*W_UQR ([H][nope+rope]);
 *   q_rope = RoPE(q[:, nope:], pos); q_lat[h] = q[h,:nope]*W_UK[h];
 *   ckr = h*(W_DKV|W_KR) (Eq. 3); cache[pos] = [RMSNorm(ckr[:kv_lora]; gamma_kv) | RoPE(ckr[kv_lora:], pos)];
 *   o_lat = attention([q_lat|q_rope], cache[0..seq_len)); o[h] = o_lat[h]*W_UV[h]; out = flatten(o)*W_O.
 * pos = seq_len - 1: seq_len counts the rows attended including the one this step writes.
 * Dense weights are K x N in `layout_dense`; W_UK is [H][nope][kv_lora], W_UV is [H][kv_lora][v],
 * row-major.  W_O may be NULL (the step then ends at o).  rope_cos_sin points at the table row for
 * pos (`rope` floats).  The narrow products of the KV chain run on `side` concurrently with the
 * tensor-core attention pass over the old rows on `main` (Data Independence condition); pass
 * side == main for a serial schedule.  Optional outputs (device, may be NULL) receive every
 * intermediate for stage-wise checking.  Workspace: nm_mla_workspace_bytes, counters cleared once
 * with nm_workspace_init.
 */
typedef struct {
    int d, q_lora, kv_lora, rope, nope, v, H;
    int seq_len;
    int layout_dense;              /* nm_layout of W_DQ, W_UQR, W_DKVKR, W_DQKV, W_O (NM_FRACTAL_NZ: single-token step only) */
    float rms_eps, softmax_scale;
    const void *h, *W_DQ, *gamma_q, *W_UQR, *W_DKVKR, *gamma_kv, *W_UK, *W_UV, *W_O;
    const float *rope_cos_sin;
    void *kv_cache;                /* [>= seq_len][kv_lora+rope] bf16; row seq_len-1 is written */
    void *out;                     /* [d] bf16 (ignored when W_O is NULL) */
    void *workspace;
    size_t workspace_bytes;
    /* optional intermediates, bf16 unless noted */
    void *c_q, *c_qn, *q, *q_full /* [H][kv_lora+rope] = q_lat | q_rope */, *ckr, *o_lat, *o;
    float *o_lat_f32;
    /* optional cudaEvent_t pair recorded on main_stream around the W_O product (for profiling) */
    void *event_before_wo, *event_after_wo;
    /* non-zero: the step's first product may start (and prefetch its weights) while the work enqueued
     * before the step on main_stream is still running - back-to-back layers or steps.  Only valid if
     * that earlier work writes none of this step's weights.  0 keeps the ordinary stream order. */
    int programmatic_entry;
    /* optional: the three down-projections stored as ONE row-major matrix [d][q_lora + kv_lora + rope] =
     * (W_DQ | W_DKV | W_KR), the paper's concatenation of Eq. 3 extended by W_DQ (all three multiply the
     * same h).  When given (and layout_dense is row-major or NM_FRACTAL_NZ) the step computes them as one product on
     * main_stream and needs no side stream; W_DQ and W_DKVKR are then ignored and may be NULL. */
    const void *W_DQKV;
} nm_mla_params;

size_t nm_mla_workspace_bytes(const nm_mla_params *p);

/* Small-batch decode: the same step for T independent sequences at once, one new token each (the paper's "larger
 * token" direction, Condition 5 of its last section, carried through the whole operator).  Every narrow product
 * takes the T tokens as its M rows, so the weights are streamed once for all of them; the vector stages and the
 * attention pass run per sequence inside shared launches.  Results are those of T single-token steps.
 *   T            1..16
 *   seq_lens     HOST array [T]: rows attended by sequence t including its new token (>= 1)
 *   h            device [T][d] bf16
 *   rope_cos_sin device [T][rope] fp32, row t for position seq_lens[t] - 1 (nm_rope_table)
 *   kv_cache     device bf16; sequence t owns rows [0, seq_lens[t]) at kv_cache + t * cache_stride elements,
 *                row width kv_lora + rope; row seq_lens[t] - 1 is written
 *   cache_stride elements between the caches of consecutive sequences (multiple of 8, >= seq_lens[t] * row width)
 *   out          device [T][d] bf16 (ignored when the params' W_O is NULL)
 *   q_full, o_lat, o   optional device outputs [T][H][kv_lora+rope], [T][H][kv_lora], [T][H][v] bf16
 *   c_q, c_qn, q, ckr  optional device outputs [T][q_lora], [T][q_lora], [T][H][nope+rope], [T][kv_lora+rope] bf16: the
 *                outputs of the down-projections, of the query latent's RMSNorm and of W_UQR, for stage-wise checking
 * From nm_mla_params it takes the dimensions, weights, rms_eps, softmax_scale, layout_dense, workspace,
 * workspace_bytes (>= nm_mla_batch_workspace_bytes(p, T)) and programmatic_entry (the first product may start under
 * the work enqueued before the call, as in the single-token step); its h, kv_cache, seq_len, rope_cos_sin, out and
 * intermediates are ignored.  Dimensions: kv_lora 512, rope 64, nope 128, v 128, H 128.  One stream; the kernels
 * are chained with programmatic dependent launch.  Errors as nm_mla_decode_step; nothing is enqueued on error
 * except as noted there. */
typedef struct nm_mla_batch {
    int T;
    const int *seq_lens;
    const void *h;
    const float *rope_cos_sin;
    void *kv_cache;
    long cache_stride;
    void *out;
    void *q_full, *o_lat, *o;
    void *c_q, *c_qn, *q, *ckr;
} nm_mla_batch;

size_t nm_mla_batch_workspace_bytes(const nm_mla_params *p, int T);
int nm_mla_decode_batch(const nm_mla_params *p, const nm_mla_batch *b, nm_stream main_stream);
int nm_mla_decode_step(const nm_mla_params *p, nm_stream main_stream, nm_stream side_stream);
/* The same step with the token and the result in HOST memory (pinned): h comes in on main_stream before the step (fetched by
 * a one-CTA kernel when the device can address h_host - the step's first product then starts under it -, else by a copy);
 * the result reaches out_host by stores of the last product when the device can address that memory (pinned or
 * registered, 16-byte aligned), otherwise by a copy after the step.  Either way it is complete when main_stream has
 * been synchronised.  h_staging / out_staging are device buffers of d bf16 each. */
int nm_mla_decode_step_host(const nm_mla_params *p, const void *h_host, void *out_host,
                            void *h_staging, void *out_staging, nm_stream main_stream, nm_stream side_stream);

/*
 * Programmatic dependent launch for nm_matmul / nm_matmul_batched (off by default).  When on,
 * a product may start streaming its weights while the previous kernel in the stream is still
 * running, and waits for that kernel only before it reads A or writes anything.  Turn it on only
 * when B is not written by the work that precedes the call in the stream (resident weights).
 */
int nm_set_programmatic_launch(int enable);

/*
 * Row-major bf16 products with M >= m and at least 32 MB of weights run on the tensor cores with the
 * operands swapped (weights as the MMA's M dimension, token rows as its N dimension): from M = 3 on
 * the CUDA-core path is bound by fp32 FMA issue rather than by HBM.  Products are exact and
 * accumulation is fp32 on both paths.  Default 3; pass 17 to keep every M on the CUDA cores (the
 * paper's placement), 1 to use the tensor cores from M = 1.
 */
int nm_set_tensor_core_min_m(int m);

/* Thread safety.  Calls that enqueue work may be made from several host threads (each on its own stream and
 * workspace).  The settings above (nm_set_workspace, nm_set_programmatic_launch, nm_set_tensor_core_min_m) and the
 * tuning aids of nm_debug.h are process-wide; they are guarded by a lock, and every call plans from one consistent
 * copy of them taken at its start, but a setting changed on one thread does apply to calls that start later on any
 * thread.  Per-device state (kernel attributes, the status word, the scratch of nm_matmul_static) is kept per device. */

#ifdef __cplusplus
}
#endif
#endif /* NM_H */
