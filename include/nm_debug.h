/*
 * nm_debug.h - tuning aids and test hooks of the nm library (sweeps, forced plans, traces, the bounded-wait probe).
 * Not needed for normal use; include/nm.h is the boundary proper.  All settings here are process-wide, guarded by a
 * lock, and read once per call (see "Thread safety" in nm.h).  The paper has no counterpart for any of these.
 *
 * Environment (read once, when the library is loaded): NM_LOG=1 prints the plan of every product (kernel family, tile
 * width, k-splits, ring depth) to stderr; NM_FORCE_KERNEL, NM_STAGES, NM_TILE_N and NM_SPLITK give nm_debug_set_kernel /
 * nm_debug_set_plan their initial values.
 */
#ifndef NM_DEBUG_H
#define NM_DEBUG_H

#include "nm.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Override the tiling heuristic: columns per CTA tile of the row-major kernel and number of
 * k-splits; 0 restores the heuristic.  Values are clamped to what the workspace bound covers. */
int nm_debug_set_plan(int tile_n, int nsplit);
/* Force the kernel family for row-major bf16 weights (-1 heuristic; 0 plain-load kernel; 3 TMA-ring
 * CUDA-core kernel; 4 swap-AB tensor-core kernel) and the ring depth in stages (0 heuristic). */
int nm_debug_set_kernel(int kind, int stages);
/* Split-K of the CUDA-core kernels: 1 (default) lets the k-splits of a column tile form a thread-block cluster whose
 * partial sums meet in the first CTA's shared memory (up to 8 splits; partial tiles up to 16 KB in the TMA-ring
 * kernel, 8 KB in the plain kernels); 0 always goes through the workspace (partial tiles, arrival counter, gather). */
int nm_debug_set_cluster_split(int enable);
/* Tuning aid: phase timestamps (ns, %globaltimer) of the decode step's kernels go to `device_buffer` (8192
 * unsigned 64-bit values) when non-null: [0,32) phases of CTA (0,0) of the attention kernel (the 64-head kernel:
 * from 4 four per cache tile - scores issued, scores seen, P written, P*V issued - for five tiles, from 24 five phases
 * of the cluster merge); from 32 four per
 * attention CTA (start, Q landed, last P*V done, end); from 1100 eight phases of two CTAs of the merge + W_UV
 * kernel; from 2048 / 4096 / 6144 four per CTA (start, inputs ready, loop done, end) of the down-projection, W_UQR
 * and W_O products; from 2688 four phases of the CTA that completes a product carrying vector stages (last arrival,
 * gather done, synchronised, sums reduced).  NULL = off. */
int nm_debug_set_attention_trace(void *device_buffer);
/* Decode step tuning: launch the merge + W_UV kernel programmatically (default 1); include W_UV in the L2
 * prefetch (default 1). */
int nm_debug_set_step_knobs(int uv_programmatic, int prefetch_w_uv);
/* Decode step, the vector stages behind the down-projections (RMSNorm / RoPE / the cache-row write): 0 as kernels of
 * their own; 1 (default) folded into the products - with the three down-projections stored as one matrix the k-splits
 * meet inside clusters, W_UQR normalises its token row while loading it and the KV consumers ride in an extra CTA of
 * the per-head query kernel; otherwise, and with 2 always, the CTA that completes the product's last tile runs them. */
int nm_debug_set_step_tails(int enable);
/* Batch decode: sequences from which the per-head products (W_UK, W_UV) run as batched products of the library with
 * RoPE and the merge as kernels of their own (default 3); below, fused per-head kernels do them.  17 = always fused. */
int nm_debug_set_batch_per_head_min_tokens(int tokens);
/* Decode step tuning: force (tile_n, nsplit, ring stages) of one of its products - which = 0 the down-projection,
 * 1 W_UQR, 2 W_O; zeros give the plan back to the planner. */
int nm_debug_set_step_plan(int which, int tile_n, int nsplit, int stages);
/* Decode step: 1 (default) runs RoPE + W_UK and attention-merge + W_UV as fused per-head kernels, 0 as
 * separate kernels (rope, batched product, merge, batched product). */
int nm_debug_set_step_fusion(int enable);
/* Decode step: MB of W_O prefetched into L2 while the attention pass runs (default 40, 0 = off). */
int nm_debug_set_step_prefetch(int megabytes);
/* Decode step: chain its kernels with programmatic dependent launch (default 1) or not (0). */
int nm_debug_set_step_pdl(int enable);
/* Attention pass: 0 (default) the wide-tile tensor-core kernel when the shape allows (single-token step and stand-alone
 * attention; the batch step keeps the older kernels: 64 heads per CTA below 65536 cache rows in the call, 128 heads per
 * CTA from there on); 1 CUDA-core kernel; 2 / 3 the older tensor-core kernels with 128 / 64 heads per CTA whatever the
 * length; 4 the wide-tile kernel. */
int nm_debug_set_attention(int impl);
/* Wide-tile attention kernel: force the cache rows per tile (64, 128, 256), the most row runs (1..64) and the number of
 * runs merged on chip (cluster of 1, 2 or 4); zeros give each choice back to the planner. */
int nm_debug_set_attention_wide(int tile_rows, int max_runs, int cluster);
/* Two-stream schedule of nm_mla_decode_step (W_DQ and W_DKV|W_KR stored apart, side_stream != main_stream): 0 (default) the
 * KV chain - the paper's MatMul 2 with RMSNorm, RoPE and the cache-row write - is forked at the start of the step and runs
 * beside the first product of the Q chain; 1 it is forked once the attention operand is ready and runs, a narrow
 * CUDA-core product, beside the tensor-core attention pass over the old cache rows (Data Independence condition: the new
 * row is only needed by the merge). */
int nm_debug_set_step_kv_beside_attention(int enable);
/* The debug build.  `python paper_2609_16009_b200/build.py --check` compiles the same sources with -DNM_BOUNDS_CHECK into
 * libnm_check.so: every hand-indexed global access of the narrow-product kernels (the CUDA-core row / column / scalar
 * kernels, the split-K gather, the token loads and the C / partial stores of the TMA ring and tensor-core kernels) is
 * checked against the extent of the operand it belongs to; an access outside raises a bit in the device status word
 * (nm_check_status returns NM_ERR_BOUNDS) and is skipped - loads yield zero, stores do nothing, nothing faults.  The paper
 * has no counterpart; it stands in for a memory checker on machines where none can be run.
 * nm_debug_bounds_checked: 1 in that build, 0 in the normal one.  nm_debug_bounds_selftest (debug build only, else
 * NM_ERR_UNSUPPORTED): `buf` is a device buffer of `bytes` bytes (>= 32, a multiple of 8, 4-byte aligned); one thread
 * stores to and loads from the first word of its second half while naming its first half as the operand - the store must
 * not happen, out_loaded[0] (device, two words) must be 0 - and then does the same inside the first half (buf[0] becomes
 * 0x600df00d, out_loaded[1] likewise); nm_check_status then reports NM_ERR_BOUNDS once. */
int nm_debug_bounds_checked(void);
int nm_debug_bounds_selftest(void *buf, size_t bytes, unsigned *out_loaded, nm_stream stream);
/* Measurement aid: a kernel that only reads `bytes` bytes of device memory once (16-byte streaming loads, the
 * products' own load instruction, ctas_per_sm x SM-count CTAs of 256 threads) - the read-only bandwidth this GPU
 * delivers, to set beside the copy bandwidth the roofline uses.  src 16-byte aligned; sink4: 4 writable bytes. */
int nm_debug_stream_read(const void *src, size_t bytes, void *sink4, int ctas_per_sm, nm_stream stream);
/* Report the plan for a problem: out[0..5] = kernel kind (0 row-major vector, 1 column-major
 * vector, 2 scalar), columns per tile, k-splits, k-rows per split, column tiles, CTAs. */
int nm_debug_get_plan(int M, int N, int K, int H, nm_dtype dtype, nm_layout layout_B, int vec_ok,
                      int *out /* host, 6 ints */);


/* Test hook for the bounded device-side waits (the only way a kernel of this library can stall is a wait on an
 * mbarrier; Algorithm 1's gather stage has the same hazard in its device-wide barrier).  Launches one CTA that waits
 * on an mbarrier nobody arrives at, with the wait limit set to `limit_ns` (1 us .. 1 s) for this launch only; the wait
 * expires, the kernel raises the status word and returns by itself - no trap, no fault.  nm_check_status(stream)
 * then reports NM_ERR_TIMEOUT once.  elapsed_ns (device, 2 x uint64, may be NULL) receives the time the waits took
 * and a bit mask of waits that reported success (expected 0). */
int nm_debug_wait_probe(unsigned long long limit_ns, unsigned long long *elapsed_ns, nm_stream stream);

/* Measurement aid: clocks of `reps` back-to-back tcgen05.mma (kind::f16, bf16, K = 16) of shape m x n issued by one
 * thread of one CTA, with the A operand in shared memory (K-major) or in TMEM and the B operand in shared memory K-major
 * or MN-major, into n_acc accumulators used in turn; consecutive MMAs step the operand addresses by the given bytes
 * (cycling over four positions).  out_clocks (device, 3 x uint64): clocks until the commit arrived, clocks until the last
 * MMA was issued, 1 if the wait succeeded.  m 64 or 128; n a multiple of 16 up to 256; n_acc * n <= 448. */
int nm_debug_mma_probe(int m, int n, int a_from_tmem, int b_mn_major, int reps, int n_acc, int a_step_bytes, int b_step_bytes,
                       unsigned long long *out_clocks, nm_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* NM_DEBUG_H */
