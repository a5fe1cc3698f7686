// Latent attention pass on the tensor cores (tcgen05 + TMEM), one sequence split per CTA pair.
//
// For all 128 heads at once and a run of cache rows, tile by tile (32 rows; two tiles in flight):
//   S[128 x 32]   = Q[128 x 576] * tile^T      tcgen05.mma, both operands K-major in shared memory
//   P             = exp2(S*c - m)              fp32 in registers (one thread per head); written to TMEM as
//                                              two bf16 terms, P_hi = bf16(P) and P_lo = bf16(P - P_hi), so
//                                              that P*V keeps about 16 bits of P instead of 8
//   O[128 x 256] += P[128 x 32] * tile[:, half]  tcgen05.mma, A from TMEM, B = the same shared-memory
//                                                bytes read MN-major
// Q and the cache tile arrive by TMA (128-byte swizzle, every CTA its own copy) and are consumed in place by
// the MMA unit; the accumulators never leave TMEM until the split is finished.  The 512 output
// columns do not fit TMEM next to S, so two CTAs share a split, each owning 256 columns.  The running
// maximum is updated lazily: O is rescaled only when a row maximum grows by more than 2^8, so the
// usual tile costs no pass over the accumulator.  The cache tiles, S and P are double-buffered: while the
// softmax threads work on tile t, the tensor pipe computes the scores of tile t+1 and the P*V of tile
// t-1, and TMA fetches the next tile.
//
// The CTAs of kAttnCluster consecutive splits form a thread-block cluster and merge their results
// through distributed shared memory before anything goes to global memory: each CTA rescales its
// O rows to the cluster-wide maximum and parks them in its own shared memory (the Q buffer is free
// by then), then each CTA sums one quarter of the heads over all peers and writes that quarter.
// Global partial traffic and the work of the final merge (attn_combine_kernel) shrink by the
// cluster size.
//
// Roles: warp 0 lane 0 issues TMA, warp 1 owns TMEM and its lane 0 issues the MMAs, warps 2-5 hold
// one head per thread, warp 6 prefetches the weights of the products that follow into L2.  Every wait is bounded (mbar_wait); on expiry the CTA raises the status word,
// skips the remaining waits, frees its TMEM and returns.
#include "nm_async.cuh"
#include "nm_mla.cuh"
#include "nm_tcgen05.cuh"

namespace nm {

namespace {

constexpr int kHeads = 128;
constexpr int kDqk = 576;                 // 512 latent + 64 rope
constexpr int kDv = 512;
constexpr int kDvHalf = 256;
constexpr int kT = 32;                    // cache rows per pipeline stage (two stages in shared memory)
constexpr int kKVStages = 2;
constexpr int kKBlocks = kDqk / 64;       // 9 blocks of 64 elements (one 128-byte swizzle span)
constexpr int kQBlockBytes = kHeads * 128;   // 16 KB
constexpr int kKVBlockBytes = kT * 128;      // 8 KB
constexpr int kQBytes = kKBlocks * kQBlockBytes;     // 147456
constexpr int kKVBytes = kKBlocks * kKVBlockBytes;   // 36864 per stage
constexpr int kSmemBytes = kQBytes + kKVStages * kKVBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int kThreads = 224;               // TMA, MMA, 4 softmax warps, weight prefetch
constexpr uint32_t kTmemCols = 512;
// TMEM columns: O (fp32, 256), then per pipeline stage kSAcc score accumulators (fp32, 32 columns each; the 36
// k-steps of a tile's scores are dealt round-robin to them, because back-to-back MMAs into one narrow
// accumulator wait for each other, and the softmax threads add them up), then P_hi and P_lo (bf16 pairs, 16 each)
constexpr int kSAcc = 3;
constexpr uint32_t kColO = 0, kColS = 256, kColP = kColS + 2 * 32 * kSAcc, kColPlo = kColP + 32;   // stage b adds 32*kSAcc*b to S, 16*b to P_hi / P_lo
static_assert(kColPlo + 32 <= 512, "TMEM columns");
constexpr float kLazyThreshold = 8.0f;    // log2 units
constexpr int kCl = kAttnCluster;          // CTAs (splits) per cluster
constexpr int kHeadsPerRank = kHeads / kCl;

// Per-sequence arguments of one launch (blockIdx.z selects the sequence; a single-sequence call fills entry 0).
struct AttnSeqs {
    CUtensorMap kv[kMaxBatch];
    int n_rows[kMaxBatch];
    int rows_per_split[kMaxBatch];
    long ml_stride, o_stride;             // floats between the partials of consecutive sequences
};

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    __syncwarp();                                                  // the aligned forms want the warp converged
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in the peer CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_smem(uint32_t local_addr, uint32_t rank)
{
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_addr), "r"(rank));
    return a;
}
__device__ __forceinline__ float4 ld_peer_f4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));     // first source -> upper half
    return r;
}

// at most 120 registers per thread: leaves room on the SM for a CTA of the merge kernel that follows
__global__ void __maxnreg__(120)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ AttnSeqs seqs, AttnPartials part,
               float scale_log2, unsigned *status, unsigned long long *trace, const L2Prefetch pf)
{
    const int seq = blockIdx.z;
    const CUtensorMap *map_kv_p = &seqs.kv[seq];
    const int n_rows = seqs.n_rows[seq], rows_per_split = seqs.rows_per_split[seq];
    part.ml += (size_t)seq * seqs.ml_stride;
    part.O += (size_t)seq * seqs.o_stride;
    // Optional phase timestamps (ns) of CTA (0,0), for tuning: trace[i] is written when non-null.
#define NM_TRACE(i) do { if (trace && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) trace[i] = global_timer_ns(); } while (0)
    // ... and four stamps of every CTA (start, Q landed, last P*V done, end) from trace[32] on
#define NM_TRACE_CTA(i) do { if (trace && blockIdx.z == 0) trace[32 + 4 * (blockIdx.y * gridDim.x + blockIdx.x) + (i)] = global_timer_ns(); } while (0)
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;            // swizzle atoms want 1024-byte alignment
    unsigned char *smem = smem_raw + (base - raw_addr);
    const uint32_t q_addr = base, kv_addr = base + kQBytes;        // kv stage b at kv_addr + b * kKVBytes
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kQBytes + kKVStages * kKVBytes);
    // q: Q landed.  Per stage b: kv_full (tile landed), s_full (scores in TMEM), p_full (P written, 128
    // arrivals), pv_done (P*V of the tile finished: frees the cache stage and the P buffers).
    const uint32_t bar_q = smem_u32(bars + 0), bar_kv_full = smem_u32(bars + 1), bar_s_full = smem_u32(bars + 3),
                   bar_p_full = smem_u32(bars + 5), bar_pv_done = smem_u32(bars + 7);
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(8) float s_mlp[kCl][kHeadsPerRank][2];   // (m in log2 units, l) of the owned heads, written by each peer
    __shared__ float s_w[kCl][kHeadsPerRank];                     // weights of the slots in the final sum

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sp = blockIdx.x, half = blockIdx.y;
    const int r0 = sp * rows_per_split, r1 = min(n_rows, r0 + rows_per_split);
    const int ntiles = (r1 > r0) ? ceil_div(r1 - r0, kT) : 0;      // 0 for the padding CTAs of the last cluster

    if (tid == 0) {
        NM_TRACE(0);
        NM_TRACE_CTA(0);
        s_abort = 0;
        mbar_init(bar_q, 1);
        for (int b = 0; b < kKVStages; ++b) {
            mbar_init(bar_kv_full + 8 * b, 1); mbar_init(bar_s_full + 8 * b, 1);
            mbar_init(bar_p_full + 8 * b, 128); mbar_init(bar_pv_done + 8 * b, 1);
        }
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(&s_tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    // First half of a cluster barrier: by the time its second half is waited for (before the merge) every
    // peer has started, which is what writing into a peer's shared memory requires.
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    pdl_launch_dependents();
    const uint32_t rank = cluster_rank();
    const int cluster_id = sp / kCl;
    float m_own = -INFINITY, l_own = 0.f;                         // softmax threads: this split's (m, l)

    // A warp of its own, once the first cache tile has landed (so that the loads the whole pass waits for
    // do not queue behind it), pulls the weights of the products that follow the attention - W_UV and the
    // head of every k-split of W_O - into L2 in 8 KB bulk prefetches: the pass needs little HBM bandwidth,
    // and those weights do not depend on its result.  The prefetch instruction stalls its thread while the
    // request queue is full (microseconds here), which is why no thread of the pipeline issues it.
    auto prefetch_weights = [&]() {
        constexpr long kChunk = 8192;
        const long block_chunks = (pf.block_bytes + kChunk - 1) / kChunk;
        const long chunks_per_range = (pf.range_bytes + kChunk - 1) / kChunk;
        const long total = block_chunks + chunks_per_range * pf.nranges;
        const long nthreads = (long)gridDim.x * gridDim.y * gridDim.z * 32;
        const long me = (((long)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) * 32 + lane;
        for (long i = me; i < total; i += nthreads) {
            const char *ptr;
            long n;
            if (i < block_chunks) {
                ptr = pf.block + i * kChunk;
                n = min(kChunk, pf.block_bytes - i * kChunk);
            } else {
                const long j = i - block_chunks, r = j / chunks_per_range, off = (j - r * chunks_per_range) * kChunk;
                ptr = pf.base + r * pf.range_stride + off;
                n = min(kChunk, pf.range_bytes - off);
            }
            n &= ~15L;
            if (n > 0) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ptr), "r"((uint32_t)n) : "memory");
        }
    };

    if (warp == 0) {
        // ---------------- TMA producer --------------------------------------------------------------
        if (lane == 0) {
            tma_prefetch_descriptor(&map_q);
            tma_prefetch_descriptor(map_kv_p);
            const uint64_t keep = l2_policy_evict_last(), stream = l2_policy_evict_first();
            auto load_tile = [&](int t) {
                const int b = t & 1;
                mbar_arrive_expect_tx(bar_kv_full + 8 * b, kKVBytes);
                for (int c = 0; c < kKBlocks; ++c)
                    tma_load_2d(kv_addr + b * kKVBytes + c * kKVBlockBytes, map_kv_p, c * 64, r0 + t * kT, bar_kv_full + 8 * b, stream);
            };
            // The cache rows were written by earlier steps, not by the kernels just before this one:
            // fetch the first two tiles before waiting for those kernels, then fetch Q, which they produce.
            for (int t = 0; t < min(ntiles, kKVStages); ++t) load_tile(t);
            // Only two tiles fit in shared memory, far too few to cover the HBM latency of a tile that
            // takes under a microsecond to consume: the rest of this split's rows are pulled into L2 now
            // (a few hundred KB), so that every later tile load is an L2 hit.
            if (half == 0)
                for (int t = kKVStages; t < ntiles; ++t)
                    for (int c = 0; c < kKBlocks; ++c) tma_prefetch_l2_2d(map_kv_p, c * 64, r0 + t * kT);
            pdl_wait_prior_grids();
            if (ntiles > 0) {                                      // a padding CTA of the last cluster loads nothing
                mbar_arrive_expect_tx(bar_q, kQBytes);
                for (int c = 0; c < kKBlocks; ++c) tma_load_2d(q_addr + c * kQBlockBytes, &map_q, c * 64, seq * kHeads, bar_q, keep);
            }
            for (int t = kKVStages; t < ntiles; ++t) {             // stage b is free once the P*V of tile t-2 is done
                const uint32_t bar = bar_pv_done + 8 * (t & 1), par = ((t - kKVStages) >> 1) & 1;
                if (!mbar_try_wait(bar, par) && !mbar_wait(bar, par, &s_abort, status)) break;
                load_tile(t);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ---------------------------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(128, kT, false, false), idesc_o = instr_desc(128, kDvHalf, false, true);
            // The descriptors of a tile's 36 k-steps differ only in the start-address field (16-byte units, no
            // carry out of it for addresses below 256 KB): one base each, compile-time offsets added per step.
            const uint64_t q_desc0 = smem_desc(q_addr, 16, 1024), kv_desc0 = smem_desc(kv_addr, 16, 1024);
            auto scores = [&](int t) {                             // S[t&1] = Q * tile(t)^T  (tile t has landed)
                const int b = t & 1;
                const uint64_t kv_desc = kv_desc0 + (uint64_t)((b * kKVBytes) >> 4);
                const uint32_t s_col = tmem + kColS + 32 * kSAcc * b;
                tc_fence_after();
#pragma unroll
                for (int step = 0; step < kKBlocks * 4; ++step) {
                    const int c = step >> 2, kk = step & 3;
                    mma_ss(s_col + 32 * (step % kSAcc), q_desc0 + (uint64_t)((c * kQBlockBytes + kk * 32) >> 4),
                           kv_desc + (uint64_t)((c * kKVBlockBytes + kk * 32) >> 4), idesc_s, step >= kSAcc);
                }
                mma_commit(bar_s_full + 8 * b);
            };
            // Scores of tiles 0 and 1 together (both landed, both S buffers free): each k-step's slice of Q is
            // read from shared memory once and used for both tiles - the Q operand is what these MMAs cost.
            auto scores_pair = [&]() {
                tc_fence_after();
#pragma unroll
                for (int step = 0; step < kKBlocks * 4; ++step) {
                    const int c = step >> 2, kk = step & 3;
                    const uint64_t qd = q_desc0 + (uint64_t)((c * kQBlockBytes + kk * 32) >> 4);
                    const uint64_t kd = kv_desc0 + (uint64_t)((c * kKVBlockBytes + kk * 32) >> 4);
                    mma_ss_a_fill(tmem + kColS + 32 * (step % kSAcc), qd, kd, idesc_s, step >= kSAcc);
                    mma_ss_a_lastuse(tmem + kColS + 32 * kSAcc + 32 * (step % kSAcc), qd, kd + (uint64_t)(kKVBytes >> 4), idesc_s, step >= kSAcc);
                }
                mma_commit(bar_s_full);
                mma_commit(bar_s_full + 8);
            };
            auto pv = [&](int t) {                                 // O += P[t&1] * tile(t)[:, half]  (P of tile t is written)
                const int b = t & 1;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kT / 16; ++kk) {
                    const uint64_t vdesc = smem_desc(kv_addr + b * kKVBytes + (4 * half) * kKVBlockBytes + kk * 2048, kKVBlockBytes, 1024);
                    mma_ts(tmem + kColO, tmem + kColP + 16 * b + kk * 8, vdesc, idesc_o, (t | kk) != 0);
                    mma_ts(tmem + kColO, tmem + kColPlo + 16 * b + kk * 8, vdesc, idesc_o, true);
                }
                mma_commit(bar_pv_done + 8 * b);
            };
            NM_TRACE(1);
            if (ntiles > 0) mbar_wait(bar_q, 0, &s_abort, status);
            NM_TRACE(2);
            NM_TRACE_CTA(1);
            // Two independent streams of work share this thread: scores of tile ts (needs the tile in
            // shared memory and S[ts&1] free, i.e. the P*V of tile ts-2 issued) and P*V of tile tp (needs
            // the softmax of tile tp).  Whichever is ready is issued; neither blocks the other.
            int ts = 0, tp = 0;
            uint64_t idle_since = 0;
            while (tp < ntiles) {
                bool progress = false;
                if (ts == 0 && ntiles >= 2 && mbar_try_wait(bar_kv_full, 0) && mbar_try_wait(bar_kv_full + 8, 0)) {
                    NM_TRACE(12);
                    scores_pair();
                    NM_TRACE(3);
                    NM_TRACE(13);
                    ts = 2;
                    progress = true;
                } else if (ts < ntiles && ts <= tp + 1 && mbar_try_wait(bar_kv_full + 8 * (ts & 1), (ts >> 1) & 1)) {
                    if (ts == 0) NM_TRACE(12);
                    scores(ts);
                    if (ts == 0) NM_TRACE(3);
                    if (ts == 1) NM_TRACE(13);
                    ++ts;
                    progress = true;
                }
                if (mbar_try_wait(bar_p_full + 8 * (tp & 1), (tp >> 1) & 1)) {
                    pv(tp);
                    ++tp;
                    progress = true;
                }
                if (progress) {
                    idle_since = 0;
                } else {                                           // bounded: give up after about a second without progress
                    if (s_abort) break;
                    const uint64_t now = global_timer_ns();
                    if (idle_since == 0) idle_since = now;
                    else if (now - idle_since > kWaitLimitNs) {
                        s_abort = 1;
                        if (status) atomicOr(status, kStatusWaitExpired);
                        break;
                    }
                }
            }
        }
    } else if (warp == 6) {
        // ---------------- weight prefetch ----------------------------------------------------------------
        if (ntiles > 0) {                                          // sleep-poll: this warp must not take issue slots from the pipeline
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(bar_kv_full, 0)) {
                __nanosleep(128);
                if (s_abort || global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
        prefetch_weights();
    } else {
        // ---------------- one head per thread: softmax, lazy rescale ------------------------------------------
        const int quad = warp & 3;                                 // TMEM lanes this warp may touch
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        float m_used = -INFINITY, l = 0.f;
        for (int t = 0; t < ntiles; ++t) {
            const int b = t & 1;
            mbar_wait(bar_s_full + 8 * b, (t >> 1) & 1, &s_abort, status);
            tc_fence_after();
            if (t == 0 && tid == 64) NM_TRACE(4);
            if (t == 1 && tid == 64) NM_TRACE(14);
            uint32_t sr[32];
            tmem_ld32(lane_base + kColS + 32 * kSAcc * b, sr);
            if (kSAcc > 1) {
                uint32_t s1[32], s2[32];
                tmem_ld32(lane_base + kColS + 32 * kSAcc * b + 32, s1);
                if (kSAcc > 2) tmem_ld32(lane_base + kColS + 32 * kSAcc * b + 64, s2);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < kT; ++j) {
                    float v = __uint_as_float(sr[j]) + __uint_as_float(s1[j]);
                    if (kSAcc > 2) v += __uint_as_float(s2[j]);
                    sr[j] = __float_as_uint(v);
                }
            } else {
                tmem_wait_ld();
            }
            const int valid = min(kT, r1 - (r0 + t * kT));
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < kT; ++j)
                if (j < valid) mx = fmaxf(mx, __uint_as_float(sr[j]));
            const float mx2 = mx * scale_log2;
            const bool grow = (t == 0) || (mx2 > m_used + kLazyThreshold);
            // P[b] was last read by the P*V of tile t-2
            if (t >= kKVStages) {
                mbar_wait(bar_pv_done + 8 * b, ((t - kKVStages) >> 1) & 1, &s_abort, status);
                tc_fence_after();
            }
            if (t > 0 && __any_sync(0xffffffffu, grow)) {
                // rare: the maximum grew by more than 2^8.  O may only be touched between two P*V passes.
                mbar_wait(bar_pv_done + 8 * ((t - 1) & 1), ((t - 1) >> 1) & 1, &s_abort, status);
                tc_fence_after();
                const float f = grow ? fast_exp2(m_used - mx2) : 1.0f;
                for (int c = 0; c < kDvHalf / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld32(lane_base + kColO + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tmem_st32(lane_base + kColO + c * 32, o);
                }
                tmem_wait_st();
                if (grow) l *= f;
            }
            if (grow) m_used = mx2;
            uint32_t pr[16], plo[16];
            float lsum = 0.f;
#pragma unroll
            for (int j = 0; j < kT; j += 2) {
                const float p0 = (j < valid) ? fast_exp2(fmaf(__uint_as_float(sr[j]), scale_log2, -m_used)) : 0.f;
                const float p1 = (j + 1 < valid) ? fast_exp2(fmaf(__uint_as_float(sr[j + 1]), scale_log2, -m_used)) : 0.f;
                lsum += p0 + p1;
                const uint32_t hi = pack_bf16x2(p0, p1);
                pr[j >> 1] = hi;
                plo[j >> 1] = pack_bf16x2(p0 - __uint_as_float(hi << 16), p1 - __uint_as_float(hi & 0xffff0000u));
            }
            l += lsum;
            tmem_st16(lane_base + kColP + 16 * b, pr);
            tmem_st16(lane_base + kColPlo + 16 * b, plo);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p_full + 8 * b);
            if (t == 0 && tid == 64) NM_TRACE(5);
            if (t == 1 && tid == 64) NM_TRACE(15);
        }
        // the last P*V must have landed before O is read
        if (ntiles > 0) {
            mbar_wait(bar_pv_done + 8 * ((ntiles - 1) & 1), ((ntiles - 1) >> 1) & 1, &s_abort, status);
            tc_fence_after();
        }
        if (tid == 64) NM_TRACE(6);
        if (tid == 64) NM_TRACE_CTA(2);
        m_own = m_used; l_own = l;
    }

    // ---- merge of the cluster's splits through distributed shared memory -----------------------------------
    // Each CTA parks its (unscaled) O rows and its (m, l) in its own shared memory as soon as its last
    // P*V is done (the Q tile is free by then; layout [head][64 float4], the float4 index XOR-ed with
    // (head & 7) so that neither the row-per-thread writes nor the row-contiguous reads conflict).
    // Its (m, l) pairs it pushes to the peers that own the heads.
    // After one cluster barrier, rank r combines heads [32r, 32r+32) over all peers - weights
    // 2^(m_peer - max m) - reading the peers' rows with many loads in flight, and writes one partial
    // per cluster.  A last barrier keeps every CTA's shared memory alive until its peers have read it.
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");       // all peers are running (they arrived at kernel start)
    if (warp >= 2 && warp < 6) {
        const int quad = warp & 3, head = quad * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        // (m, l) goes straight into the shared memory of the peer that owns the head: after the barrier the
        // owner finds all four pairs locally
        const uint32_t slot = peer_smem(smem_u32(&s_mlp[rank][head % kHeadsPerRank][0]), (uint32_t)head / kHeadsPerRank);
        asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(slot), "f"((ntiles > 0) ? m_own : -INFINITY), "f"(l_own) : "memory");
        if (ntiles > 0) {
            for (int c = 0; c < kDvHalf / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(lane_base + kColO + c * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    const uint32_t q4 = (uint32_t)(c * 8 + i / 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(q_addr + (uint32_t)(head * 64 + (q4 ^ (head & 7u))) * 16u),
                                 "r"(o[i]), "r"(o[i + 1]), "r"(o[i + 2]), "r"(o[i + 3]) : "memory");
                }
            }
        }
        if (tid == 64) NM_TRACE(7);
    }
    cluster_sync_all();                                            // every peer's rows and (m, l) are parked
    if (tid == 64) NM_TRACE(8);
    if (warp >= 2 && warp < 6) {
        const int t = tid - 64;                                    // 0..127
        if (t < kCl * kHeadsPerRank) {                             // weight of peer r for owned head hl
            const int hl = t % kHeadsPerRank, r = t / kHeadsPerRank, head = (int)rank * kHeadsPerRank + hl;
            float pm[kCl], pl[kCl], M = -INFINITY;
#pragma unroll
            for (int rr = 0; rr < kCl; ++rr) {
                pm[rr] = s_mlp[rr][hl][0]; pl[rr] = s_mlp[rr][hl][1];
                M = fmaxf(M, pm[rr]);
            }
            s_w[r][hl] = (pm[r] == -INFINITY) ? 0.f : fast_exp2(pm[r] - M);
            if (r == 0 && half == 0) {
                float Ltot = 0.f;
#pragma unroll
                for (int rr = 0; rr < kCl; ++rr) Ltot = fmaf(pm[rr] == -INFINITY ? 0.f : fast_exp2(pm[rr] - M), pl[rr], Ltot);
                part.ml[((size_t)cluster_id * kHeads + head) * 2] = M * 0.6931471805599453f;     // natural-log units
                part.ml[((size_t)cluster_id * kHeads + head) * 2 + 1] = Ltot;
            }
        }
        named_barrier_sync(1, 128);
        if (tid == 64) NM_TRACE(9);
        constexpr int kIters = kHeadsPerRank * 64 / 128, kBatch = 4;
        for (int i0 = 0; i0 < kIters; i0 += kBatch) {
            float4 v[kBatch][kCl];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {                     // kBatch * kCl remote loads in flight
                const int idx = t + 128 * (i0 + b);
                const int hl = idx / 64, q4 = idx % 64, head = (int)rank * kHeadsPerRank + hl;
                const uint32_t local = q_addr + (uint32_t)(head * 64 + (q4 ^ (head & 7))) * 16u;
#pragma unroll
                for (int r = 0; r < kCl; ++r)
                    v[b][r] = (s_w[r][hl] != 0.f) ? ld_peer_f4(peer_smem(local, r)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int idx = t + 128 * (i0 + b);
                const int hl = idx / 64, q4 = idx % 64, head = (int)rank * kHeadsPerRank + hl;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < kCl; ++r) {                    // rank order: deterministic
                    const float w = s_w[r][hl];
                    acc.x = fmaf(w, v[b][r].x, acc.x); acc.y = fmaf(w, v[b][r].y, acc.y);
                    acc.z = fmaf(w, v[b][r].z, acc.z); acc.w = fmaf(w, v[b][r].w, acc.w);
                }
                *reinterpret_cast<float4 *>(part.O + ((size_t)cluster_id * kHeads + head) * kDv + half * kDvHalf + q4 * 4) = acc;
            }
        }
    }
    if (tid == 64) NM_TRACE(10);
    cluster_sync_all();                                            // peers are done reading this CTA's shared memory

    // ---- teardown: TMEM goes back ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (s_abort && tid == 0) {
        // a wait expired: give copies already issued a bounded chance to land before the CTA exits
        for (int i = 0; i < (1 << 16) && ntiles > 0 && !mbar_try_wait(bar_q, 0); ++i) {}
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (tid == 0) NM_TRACE(11);
    if (tid == 0) NM_TRACE_CTA(3);
#undef NM_TRACE
#undef NM_TRACE_CTA
}

// Tensor maps: bf16 [rows][576], boxes of 64 columns (128 bytes, the swizzle span) x box_rows rows.
bool encode_rows_map(CUtensorMap *map, const void *ptr, int rows, int box_rows)
{
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)kDqk, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kDqk * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

static std::atomic<unsigned long long *> g_attn_trace{nullptr};
void set_attention_trace(unsigned long long *p) { g_attn_trace.store(p, std::memory_order_relaxed); }
unsigned long long *attention_trace() { return g_attn_trace.load(std::memory_order_relaxed); }

static int launch_attn_tc(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split, int nsplit,
                          AttnPartials part, long ml_stride, long o_stride, float scale, cudaStream_t stream, bool programmatic_launch,
                          L2Prefetch prefetch)
{
    if (nseq < 1 || nseq > kMaxBatch || nsplit < 1) return NM_ERR_UNSUPPORTED;
    if ((uintptr_t)Q & 15u) return NM_ERR_UNSUPPORTED;
    CUtensorMap map_q;
    AttnSeqs seqs{};
    seqs.ml_stride = ml_stride; seqs.o_stride = o_stride;
    if (!encode_rows_map(&map_q, Q, nseq * kHeads, kHeads)) return NM_ERR_UNSUPPORTED;
    for (int t = 0; t < nseq; ++t) {
        seqs.n_rows[t] = n_rows[t];
        seqs.rows_per_split[t] = rows_per_split[t];
        if (n_rows[t] < 1) {                                       // nothing to attend: its CTAs find no tiles and load nothing
            seqs.kv[t] = map_q;
            seqs.rows_per_split[t] = kT;
            continue;
        }
        if ((uintptr_t)caches[t] & 15u) return NM_ERR_UNSUPPORTED;
        // The cache map covers exactly the rows attended: rows past n_rows read as zeros (and are masked),
        // whatever the rest of the buffer holds.
        if (!encode_rows_map(&seqs.kv[t], caches[t], n_rows[t], kT)) return NM_ERR_UNSUPPORTED;
    }
    static std::atomic<unsigned long long> configured{0};          // one bit per device
    {
        cudaError_t e = ensure_dynamic_smem(attn_tc_kernel, kSmemBytes, configured);
        if (e != cudaSuccess) return record_cuda_error(e, "attention kernel attribute");
    }
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(nsplit, kCl) * kCl, 2, nseq);      // padded to whole clusters; padding CTAs have no rows
    // the prefetch warp is launched only when there is something to prefetch (fewer registers held on the SM)
    const bool has_prefetch = prefetch.block_bytes > 0 || (prefetch.nranges > 0 && prefetch.range_bytes > 0);
    cfg.blockDim = dim3(has_prefetch ? kThreads : kThreads - 32);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic_launch ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_tc_kernel, map_q, seqs, part, scale_log2, device_status_ptr(), attention_trace(), prefetch);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention (tensor cores) launch");
}

int attention_partial_tc(const void *Q, const void *cache, AttnPartials part, AttnPlan plan, int n_rows, float scale,
                         cudaStream_t stream, bool programmatic_launch, L2Prefetch prefetch)
{
    if (n_rows < 1 || plan.nsplit < 1) return NM_ERR_UNSUPPORTED;
    return launch_attn_tc(Q, 1, &cache, &n_rows, &plan.rows_per_split, plan.nsplit, part, 0, 0, scale, stream, programmatic_launch, prefetch);
}

int attention_partial_tc_batch(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split,
                               int nsplit, AttnPartials part, int slot_stride, float scale, cudaStream_t stream,
                               bool programmatic_launch, L2Prefetch prefetch)
{
    return launch_attn_tc(Q, nseq, caches, n_rows, rows_per_split, nsplit, part, (long)slot_stride * kHeads * 2,
                          (long)slot_stride * kHeads * kDv, scale, stream, programmatic_launch, prefetch);
}

}  // namespace nm
