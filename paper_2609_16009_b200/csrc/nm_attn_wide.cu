// Latent attention pass on the tensor cores with WIDE score tiles: all 128 heads per CTA, up to 256 cache rows per
// tcgen05.mma.
//
// What a tcgen05.mma costs here (nm_debug_mma_probe, bf16, K = 16, one issuing thread, back to back): max(50, N / 2)
// clocks - whatever M (64 or 128), whichever operand comes from TMEM, K-major or MN-major B.  So M = 128 is the only
// shape that uses the whole tensor pipe (M = 64 takes the same time for half the work), an MMA over fewer than 100
// cache rows pays the 50-clock floor (the 32-row scores MMAs of nm_attn_tc.cu run at a sixth of the rate, the 64-row
// ones of nm_attn_tc64.cu at a third, on half the heads), and the scores S = Q * tile^T want all 128 heads and as
// many cache rows per instruction as TMEM has columns for: up to 256 here.  With the MMAs that cheap, what bounds the
// pass is the traffic from L2 into shared memory - Q (147 KB) once per CTA, every cache row once per column half
// and once more for P * V - and the exponentials.
//
// Per CTA: one run of cache rows x one half of the 512 output columns x all 128 heads (O[128 x 256] fp32 is half of
// TMEM; the other half holds S[128 x R], R = 64, 128 or 256 rows per tile).  Nothing is resident in shared memory:
// with one tile per CTA (the usual case) every 64-column block of Q is used exactly once, so Q streams through the
// same ring as the cache rows - 192 KB of stages, all of it in flight, because a stage that is refilled only after
// its MMAs are done makes the loop a chain of L2 round trips.  Per tile:
//   scores   nine stages [Q block 128 heads x 64 columns | K block R rows x 64 columns] (128-byte swizzle, K-major
//            operands), four MMAs M128 N=R K16 each
//   P * V    R/64 stages with a V slab [64 rows x 256 columns of this CTA's half] (the same bytes read MN-major), per
//            slab four k-steps x two bf16 terms of P (hi + lo, about 16 bits of P) = eight MMAs M128 N256 K16, A from TMEM
// The second read of a row comes from L2.  The softmax of a head: a first pass over S for the row
// maximum (updated lazily: O is rescaled only when a maximum grows by more than 2^8), a second pass that writes P
// over the very columns of S it has just read, 16 rows at a time (hi in the first 8 columns, lo in the next 8),
// and signals every 64 rows so that P * V of the first slab runs while the rest of the tile is still in the
// exponentials.  One thread per head (kSets = 1; with two, the head's threads alternate over the 32-row chunks and
// exchange maxima and sums through shared memory - measured slower per step, 84.0 against 82.7 us at 16384 rows, although
// the exponentials go faster).  A run on its own leaves as one partial by tiled TMA stores; the CTAs of a cluster (2 or 4
// row runs) merge their results through distributed shared memory first, as in the older kernels.  Every wait is bounded
// (mbar_wait); on expiry the CTA raises the status word, skips the remaining waits, frees its TMEM and returns.
#include "nm_async.cuh"
#include "nm_mla.cuh"
#include "nm_tcgen05.cuh"

namespace nm {

namespace {

constexpr int kHeads = 128;
constexpr int kDqk = 576;                 // 512 latent + 64 rope
constexpr int kDv = 512;
constexpr int kDvHalf = 256;
constexpr int kKBlocks = kDqk / 64;       // 9 blocks of 64 elements (one 128-byte swizzle span)
constexpr int kQBlockBytes = kHeads * 128;            // 16 KB
constexpr int kRingBytes = 196608;                    // all stages together
constexpr int kSlabRows = 64;                         // cache rows per V slab
constexpr int kSlabBytes = 32768;                     // [64 rows x 256 columns]
constexpr int kSubBlockBytes = kSlabRows * 128;       // one [64 rows x 64 columns] piece of a slab
// a stage holds a Q block and a K block of R rows, or a V slab
__host__ __device__ constexpr int stage_bytes(int R) { return kQBlockBytes + R * 128 > kSlabBytes ? kQBlockBytes + R * 128 : kSlabBytes; }
constexpr int kMaxStages = 6;
constexpr int kSmemBytes = kRingBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int kSets = 1;                  // softmax threads per head
constexpr int kSoftmaxThreads = 128 * kSets;
constexpr int kThreads = 64 + kSoftmaxThreads + 32;      // TMA, MMA, kSets x 4 softmax warps, weight prefetch
constexpr int kPrefetchWarp = 2 + 4 * kSets;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 0, kColS = 256;            // O fp32 [128 x 256]; S fp32 [128 x R], P over it
constexpr float kLazyThreshold = 8.0f;    // log2 units
constexpr int kMaxSlabs = 4;

struct WideSeqs {
    CUtensorMap k[kMaxBatch];             // boxes of 64 columns x R rows
    CUtensorMap v[kMaxBatch];             // boxes of 64 columns x 64 rows
    CUtensorMap o;                        // the partial outputs as fp32 [slots x 128 heads][512], boxes of 32 columns x 128 rows
    int o_rows_per_seq;                   // rows of that tensor between consecutive sequences
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

// kR: cache rows per tile (one scores MMA covers them all); kCl: row runs merged on chip (cluster size)
template <int kR, int kCl>
__global__ void __maxnreg__(112)
attn_wide_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ WideSeqs seqs, AttnPartials part,
                 float scale_log2, unsigned *status, unsigned long long *trace, const L2Prefetch pf)
{
    static_assert(kR == 64 || kR == 128 || kR == 256, "rows per tile");
    constexpr int kHeadsPerRank = kHeads / kCl;
    constexpr int kSlabs = kR / kSlabRows;
    constexpr int kStageBytes = stage_bytes(kR), kStages = kRingBytes / kStageBytes;     // 4 stages of 48 KB, or 6 of 32 KB
    static_assert(kStages >= 2 && kStages <= kMaxStages && kRingBytes >= kHeads * kDvHalf * 4, "ring");
    const int seq = blockIdx.z;
    const CUtensorMap *map_k = &seqs.k[seq], *map_v = &seqs.v[seq];
    const int n_rows = seqs.n_rows[seq], rows_per_split = seqs.rows_per_split[seq];
    part.ml += (size_t)seq * seqs.ml_stride;
    part.O += (size_t)seq * seqs.o_stride;
    // Tuning aid: four stamps of every CTA of sequence 0 (start, Q landed, last P*V done, end) from trace[32] on, and of
    // CTA (0,0): trace[4..] = first scores issued, scores seen, maximum known, first P signalled, last P signalled;
    // trace[24..] = rows parked, cluster barrier passed, weights known, rows pulled and stored, second barrier passed
#define NM_TRACE(i) do { if (trace && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) trace[i] = global_timer_ns(); } while (0)
#define NM_TRACE_CTA(i) do { if (trace && blockIdx.z == 0) trace[32 + 4 * (blockIdx.y * gridDim.x + blockIdx.x) + (i)] = global_timer_ns(); } while (0)
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;            // swizzle atoms want 1024-byte alignment
    unsigned char *smem = smem_raw + (base - raw_addr);
    const uint32_t ring_addr = base, park_addr = base;            // the merge parks O in the ring once the loop is over
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kRingBytes);
    // Ring: full[b] (a stage's copies landed), empty[b] (the MMAs that read it are done).  Per tile:
    // s_full (scores in TMEM), p_ready[q] (P of slab q written, 128 arrivals), pv_done (P*V of the tile finished).
    const uint32_t bar_full = smem_u32(bars + 0), bar_empty = smem_u32(bars + kMaxStages),
                   bar_s_full = smem_u32(bars + 2 * kMaxStages), bar_p_ready = smem_u32(bars + 2 * kMaxStages + 1),
                   bar_pv_done = smem_u32(bars + 2 * kMaxStages + 1 + kMaxSlabs);
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(8) float s_mlp[kCl][kHeadsPerRank][2];   // (m in log2 units, l) of the owned heads, written by each peer
    __shared__ float s_w[kCl][kHeadsPerRank];                     // weights of the slots in the final sum
    __shared__ float s_pair[2][kHeads];                           // what the two softmax threads of a head tell each other

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sp = blockIdx.x, half = blockIdx.y;
    const int r0 = sp * rows_per_split, r1 = min(n_rows, r0 + rows_per_split);
    const int ntiles = (r1 > r0) ? ceil_div(r1 - r0, kR) : 0;      // 0 for the padding CTAs of the last cluster
    if constexpr (kCl == 1) {
        if (ntiles == 0) return;                                   // no peers wait for a CTA without rows
    }

    if (tid == 0) {
        NM_TRACE(0);
        NM_TRACE_CTA(0);
        s_abort = 0;
        for (int b = 0; b < kStages; ++b) { mbar_init(bar_full + 8 * b, 1); mbar_init(bar_empty + 8 * b, 1); }
        mbar_init(bar_s_full, 1);
        for (int q = 0; q < kMaxSlabs; ++q) mbar_init(bar_p_ready + 8 * q, kSoftmaxThreads);
        mbar_init(bar_pv_done, 1);
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
    if constexpr (kCl > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    pdl_launch_dependents();
    const uint32_t rank = cluster_rank();
    const int cluster_id = sp / kCl;
    float m_own = -INFINITY, l_own = 0.f;                         // softmax threads: this run's (m, l)
    // slabs of tile t that hold at least one attended row (only a run's last tile can be short)
    auto slabs_of = [&](int t) { return min(kSlabs, ceil_div(r1 - (r0 + t * kR), kSlabRows)); };

    if (warp == 0) {
        // ---------------- TMA producer --------------------------------------------------------------
        if (lane == 0) {
            tma_prefetch_descriptor(&map_q);
            tma_prefetch_descriptor(map_k);
            tma_prefetch_descriptor(map_v);
            const uint64_t keep = l2_policy_evict_last();
            int item = 0;
            bool ok = true, waited = false;
            auto acquire = [&]() {                                 // the stage of ring item `item`, free again
                const int b = item % kStages;
                if (item >= kStages) {
                    const uint32_t bar = bar_empty + 8 * b, par = ((item / kStages) - 1) & 1;
                    if (!mbar_try_wait(bar, par) && !mbar_wait(bar, par, &s_abort, status)) ok = false;
                }
                return b;
            };
            // The cache rows were written by earlier steps, not by the kernels just before this one: the K blocks of the
            // first stages are on their way before this CTA waits for those kernels; the Q blocks, which they produce,
            // follow into the same stages.
            const int early = min(kStages, ntiles > 0 ? kKBlocks : 0);
            for (int c = 0; c < early; ++c) {
                mbar_arrive_expect_tx(bar_full + 8 * c, kQBlockBytes + kR * 128);
                tma_load_2d(ring_addr + c * kStageBytes + kQBlockBytes, map_k, c * 64, r0, bar_full + 8 * c, keep);
            }
            pdl_wait_prior_grids();
            waited = true;
            for (int c = 0; c < early; ++c) tma_load_2d(ring_addr + c * kStageBytes, &map_q, c * 64, seq * kHeads, bar_full + 8 * c, keep);
            for (int t = 0; t < ntiles && ok; ++t) {
                const int row = r0 + t * kR;
                for (int c = 0; c < kKBlocks && ok; ++c) {
                    if (t == 0 && c < early) { ++item; continue; }
                    const int b = acquire();
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar_full + 8 * b, kQBlockBytes + kR * 128);
                    tma_load_2d(ring_addr + b * kStageBytes + kQBlockBytes, map_k, c * 64, row, bar_full + 8 * b, keep);
                    tma_load_2d(ring_addr + b * kStageBytes, &map_q, c * 64, seq * kHeads, bar_full + 8 * b, keep);
                    ++item;
                }
                const int ns = slabs_of(t);
                for (int q = 0; q < ns && ok; ++q) {
                    const int b = acquire();
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar_full + 8 * b, kSlabBytes);
                    for (int i = 0; i < 4; ++i)
                        tma_load_2d(ring_addr + b * kStageBytes + i * kSubBlockBytes, map_v, half * kDvHalf + 64 * i, row + q * kSlabRows,
                                    bar_full + 8 * b, keep);
                    ++item;
                }
            }
            (void)waited;
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ---------------------------------------------------------------
        if (lane == 0 && ntiles > 0) {
            constexpr uint32_t idesc_s = instr_desc(128, kR, false, false), idesc_o = instr_desc(128, kDvHalf, false, true);
            bool ok = true;
            int item = 0;
            for (int t = 0; t < ntiles && ok; ++t) {
                // S is free: the P*V of the previous tile was issued before these MMAs and the pipe runs in order
                for (int c = 0; c < kKBlocks && ok; ++c) {
                    const int b = item % kStages;
                    ok = mbar_wait(bar_full + 8 * b, (item / kStages) & 1, &s_abort, status);
                    if (!ok) break;
                    if (item == 0) NM_TRACE_CTA(1);
                    tc_fence_after();
                    const uint64_t q_desc0 = smem_desc(ring_addr + b * kStageBytes, 16, 1024);
                    const uint64_t k_desc0 = smem_desc(ring_addr + b * kStageBytes + kQBlockBytes, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ss(tmem + kColS, q_desc0 + (uint64_t)((kk * 32) >> 4), k_desc0 + (uint64_t)((kk * 32) >> 4), idesc_s, (c | kk) != 0);
                    mma_commit(bar_empty + 8 * b);
                    ++item;
                    if (t == 0 && c == 0) NM_TRACE(4);
                }
                if (!ok) break;
                mma_commit(bar_s_full);
                const int ns = slabs_of(t);
                for (int q = 0; q < ns && ok; ++q) {
                    const int b = item % kStages;
                    ok = mbar_wait(bar_full + 8 * b, (item / kStages) & 1, &s_abort, status) &&
                         mbar_wait(bar_p_ready + 8 * q, t & 1, &s_abort, status);
                    if (!ok) break;
                    tc_fence_after();
                    if (t == 0) NM_TRACE(12 + q);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        // rows 64 q + 16 kk ..: P sits over the 16 columns of S it came from, hi in the first 8 (bf16 pairs), lo in the next 8
                        const uint32_t p_hi = tmem + kColS + 16 * (4 * q + kk), p_lo = p_hi + 8;
                        const uint64_t vdesc = smem_desc(ring_addr + b * kStageBytes + kk * 2048, kSubBlockBytes, 1024);
                        mma_ts(tmem + kColO, p_hi, vdesc, idesc_o, (t | q | kk) != 0);
                        mma_ts(tmem + kColO, p_lo, vdesc, idesc_o, true);
                    }
                    mma_commit(bar_empty + 8 * b);
                    if (t == 0) NM_TRACE(16 + q);
                    ++item;
                }
                if (!ok) break;
                mma_commit(bar_pv_done);
            }
        }
    } else if (warp == kPrefetchWarp) {
        // ---------------- weight prefetch (launched only when there is something to prefetch) ----------------------
        if (ntiles > 0) {                                          // sleep-poll: this warp must not take issue slots from the pipeline
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(bar_full, 0)) {
                __nanosleep(128);
                if (s_abort || global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
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
    } else if (warp >= 2 && warp < 2 + 4 * kSets) {
        // ---------------- softmax, lazy rescale: two threads per head (warps 2-5 take the even 32-row chunks of a tile,
        //                  warps 6-9 the odd ones; warp w may touch the TMEM lanes of quarter w % 4) -----------------
        const int set = (warp - 2) >> 2, quad = warp & 3, head = quad * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        for (int t = 0; t < ntiles; ++t) {
            // (after an expired wait every later wait returns at once: the loop runs on, so that all 256 threads keep meeting
            // at the named barriers below, and ends with a result that the status word disowns)
            ok = mbar_wait(bar_s_full, t & 1, &s_abort, status) && ok;
            tc_fence_after();
            if (t == 0 && tid == 64) NM_TRACE(5);
            const int valid = min(kR, r1 - (r0 + t * kR));
            const int nchunks = ceil_div(valid, 32);
            // pass 1: the row maximum of this tile, each thread over its chunks, then both together
            float mx = -INFINITY;
            {
                float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;      // four chains instead of one
                for (int j = set; j < nchunks; j += kSets) {
                    uint32_t sa[16], sb[16];                        // both halves of the chunk requested before either is used
                    tmem_ld16(lane_base + kColS + 32 * j, sa);
                    tmem_ld16(lane_base + kColS + 32 * j + 16, sb);
                    tmem_wait_ld();
                    if (32 * j + 32 <= valid) {
#pragma unroll
                        for (int i = 0; i < 16; i += 2) {
                            m0 = fmaxf(m0, __uint_as_float(sa[i])); m1 = fmaxf(m1, __uint_as_float(sa[i + 1]));
                            m2 = fmaxf(m2, __uint_as_float(sb[i])); m3 = fmaxf(m3, __uint_as_float(sb[i + 1]));
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            if (32 * j + i < valid) m0 = fmaxf(m0, __uint_as_float(sa[i]));
                            if (32 * j + 16 + i < valid) m2 = fmaxf(m2, __uint_as_float(sb[i]));
                        }
                    }
                }
                mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
            }
            if constexpr (kSets == 2) {
                s_pair[set][head] = mx;
                named_barrier_sync(2, kSoftmaxThreads);
                mx = fmaxf(s_pair[0][head], s_pair[1][head]);
            }
            const float mx2 = mx * scale_log2;
            const bool grow = (t == 0) || (mx2 > m_used + kLazyThreshold);
            // s_full of this tile was committed behind the P*V of the previous one: O is at rest
            if (t > 0 && __any_sync(0xffffffffu, grow)) {
                // rare: the maximum grew by more than 2^8; each of the head's two threads rescales half of the columns
                const float f = grow ? fast_exp2(m_used - mx2) : 1.0f;
                for (int c = (16 / kSets) * set; c < (16 / kSets) * (set + 1); ++c) {
                    uint32_t o[16];
                    tmem_ld16(lane_base + kColO + c * 16, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tmem_st16(lane_base + kColO + c * 16, o);
                }
                tmem_wait_st();
                if (grow) l *= f;
            }
            if (grow) m_used = mx2;
            if (t == 0 && tid == 64) NM_TRACE(6);
            // pass 2: P over the columns of S just read, 16 rows at a time (hi in the first 8 columns, lo in the next 8);
            // a signal from every thread per 64-row slab, whether or not it had a chunk of it
            float lsum = 0.f, lsum1 = 0.f;
            const int ns = slabs_of(t);
            uint32_t sr[32], nx[32];                                // this chunk's scores, and the next chunk's on their way
            if (set < 2 * ns) {
                tmem_ld16(lane_base + kColS + 32 * set, reinterpret_cast<uint32_t (&)[16]>(nx[0]));
                tmem_ld16(lane_base + kColS + 32 * set + 16, reinterpret_cast<uint32_t (&)[16]>(nx[16]));
            }
            for (int j = set; j < 2 * ns; j += kSets) {
                const uint32_t col = lane_base + kColS + 32 * j;
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) sr[i] = nx[i];
                if (j + kSets < 2 * ns) {                          // requested before this chunk's exponentials, used after them
                    tmem_ld16(col + 32 * kSets, reinterpret_cast<uint32_t (&)[16]>(nx[0]));
                    tmem_ld16(col + 32 * kSets + 16, reinterpret_cast<uint32_t (&)[16]>(nx[16]));
                }
                const bool full = 32 * j + 32 <= valid;
#pragma unroll
                for (int hq = 0; hq < 2; ++hq) {
                    uint32_t pr[8], plo[8];
                    const int row0 = 32 * j + 16 * hq;
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float p0 = fast_exp2(fmaf(__uint_as_float(sr[16 * hq + i]), scale_log2, -m_used));
                        float p1 = fast_exp2(fmaf(__uint_as_float(sr[16 * hq + i + 1]), scale_log2, -m_used));
                        if (!full) {
                            if (row0 + i >= valid) p0 = 0.f;
                            if (row0 + i + 1 >= valid) p1 = 0.f;
                        }
                        lsum += p0; lsum1 += p1;
                        // P = hi + lo in two bf16 terms, both by truncation (a mask and a byte permute; the float-to-bf16
                        // conversion shares the 16-lane unit with the exponentials, which bound this loop): hi keeps the top
                        // 8 significand bits, lo the next 8 of the exact remainder - about 2^-16 relative, from below
                        const uint32_t u0 = __float_as_uint(p0), u1 = __float_as_uint(p1);
                        const float r0 = p0 - __uint_as_float(u0 & 0xffff0000u), r1 = p1 - __uint_as_float(u1 & 0xffff0000u);
                        pr[i >> 1] = __byte_perm(u0, u1, 0x7632);
                        plo[i >> 1] = __byte_perm(__float_as_uint(r0), __float_as_uint(r1), 0x7632);
                    }
                    tmem_st8(col + 16 * hq, pr);
                    tmem_st8(col + 16 * hq + 8, plo);
                }
                if (kSets == 2 || (j & 1)) {                        // this thread's part of the 64-row slab is written
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar_p_ready + 8 * (j >> 1));
                    if (t == 0 && tid == 64) NM_TRACE((j >> 1) == 0 ? 7 : 19 + (j >> 1));
                }
            }
            lsum += lsum1;
            l += lsum;
            if (t == 0 && tid == 64) NM_TRACE(8);
            // the next tile's scores overwrite P: they are issued behind this tile's P*V, nothing to wait for here
        }
        // the last P*V must have landed before O is read
        if (ntiles > 0) {
            mbar_wait(bar_pv_done, (ntiles - 1) & 1, &s_abort, status);
            tc_fence_after();
        }
        (void)ok;
        if (tid == 64) NM_TRACE_CTA(2);
        // the head's sum: first thread's chunks, then the second's (fixed order)
        m_own = m_used; l_own = l;
        if constexpr (kSets == 2) {
            s_pair[set][head] = l;
            named_barrier_sync(2, kSoftmaxThreads);
            l_own = s_pair[0][head] + s_pair[1][head];
        }
    }

    // ---- a run on its own (cluster of one): its O rows go out as one partial through shared memory and tiled TMA
    //      stores - eight [128 heads x 32 columns] boxes in the 128-byte swizzle, written one row per thread without
    //      bank conflicts and copied out by the copy engine while the next box is being filled ----------------------
    if constexpr (kCl == 1) {
        if (warp >= 2 && warp < 2 + 4 * kSets) {
            const int set = (warp - 2) >> 2, quad = warp & 3, head = quad * 32 + lane;
            const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
            if (half == 0 && set == 0) {
                part.ml[((size_t)sp * kHeads + head) * 2] = m_own * 0.6931471805599453f;       // natural-log units
                part.ml[((size_t)sp * kHeads + head) * 2 + 1] = l_own;
            }
            // each of the head's threads moves its share of the columns, kBoxGroup boxes between barriers: the loads of a
            // group are all requested before the first is used, and the copy engine works on one group while the next is filled
            constexpr int kBoxGroup = 4;
            for (int c0 = (8 / kSets) * set; c0 < (8 / kSets) * (set + 1); c0 += kBoxGroup) {
                uint32_t o[2][32];
                tmem_ld16(lane_base + kColO + c0 * 32, reinterpret_cast<uint32_t (&)[16]>(o[0][0]));
                tmem_ld16(lane_base + kColO + c0 * 32 + 16, reinterpret_cast<uint32_t (&)[16]>(o[0][16]));
#pragma unroll
                for (int g = 0; g < kBoxGroup; ++g) {
                    const int c = c0 + g;
                    tmem_wait_ld();
                    if (g + 1 < kBoxGroup) {
                        tmem_ld16(lane_base + kColO + (c + 1) * 32, reinterpret_cast<uint32_t (&)[16]>(o[(g + 1) & 1][0]));
                        tmem_ld16(lane_base + kColO + (c + 1) * 32 + 16, reinterpret_cast<uint32_t (&)[16]>(o[(g + 1) & 1][16]));
                    }
                    const uint32_t row = park_addr + (uint32_t)c * 16384u + (uint32_t)head * 128u;
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + ((uint32_t)(i / 4) ^ ((uint32_t)head & 7u)) * 16u),
                                     "r"(o[g & 1][i]), "r"(o[g & 1][i + 1]), "r"(o[g & 1][i + 2]), "r"(o[g & 1][i + 3]) : "memory");
                }
                fence_proxy_async();
                named_barrier_sync(3 + set, 128);
                if (lane == 0 && quad == 2) {                      // threads 64 and 192
                    for (int c = c0; c < c0 + kBoxGroup; ++c)
                        tma_store_2d(&seqs.o, half * kDvHalf + 32 * c, seq * seqs.o_rows_per_seq + sp * kHeads, park_addr + (uint32_t)c * 16384u);
                    bulk_commit_group();
                }
            }
            if (lane == 0 && quad == 2) {
                if (tid == 64) NM_TRACE(24);
                bulk_wait_all();
                if (tid == 64) NM_TRACE(27);
            }
        }
        tc_fence_before();
        __syncthreads();
        if (s_abort && tid == 0) {
            // a wait expired: give copies already issued a bounded chance to land before the CTA exits
            for (int i = 0; i < (1 << 16) && !mbar_try_wait(bar_full, 0); ++i) {}
        }
        if (warp == 1) {
            tc_fence_after();
            tmem_dealloc(tmem, kTmemCols);
        }
        if (tid == 0) NM_TRACE_CTA(3);
        return;
    }

    // ---- merge of the cluster's row runs through distributed shared memory -----------------------------------
    // Each CTA parks its (unscaled) O rows in its own shared memory (the Q tile is free by then; layout [head][64 float4],
    // the float4 index XOR-ed with (head & 7) so that neither the row-per-thread writes nor the row-contiguous reads
    // conflict) and pushes its (m, l) pairs to the peers that own the heads.  After one cluster barrier, rank r combines
    // heads [128/kCl * r, ...) over all peers - weights 2^(m_peer - max m) - and writes one partial per cluster.  A
    // last barrier keeps every CTA's shared memory alive until its peers have read it.
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");       // all peers are running (they arrived at kernel start)
    if (warp >= 2 && warp < 2 + 4 * kSets) {
        const int set = (warp - 2) >> 2, quad = warp & 3, head = quad * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        if (set == 0) {
            const uint32_t slot = peer_smem(smem_u32(&s_mlp[rank][head % kHeadsPerRank][0]), (uint32_t)head / kHeadsPerRank);
            asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(slot), "f"((ntiles > 0) ? m_own : -INFINITY), "f"(l_own) : "memory");
        }
        if (ntiles > 0) {
            for (int c = (16 / kSets) * set; c < (16 / kSets) * (set + 1); ++c) {          // each of the head's threads parks its share of the columns
                uint32_t o[16];
                tmem_ld16(lane_base + kColO + c * 16, o);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    const uint32_t q4 = (uint32_t)(c * 4 + i / 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(park_addr + (uint32_t)(head * 64 + (q4 ^ (head & 7u))) * 16u),
                                 "r"(o[i]), "r"(o[i + 1]), "r"(o[i + 2]), "r"(o[i + 3]) : "memory");
                }
            }
        }
        if (tid == 64) NM_TRACE(24);
    }
    cluster_sync_all();                                            // every peer's rows and (m, l) are parked
    if (tid == 64) NM_TRACE(25);
    if (warp >= 2 && warp < 2 + 4 * kSets) {
        const int t = tid - 64;                                    // 0..kSoftmaxThreads-1
        if (t < 128) {                                             // weight of peer r for owned head hl
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
        named_barrier_sync(2, kSoftmaxThreads);
        if (tid == 64) NM_TRACE(26);
        constexpr int kIters = kHeadsPerRank * 64 / kSoftmaxThreads, kBatch = 4;
        for (int i0 = 0; i0 < kIters; i0 += kBatch) {
            float4 v[kBatch][kCl];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {                     // kBatch * kCl remote loads in flight
                const int idx = t + kSoftmaxThreads * (i0 + b);
                const int hl = idx / 64, q4 = idx % 64, head = (int)rank * kHeadsPerRank + hl;
                const uint32_t local = park_addr + (uint32_t)(head * 64 + (q4 ^ (head & 7))) * 16u;
#pragma unroll
                for (int r = 0; r < kCl; ++r)
                    v[b][r] = (s_w[r][hl] != 0.f) ? ld_peer_f4(peer_smem(local, r)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int idx = t + kSoftmaxThreads * (i0 + b);
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
    if (tid == 64) NM_TRACE(27);
    cluster_sync_all();                                            // peers are done reading this CTA's shared memory
    if (tid == 64) NM_TRACE(28);

    // ---- teardown: TMEM goes back ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (s_abort && tid == 0) {
        // a wait expired: give copies already issued a bounded chance to land before the CTA exits
        for (int i = 0; i < (1 << 16) && ntiles > 0 && !mbar_try_wait(bar_full, 0); ++i) {}
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
    if (tid == 0) NM_TRACE_CTA(3);
#undef NM_TRACE
#undef NM_TRACE_CTA
}

// Tensor maps: bf16 [rows][576], boxes of 64 columns (128 bytes, the swizzle span) x box_rows rows.
bool encode_rows_map_wide(CUtensorMap *map, const void *ptr, int rows, int box_rows)
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

template <int kR, int kCl>
int launch_wide(const CUtensorMap &map_q, const WideSeqs &seqs, int nseq, int nsplit, AttnPartials part, float scale, cudaStream_t stream,
                bool programmatic_launch, const L2Prefetch &prefetch)
{
    static std::atomic<unsigned long long> configured{0};          // per instantiation, one bit per device
    cudaError_t e = ensure_dynamic_smem(attn_wide_kernel<kR, kCl>, kSmemBytes, configured);
    if (e != cudaSuccess) return record_cuda_error(e, "attention kernel attribute");
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(nsplit, kCl) * kCl, 2, nseq);      // padded to whole clusters; padding CTAs have no rows
    const bool has_prefetch = prefetch.block_bytes > 0 || (prefetch.nranges > 0 && prefetch.range_bytes > 0);
    cfg.blockDim = dim3(has_prefetch ? kThreads : kThreads - 32);       // the prefetch warp is the last one
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic_launch ? 2 : 1;
    e = cudaLaunchKernelEx(&cfg, attn_wide_kernel<kR, kCl>, map_q, seqs, part, scale_log2, device_status_ptr(), attention_trace(), prefetch);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention (tensor cores, wide tiles) launch");
}

template <int kR>
int launch_wide_r(int cluster, const CUtensorMap &map_q, const WideSeqs &seqs, int nseq, int nsplit, AttnPartials part, float scale,
                  cudaStream_t stream, bool pdl, const L2Prefetch &prefetch)
{
    if (cluster == 4) return launch_wide<kR, 4>(map_q, seqs, nseq, nsplit, part, scale, stream, pdl, prefetch);
    if (cluster == 2) return launch_wide<kR, 2>(map_q, seqs, nseq, nsplit, part, scale, stream, pdl, prefetch);
    return launch_wide<kR, 1>(map_q, seqs, nseq, nsplit, part, scale, stream, pdl, prefetch);
}

}  // namespace

int attention_partial_wide(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split, int nsplit,
                           int tile_rows, int cluster, AttnPartials part, int slot_stride, float scale, cudaStream_t stream,
                           bool programmatic_launch, L2Prefetch prefetch)
{
    if (nseq < 1 || nseq > kMaxBatch || nsplit < 1) return NM_ERR_UNSUPPORTED;
    if (cluster != 1 && cluster != 2 && cluster != 4) return NM_ERR_UNSUPPORTED;
    if (tile_rows != 64 && tile_rows != 128 && tile_rows != 256) return NM_ERR_UNSUPPORTED;
    if ((uintptr_t)Q & 15u) return NM_ERR_UNSUPPORTED;
    CUtensorMap map_q;
    WideSeqs seqs{};
    seqs.ml_stride = (long)slot_stride * kHeads * 2;
    seqs.o_stride = (long)slot_stride * kHeads * kDv;
    if (!encode_rows_map_wide(&map_q, Q, nseq * kHeads, kHeads)) return NM_ERR_UNSUPPORTED;
    for (int t = 0; t < nseq; ++t) {
        seqs.n_rows[t] = n_rows[t];
        seqs.rows_per_split[t] = rows_per_split[t];
        if (n_rows[t] < 1) {                                       // nothing to attend: its CTAs find no tiles and load nothing
            seqs.k[t] = map_q; seqs.v[t] = map_q;
            seqs.rows_per_split[t] = tile_rows;
            continue;
        }
        if (rows_per_split[t] % tile_rows != 0) return NM_ERR_UNSUPPORTED;
        if ((uintptr_t)caches[t] & 15u) return NM_ERR_UNSUPPORTED;
        // The cache maps cover exactly the rows attended: rows past n_rows read as zeros (and are masked),
        // whatever the rest of the buffer holds.
        if (!encode_rows_map_wide(&seqs.k[t], caches[t], n_rows[t], tile_rows)) return NM_ERR_UNSUPPORTED;
        if (!encode_rows_map_wide(&seqs.v[t], caches[t], n_rows[t], kSlabRows)) return NM_ERR_UNSUPPORTED;
    }
    if (cluster == 1) {
        // the partials as one fp32 tensor [rows][512]: row = (sequence * slot_stride + run) * 128 + head
        EncodeTiledFn enc = tensor_map_encoder();
        const long rows = (nseq > 1 ? (long)nseq * slot_stride : (long)nsplit) * kHeads;
        if (!enc || ((uintptr_t)part.O & 15u)) return NM_ERR_UNSUPPORTED;
        const cuuint64_t dims[2] = {(cuuint64_t)kDv, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)kDv * 4};
        const cuuint32_t box[2] = {32, (cuuint32_t)kHeads};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&seqs.o, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, part.O, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return NM_ERR_UNSUPPORTED;
        seqs.o_rows_per_seq = slot_stride * kHeads;
    }
    if (tile_rows == 256) return launch_wide_r<256>(cluster, map_q, seqs, nseq, nsplit, part, scale, stream, programmatic_launch, prefetch);
    if (tile_rows == 128) return launch_wide_r<128>(cluster, map_q, seqs, nseq, nsplit, part, scale, stream, programmatic_launch, prefetch);
    return launch_wide_r<64>(cluster, map_q, seqs, nseq, nsplit, part, scale, stream, programmatic_launch, prefetch);
}

}  // namespace nm
