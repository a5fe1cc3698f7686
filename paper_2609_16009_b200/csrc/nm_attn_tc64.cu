// Latent attention pass on the tensor cores, 64 heads per CTA (tcgen05.mma with M = 64).
//
// The 128-head kernel of nm_attn_tc.cu keeps all of Q (147 KB) in shared memory, which leaves room for two
// 32-row cache stages only; its scores MMAs (M128 N32 K16) are bound by re-reading a 4 KB slice of Q from
// shared memory for every 32 cache rows.  Here a CTA takes one half of the heads: Q is 72 KB, the two cache
// stages hold 64 rows each, and one M64 N64 K16 MMA reads 2 KB of Q per 64 rows - a quarter of the shared
// memory traffic per score.  Four CTAs share a sequence split: (head half) x (half of the 512 output columns).
// Per CTA the partial result is 64 heads x 256 columns, so the cluster merge moves half as much per CTA, and
// with 32 splits instead of 64 the final merge reads half as many partials.
//
// For a tile of 64 cache rows:
//   S[64 x 64]    = Q[64 x 576] * tile^T        36 MMAs dealt to two accumulators (a chain of MMAs into one
//                                               accumulator waits for its predecessor), added by the softmax
//   P             = exp2(S*c - m)               two threads per head: with M = 64 the accumulator rows sit in
//                                               lanes 0-15 of each 32-lane quarter of TMEM; the half-split
//                                               load/store shape gives thread l columns 0-31 of row l and
//                                               thread l + 16 columns 32-63, so the whole warp works
//   O[64 x 256]  += P[64 x 64] * tile[:, half]  P from TMEM as two bf16 terms (hi + lo), over the columns of
//                                               the first score accumulator, which is free once it was read
// Everything else - TMA with 128-byte swizzle, lazy rescale, double-buffered stages, bounded waits, the
// cluster-of-four merge through distributed shared memory, the optional L2 prefetch warp - is as in the
// 128-head kernel.
#include "nm_async.cuh"
#include "nm_mla.cuh"
#include "nm_tcgen05.cuh"

namespace nm {

namespace {

constexpr int kHeads = 128;
constexpr int kHeadsCta = 64;             // heads per CTA (the MMA's M)
constexpr int kDqk = 576;
constexpr int kDv = 512;
constexpr int kDvHalf = 256;
constexpr int kT = 64;                    // cache rows per stage
constexpr int kKVStages = 2;
constexpr int kKBlocks = kDqk / 64;       // 9 blocks of 64 elements (one 128-byte swizzle span)
constexpr int kQBlockBytes = kHeadsCta * 128;        // 8 KB
constexpr int kKVBlockBytes = kT * 128;              // 8 KB
constexpr int kQBytes = kKBlocks * kQBlockBytes;     // 73728
constexpr int kKVBytes = kKBlocks * kKVBlockBytes;   // 73728 per stage
constexpr int kSmemBytes = kQBytes + kKVStages * kKVBytes + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int kThreads = 224;             // TMA, MMA, 4 softmax warps, weight prefetch
constexpr uint32_t kTmemCols = 512;
constexpr int kSAcc = 2;
// TMEM columns: O (fp32, 256); per stage b two score accumulators of 64 columns at 256 + 128 b (+ 64); P_hi and
// P_lo (bf16 pairs, 32 columns each) over the first accumulator of the same stage
constexpr uint32_t kColO = 0, kColS = 256;
constexpr float kLazyThreshold = 8.0f;    // log2 units
// The splits merged on chip form a cluster of kCl CTAs (template argument: 4, 2 or 1); rank r owns kHeadsCta / kCl heads
// in the merge (with four ranks: the 16 heads of softmax warp r).

struct AttnSeqs64 {
    CUtensorMap kv[kMaxBatch];
    int n_rows[kMaxBatch];
    int rows_per_split[kMaxBatch];
    long ml_stride, o_stride;
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
    __syncwarp();
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
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int kCl>
__global__ void __maxnreg__(120)
attn_tc64_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ AttnSeqs64 seqs, AttnPartials part,
                 float scale_log2, unsigned *status, unsigned long long *trace, const L2Prefetch pf)
{
    constexpr int kHeadsPerRank = kHeadsCta / kCl;
    const int seq = blockIdx.z;
    const CUtensorMap *map_kv_p = &seqs.kv[seq];
    const int n_rows = seqs.n_rows[seq], rows_per_split = seqs.rows_per_split[seq];
    part.ml += (size_t)seq * seqs.ml_stride;
    part.O += (size_t)seq * seqs.o_stride;
    // Tuning aid: four stamps of every CTA of sequence 0 (start, Q landed, last P*V done, end) from trace[32] on
    // ... and of CTA (0,0) of sequence 0 per tile t < 5: trace[4 + 4 t ..] = scores issued, scores seen, P written, P*V issued;
    // trace[24..28] = rows parked, cluster barrier passed, weights known, rows pulled and stored, second barrier passed
#define NM_TRACE_TILE(t, i) do { if (trace && (t) < 5 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) trace[4 + 4 * (t) + (i)] = global_timer_ns(); } while (0)
#define NM_TRACE_MERGE(i) do { if (trace && tid == 64 && (blockIdx.x | blockIdx.y | blockIdx.z) == 0) trace[24 + (i)] = global_timer_ns(); } while (0)
#define NM_TRACE_CTA(i) do { if (trace && blockIdx.z == 0) trace[32 + 4 * (blockIdx.y * gridDim.x + blockIdx.x) + (i)] = global_timer_ns(); } while (0)
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    unsigned char *smem = smem_raw + (base - raw_addr);
    const uint32_t q_addr = base, kv_addr = base + kQBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kQBytes + kKVStages * kKVBytes);
    const uint32_t bar_q = smem_u32(bars + 0), bar_kv_full = smem_u32(bars + 1), bar_s_full = smem_u32(bars + 3),
                   bar_p_full = smem_u32(bars + 5), bar_pv_done = smem_u32(bars + 7);
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(8) float s_mlp[kCl][kHeadsPerRank][2];   // (m in log2 units, l) of the owned heads, written by each peer
    __shared__ float s_w[kCl][kHeadsPerRank];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sp = blockIdx.x, half = blockIdx.y & 1, hh = blockIdx.y >> 1;     // column half, head half
    const int r0 = sp * rows_per_split, r1 = min(n_rows, r0 + rows_per_split);
    const int ntiles = (r1 > r0) ? ceil_div(r1 - r0, kT) : 0;
    // Without cluster peers a CTA that has no rows (the surplus of a short sequence's grid row) has nothing to contribute
    // and nobody waiting for it: the final merge reads only the partials of splits that have rows.
    if constexpr (kCl == 1) {
        if (ntiles == 0) return;
    }

    if (tid == 0) {
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
    // First half of a cluster barrier: when its second half is waited for (before the merge) every peer has started,
    // which is what writing into a peer's shared memory requires.
    __syncwarp();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    pdl_launch_dependents();
    const uint32_t rank = cluster_rank();
    const int cluster_id = sp / kCl;
    float m_own = -INFINITY, l_own = 0.f;

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
            // The cache rows were written by earlier steps: fetch the first two tiles before waiting for the kernels
            // just before this one, pull the rest of the split's rows into L2, then fetch Q, which they produce.
            for (int t = 0; t < min(ntiles, kKVStages); ++t) load_tile(t);
            if (blockIdx.y == 0)
                for (int t = kKVStages; t < ntiles; ++t)
                    for (int c = 0; c < kKBlocks; ++c) tma_prefetch_l2_2d(map_kv_p, c * 64, r0 + t * kT);
            pdl_wait_prior_grids();
            if (ntiles > 0) {
                mbar_arrive_expect_tx(bar_q, kQBytes);
                for (int c = 0; c < kKBlocks; ++c)
                    tma_load_2d(q_addr + c * kQBlockBytes, &map_q, c * 64, seq * kHeads + hh * kHeadsCta, bar_q, keep);
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
            constexpr uint32_t idesc_s = instr_desc(kHeadsCta, kT, false, false), idesc_o = instr_desc(kHeadsCta, kDvHalf, false, true);
            const uint64_t q_desc0 = smem_desc(q_addr, 16, 1024), kv_desc0 = smem_desc(kv_addr, 16, 1024);
            auto scores = [&](int t) {                             // S[t&1] = Q * tile(t)^T  (tile t has landed)
                const int b = t & 1;
                const uint64_t kv_desc = kv_desc0 + (uint64_t)((b * kKVBytes) >> 4);
                const uint32_t s_col = tmem + kColS + 128 * b;
                tc_fence_after();
#pragma unroll
                for (int step = 0; step < kKBlocks * 4; ++step) {
                    const int c = step >> 2, kk = step & 3;
                    mma_ss(s_col + 64 * (step % kSAcc), q_desc0 + (uint64_t)((c * kQBlockBytes + kk * 32) >> 4),
                           kv_desc + (uint64_t)((c * kKVBlockBytes + kk * 32) >> 4), idesc_s, step >= kSAcc);
                }
                mma_commit(bar_s_full + 8 * b);
            };
            auto pv = [&](int t) {                                 // O += P[t&1] * tile(t)[:, half]  (P of tile t is written)
                const int b = t & 1;
                const uint32_t p_hi = tmem + kColS + 128 * b, p_lo = p_hi + 32;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kT / 16; ++kk) {
                    const uint64_t vdesc = smem_desc(kv_addr + b * kKVBytes + (4 * half) * kKVBlockBytes + kk * 2048, kKVBlockBytes, 1024);
                    mma_ts(tmem + kColO, p_hi + kk * 8, vdesc, idesc_o, (t | kk) != 0);
                    mma_ts(tmem + kColO, p_lo + kk * 8, vdesc, idesc_o, true);
                }
                mma_commit(bar_pv_done + 8 * b);
            };
            if (ntiles > 0) mbar_wait(bar_q, 0, &s_abort, status);
            NM_TRACE_CTA(1);
            // scores of tile ts (needs the tile, and S[ts&1] free: the P*V of tile ts-2 issued) and P*V of tile tp
            // (needs the softmax of tile tp): whichever is ready is issued; neither blocks the other
            int ts = 0, tp = 0;
            uint64_t idle_since = 0;
            while (tp < ntiles) {
                bool progress = false;
                if (ts < ntiles && ts <= tp + 1 && mbar_try_wait(bar_kv_full + 8 * (ts & 1), (ts >> 1) & 1)) {
                    scores(ts);
                    NM_TRACE_TILE(ts, 0);
                    ++ts;
                    progress = true;
                }
                if (mbar_try_wait(bar_p_full + 8 * (tp & 1), (tp >> 1) & 1)) {
                    pv(tp);
                    NM_TRACE_TILE(tp, 3);
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
        if (ntiles > 0) {
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(bar_kv_full, 0)) {
                __nanosleep(128);
                if (s_abort || global_timer_ns() - t0 > kWaitLimitNs) break;
            }
        }
        prefetch_weights();
    } else {
        // ---------------- softmax, lazy rescale: two threads per head.  The accumulator rows sit in lanes 0-15 of
        //                  each TMEM quarter; the half-split load shape hands columns 0-31 of row l to thread l and
        //                  columns 32-63 to thread l + 16, so all 32 threads of the warp work -----------------------
        const int quad = warp & 3, ch = lane >> 4;
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        float m_used = -INFINITY, l = 0.f;
        for (int t = 0; t < ntiles; ++t) {
            const int b = t & 1;
            mbar_wait(bar_s_full + 8 * b, (t >> 1) & 1, &s_abort, status);
            tc_fence_after();
            if (tid == 64) NM_TRACE_TILE(t, 1);
            const uint32_t s_col = lane_base + kColS + 128 * b;
            float s[32];
            {
                uint32_t a0[32], a1[32];
                tmem_ld32_halves<32>(s_col, a0);
                tmem_ld32_halves<32>(s_col + 64, a1);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) s[j] = __uint_as_float(a0[j]) + __uint_as_float(a1[j]);
            }
            const int valid = min(kT, r1 - (r0 + t * kT)) - 32 * ch;       // of this thread's 32 columns
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j < valid) mx = fmaxf(mx, s[j]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float mx2 = mx * scale_log2;
            const bool grow = (t == 0) || (mx2 > m_used + kLazyThreshold);
            // P[b] lies over S[b]'s first accumulator, which the loads above have emptied; it was last read by the
            // P*V of tile t-2, which the scores of this tile were issued behind
            if (t > 0 && __any_sync(0xffffffffu, grow)) {
                // rare: the maximum grew by more than 2^8.  O may only be touched between two P*V passes.
                mbar_wait(bar_pv_done + 8 * ((t - 1) & 1), ((t - 1) >> 1) & 1, &s_abort, status);
                tc_fence_after();
                const float f = grow ? fast_exp2(m_used - mx2) : 1.0f;
                for (int c = 0; c < kDvHalf / 64; ++c) {
                    uint32_t o[32];
                    tmem_ld32_halves<32>(lane_base + kColO + c * 64, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tmem_st32_halves<32>(lane_base + kColO + c * 64, o);
                }
                tmem_wait_st();
                if (grow) l *= f;
            }
            if (grow) m_used = mx2;
            float lsum = 0.f;
            uint32_t pr[16], plo[16];
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
                const float p0 = (j < valid) ? fast_exp2(fmaf(s[j], scale_log2, -m_used)) : 0.f;
                const float p1 = (j + 1 < valid) ? fast_exp2(fmaf(s[j + 1], scale_log2, -m_used)) : 0.f;
                lsum += p0 + p1;
                const uint32_t hi = pack_bf16x2(p0, p1);
                pr[j >> 1] = hi;
                plo[j >> 1] = pack_bf16x2(p0 - __uint_as_float(hi << 16), p1 - __uint_as_float(hi & 0xffff0000u));
            }
            l += lsum;
            tmem_st16_halves<16>(s_col, pr);                       // k 0-31 -> words 0-15, k 32-63 -> words 16-31
            tmem_st16_halves<16>(s_col + 32, plo);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p_full + 8 * b);
            if (tid == 64) NM_TRACE_TILE(t, 2);
        }
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        if (ntiles > 0) {                                          // the last P*V must have landed before O is read
            mbar_wait(bar_pv_done + 8 * ((ntiles - 1) & 1), ((ntiles - 1) >> 1) & 1, &s_abort, status);
            tc_fence_after();
        }
        if (tid == 64) NM_TRACE_CTA(2);
        m_own = m_used; l_own = l;
    }

    // ---- merge of the cluster's splits through distributed shared memory (as in the 128-head kernel; 64 heads,
    //      16 per rank = the heads of softmax warp `rank`) -----------------------------------------------------
    __syncwarp();
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");       // all peers are running (they arrived at kernel start)
    if (warp >= 2 && warp < 6) {
        const int quad = warp & 3, head = quad * 16 + lane;        // head within this CTA's 64 (lanes 0-15)
        const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16);
        if (lane < 16) {                                           // (m, l) to the rank that owns the head
            const int hd = quad * 16 + lane;
            const uint32_t slot = peer_smem(smem_u32(&s_mlp[rank][hd % kHeadsPerRank][0]), (uint32_t)(hd / kHeadsPerRank));
            asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(slot), "f"((ntiles > 0) ? m_own : -INFINITY), "f"(l_own) : "memory");
        }
        if (ntiles > 0) {
            // both halves of the warp park: thread l has columns 0-31 of a 64-column chunk of row l % 16, thread l + 16
            // columns 32-63 (the half-split load shape, as in the softmax)
            const uint32_t prow = (uint32_t)(quad * 16 + (lane & 15)), pch = (uint32_t)(lane >> 4);
            for (int c = 0; c < kDvHalf / 64; ++c) {
                uint32_t o[32];
                tmem_ld32_halves<32>(lane_base + kColO + c * 64, o);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    const uint32_t q4 = (uint32_t)(c * 16) + pch * 8 + (uint32_t)(i / 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(q_addr + (prow * 64 + (q4 ^ (prow & 7u))) * 16u),
                                 "r"(o[i]), "r"(o[i + 1]), "r"(o[i + 2]), "r"(o[i + 3]) : "memory");
                }
            }
        }
    }
    NM_TRACE_MERGE(0);
    cluster_sync_all();                                            // every peer's rows are parked, its (m, l) here
    NM_TRACE_MERGE(1);
    if (warp >= 2 && warp < 6) {
        const int t = tid - 64;                                    // 0..127
        if (t < kCl * kHeadsPerRank) {                             // weight of peer r for owned head hl
            const int hl = t % kHeadsPerRank, r = t / kHeadsPerRank, head_g = hh * kHeadsCta + (int)rank * kHeadsPerRank + hl;
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
                part.ml[((size_t)cluster_id * kHeads + head_g) * 2] = M * 0.6931471805599453f;     // natural-log units
                part.ml[((size_t)cluster_id * kHeads + head_g) * 2 + 1] = Ltot;
            }
        }
        named_barrier_sync(1, 128);
        NM_TRACE_MERGE(2);
        constexpr int kIters = kHeadsPerRank * 64 / 128, kBatch = 4;       // 8 float4 outputs per thread
        for (int i0 = 0; i0 < kIters; i0 += kBatch) {
            float4 v[kBatch][kCl];
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
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
                const int hl = idx / 64, q4 = idx % 64, head_g = hh * kHeadsCta + (int)rank * kHeadsPerRank + hl;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < kCl; ++r) {                    // rank order: deterministic
                    const float w = s_w[r][hl];
                    acc.x = fmaf(w, v[b][r].x, acc.x); acc.y = fmaf(w, v[b][r].y, acc.y);
                    acc.z = fmaf(w, v[b][r].z, acc.z); acc.w = fmaf(w, v[b][r].w, acc.w);
                }
                *reinterpret_cast<float4 *>(part.O + ((size_t)cluster_id * kHeads + head_g) * kDv + half * kDvHalf + q4 * 4) = acc;
            }
        }
    }
    NM_TRACE_MERGE(3);
    cluster_sync_all();                                            // peers are done reading this CTA's shared memory
    NM_TRACE_MERGE(4);

    // ---- teardown: TMEM goes back ---------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (s_abort && tid == 0) {
        for (int i = 0; i < (1 << 16) && ntiles > 0 && !mbar_try_wait(bar_q, 0); ++i) {}
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
    if (tid == 0) NM_TRACE_CTA(3);
#undef NM_TRACE_CTA
#undef NM_TRACE_MERGE
#undef NM_TRACE_TILE
}

bool encode_rows_map64(CUtensorMap *map, const void *ptr, int rows, int box_rows)
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

namespace {
template <int kCl>
int configure_tc64()
{
    static std::atomic<unsigned long long> configured{0};          // per instantiation, one bit per device
    cudaError_t e = ensure_dynamic_smem(attn_tc64_kernel<kCl>, kSmemBytes, configured);
    if (e != cudaSuccess) return record_cuda_error(e, "attention kernel attribute");
    return NM_OK;
}
// Clusters of kCl CTAs of this kernel that the device holds at once (clusters do not straddle GPCs, so this is
// fewer than SMs / kCl); 0 if the query fails.
template <int kCl>
int max_clusters_tc64()
{
    if (configure_tc64<kCl>() != NM_OK) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kCl, 4, 1); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kCl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return max_clusters_cached(attn_tc64_kernel<kCl>, cfg, kCl);
}
template <int kCl>
int launch_tc64(const CUtensorMap &map_q, const AttnSeqs64 &seqs, int nseq, int nsplit, AttnPartials part, float scale, cudaStream_t stream,
                bool programmatic_launch, const L2Prefetch &prefetch)
{
    if (int rc = configure_tc64<kCl>()) return rc;
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(nsplit, kCl) * kCl, 4, nseq);      // y: column half + 2 * head half; padding CTAs have no rows
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_tc64_kernel<kCl>, map_q, seqs, part, scale_log2, device_status_ptr(), attention_trace(), prefetch);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention (tensor cores, 64 heads per CTA) launch");
}
}  // namespace

int attention_tc64_max_clusters(int cluster)
{
    return cluster == 4 ? max_clusters_tc64<4>() : (cluster == 2 ? max_clusters_tc64<2>() : (cluster == 1 ? max_clusters_tc64<1>() : 0));
}

int attention_partial_tc64(const void *Q, int nseq, const void *const *caches, const int *n_rows, const int *rows_per_split, int nsplit,
                           int cluster, AttnPartials part, int slot_stride, float scale, cudaStream_t stream, bool programmatic_launch,
                           L2Prefetch prefetch)
{
    if (nseq < 1 || nseq > kMaxBatch || nsplit < 1) return NM_ERR_UNSUPPORTED;
    if (cluster != 1 && cluster != 2 && cluster != 4) return NM_ERR_UNSUPPORTED;
    if ((uintptr_t)Q & 15u) return NM_ERR_UNSUPPORTED;
    CUtensorMap map_q;
    AttnSeqs64 seqs{};
    seqs.ml_stride = (long)slot_stride * kHeads * 2;
    seqs.o_stride = (long)slot_stride * kHeads * kDv;
    if (!encode_rows_map64(&map_q, Q, nseq * kHeads, kHeadsCta)) return NM_ERR_UNSUPPORTED;
    for (int t = 0; t < nseq; ++t) {
        seqs.n_rows[t] = n_rows[t];
        seqs.rows_per_split[t] = rows_per_split[t];
        if (n_rows[t] < 1) {                                       // nothing to attend: its CTAs find no tiles and load nothing
            seqs.kv[t] = map_q;
            seqs.rows_per_split[t] = kT;
            continue;
        }
        if (rows_per_split[t] % kT != 0) return NM_ERR_UNSUPPORTED;
        if ((uintptr_t)caches[t] & 15u) return NM_ERR_UNSUPPORTED;
        // the cache map covers exactly the rows attended: rows past n_rows read as zeros (and are masked)
        if (!encode_rows_map64(&seqs.kv[t], caches[t], n_rows[t], kT)) return NM_ERR_UNSUPPORTED;
    }
    if (cluster == 4) return launch_tc64<4>(map_q, seqs, nseq, nsplit, part, scale, stream, programmatic_launch, prefetch);
    if (cluster == 2) return launch_tc64<2>(map_q, seqs, nseq, nsplit, part, scale, stream, programmatic_launch, prefetch);
    return launch_tc64<1>(map_q, seqs, nseq, nsplit, part, scale, stream, programmatic_launch, prefetch);
}

}  // namespace nm
