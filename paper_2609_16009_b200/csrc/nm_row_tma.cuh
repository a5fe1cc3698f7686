// Row-major narrow product with a TMA-fed shared-memory ring (bf16 weights).
//
// One producer thread streams [KT x TN] boxes of B into a ring of NS stages with tiled TMA copies
// (cp.async.bulk.tensor, completion on an mbarrier, L2 evict-first: every weight byte is used
// once).  Eight consumer warps read the stage with 16-byte shared loads - each thread owns eight
// consecutive columns of C for all M rows - and accumulate in fp32 with packed two-wide FMAs
// (fma.rn.f32x2) whose pairs run along m.  The token rows A are kept in shared memory as
// fp32 [k][m], one chunk at a time; the next chunk is fetched into registers while the current one
// is in use.  The ring decouples the bytes in flight from the register budget, which is what lets
// one SM keep tens of kilobytes of HBM reads outstanding for every M.
//
// Split-K, partial sums and the arrival-counter gather are shared with the other kernels
// (Algorithm 1: compute stage, Partial Sum Buffer, gather stage).
#pragma once

#include "nm_async.cuh"
#include "nm_matmul_kernels.cuh"

namespace nm {

constexpr int kTmaConsumers = 256;
constexpr int kTmaThreads = kTmaConsumers + 32;
constexpr int kAChunkFloats = 4096;                       // 16 KB of A as fp32 [k][m]

template <int TPR> struct TmaTile {
    static constexpr int kTN = TPR * 8;                    // columns per CTA
    static constexpr int kRG = kTmaConsumers / TPR;        // row groups
    static constexpr int kRPT = 4;                         // rows per thread per stage
    static constexpr int kKT = kRG * kRPT;                 // k-rows per stage: 128 / 64 / 32
    static constexpr int kStageBytes = kKT * kTN * 2;      // always 16 KB
};

template <int M> struct TmaCfg {
    static constexpr int kMP = (M == 1) ? 1 : ((M + 1) / 2) * 2;     // m padded to a pair
    static constexpr int kPairs = kMP / 2;
    static constexpr int kMinBlocks = (M <= 8) ? 2 : 1;
    static constexpr int kPass = (kMP < 4) ? kMP : 4;
};

template <int M, int TPR, typename TO>
__global__ void __launch_bounds__(kTmaThreads, TmaCfg<M>::kMinBlocks)
nm_row_tma_kernel(const __grid_constant__ CUtensorMap tmap, const TmaArgs ta)
{
    using T = TmaTile<TPR>;
    using Cfg = TmaCfg<M>;
    constexpr int TN = T::kTN, RG = T::kRG, KT = T::kKT, RPT = T::kRPT, STAGE = T::kStageBytes;
    constexpr int MP = Cfg::kMP, MP2 = Cfg::kPairs, MPASS = Cfg::kPass;
    constexpr int KCH = ((kAChunkFloats / MP) / KT) * KT;            // k-rows of A per chunk
    constexpr int ITS_PER_CHUNK = KCH / KT;
    constexpr int GROUPS = (KCH / 8) * M;                            // 16-byte groups of A per chunk
    constexpr int GPT = (GROUPS + kTmaConsumers - 1) / kTmaConsumers; // groups per consumer thread
    const MatmulArgs &a = ta.base;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char *ring = smem_raw;
    // FRACTAL_NZ: a stage arrives as TN/16 fractal columns of [KT rows][16 columns] (KT * 32 bytes each)
    constexpr int NZ_COL = KT * 32;
    constexpr uint32_t stage_stride = STAGE;
    float *As = reinterpret_cast<float *>(smem_raw + (size_t)ta.nstage * stage_stride);
    uint64_t *bars = reinterpret_cast<uint64_t *>(As + kAChunkFloats);
    __shared__ int s_last;
    __shared__ int s_abort;
    __shared__ int s_issued;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, split = blockIdx.y, h = blockIdx.z;
    const int NS = ta.nstage;
    const int kb = split * a.kr;
    const int ke = min(a.K, kb + a.kr);
    const int n_it = ceil_div(ke - kb, KT);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + NS);
    unsigned long long *trace = ta.trace ? ta.trace + 4 * (((size_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x) : nullptr;

    if (tid == 0) {
        if (trace) trace[0] = global_timer_ns();
        s_abort = 0;
        s_issued = 0;
        for (int s = 0; s < NS; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, kTmaConsumers / 32);
        }
        mbar_init_fence();
    }
    __syncthreads();
    pdl_launch_dependents();
    // Split-K inside a cluster: first half of a cluster barrier; once its second half has been waited for (before
    // the partial sums are pushed) every peer is running, which writing into a peer's shared memory requires.
    if (ta.cluster_split) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

    float2 acc[MP2 > 0 ? MP2 : 1][8];
    float acc1[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        acc1[j] = 0.f;
#pragma unroll
        for (int p = 0; p < (MP2 > 0 ? MP2 : 1); ++p) acc[p][j] = make_float2(0.f, 0.f);
    }

    if (warp == kTmaConsumers / 32) {
        // ---------------- producer: weights never depend on an earlier kernel, so start at once ----
        if (lane == 0) {
            tma_prefetch_descriptor(&tmap);
            const uint64_t policy = l2_policy_evict_first();
            int it = 0, s = 0;
            uint32_t ph = 1;                                   // parity of the "previous" phase of an empty barrier
#pragma unroll 1
            for (; it < n_it; ++it) {
                if (it >= NS && !mbar_try_wait(empty0 + 8 * s, ph) && !mbar_wait(empty0 + 8 * s, ph, &s_abort, ta.status)) break;
                mbar_arrive_expect_tx(full0 + 8 * s, STAGE);
                if (ta.fractal_nz) {    // coordinates: element in fractal, fractal row, fractal column, head
                    tma_load_4d(smem_u32(ring + (size_t)s * stage_stride), &tmap, 0, (kb + it * KT) / 16, tile * (TN / 16), h, full0 + 8 * s, policy);
                } else {
                    tma_load_3d(smem_u32(ring + (size_t)s * stage_stride), &tmap, tile * TN, kb + it * KT, h, full0 + 8 * s, policy);
                }
                if (++s == NS) { s = 0; ph ^= 1; }
            }
            s_issued = it;
        }
    } else {
        // ---------------- consumers ---------------------------------------------------------------
        const int tx = tid % TPR, ty_plain = tid / TPR;
        // FRACTAL_NZ: the eight threads that read together hold four fractal columns, whose rows alias in the shared-memory
        // banks; fractal column g therefore takes the rows of every group of four in the order rotated by g
        const int ty = ta.fractal_nz ? ((ty_plain & ~3) | ((ty_plain + (tx >> 1)) & 3)) : ty_plain;
        const bf16_t *__restrict__ A = (const bf16_t *)a.A + (long)h * a.strideA;
        if constexpr (M == 1 && sizeof(TO) == 2) {
            // whichever CTA ends up running the vector stages wants their constants in L2 by then
            if (ta.tail.enabled) {
                if (ta.tail.q_lora > 0 && tid * 64 < ta.tail.q_lora) asm volatile("prefetch.global.L2 [%0];" ::"l"(ta.tail.gamma_q + tid * 64));
                if (ta.tail.dc > 0 && tid * 64 < ta.tail.dc) asm volatile("prefetch.global.L2 [%0];" ::"l"(ta.tail.gamma_kv + tid * 64));
                if (ta.tail.dc > 0 && tid * 32 < ta.tail.rope) asm volatile("prefetch.global.L2 [%0];" ::"l"(ta.tail.cos_sin + tid * 32));
            }
        }
        if (MP != M)
            for (int i = tid; i < kAChunkFloats; i += kTmaConsumers) As[i] = 0.f;
        if constexpr (M == 1 && sizeof(TO) == 2) {
            // the RMSNorm weights are read once per step and are long gone from L2: ask for them before the wait
            if (ta.norm.enabled && tid * 64 < ta.norm.n) asm volatile("prefetch.global.L2 [%0];" ::"l"(ta.norm.gamma + tid * 64));
        }
        pdl_wait_prior_grids();                       // A (and the workspace) come from earlier kernels

        constexpr bool kCanNorm = (M == 1 && sizeof(TO) == 2);
        const bool norm_on = kCanNorm && ta.norm.enabled;
        uint4 apre[GPT];
        uint4 gpre[kCanNorm ? GPT : 1];
        float rnorm = 1.f;
        int norm_k0 = 0;                              // first k of the chunk held in apre
        auto fetch_chunk = [&](int kc) {              // global -> registers
            norm_k0 = kc;
#pragma unroll
            for (int g = 0; g < GPT; ++g) {
                const int grp = tid + g * kTmaConsumers;
                const int m = grp % M, kg = grp / M;
                const int k = kc + kg * 8;
                uint4 v = make_uint4(0, 0, 0, 0);
                if constexpr (kCanNorm) {
                    if (norm_on) gpre[g] = (grp < GROUPS && k + 8 <= a.K) ? __ldg(reinterpret_cast<const uint4 *>(ta.norm.gamma + k)) : make_uint4(0, 0, 0, 0);
                }
                if (grp < GROUPS && k < ke) {
                    const bf16_t *src = A + (long)m * a.lda + k;
                    if (k + 8 <= a.K) {
                        v = NM_LDG16(reinterpret_cast<const uint4 *>(src), span_of_A<bf16_t>(a), ta.status);
                    } else {
                        uint16_t e[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) e[i] = (k + i < a.K) ? NM_LD(&src[i], span_of_A<bf16_t>(a), ta.status).bits : (uint16_t)0;
                        v.x = e[0] | ((uint32_t)e[1] << 16); v.y = e[2] | ((uint32_t)e[3] << 16);
                        v.z = e[4] | ((uint32_t)e[5] << 16); v.w = e[6] | ((uint32_t)e[7] << 16);
                    }
                }
                apre[g] = v;
            }
        };
        auto store_chunk = [&]() {                    // registers -> As[k][m] as fp32
#pragma unroll
            for (int g = 0; g < GPT; ++g) {
                const int grp = tid + g * kTmaConsumers;
                if (grp < GROUPS) {
                    const int m = grp % M, kg = grp / M;
                    float f[8];
                    Elem<bf16_t>::unpack(apre[g], f);
                    if constexpr (kCanNorm) {
                        if (norm_on) {                               // x * r * gamma, rounded to bf16 as a stored row would be
                            float gm[8];
                            Elem<bf16_t>::unpack(gpre[g], gm);
                            uint4 o;
                            o.x = pack2_bf16_rn(f[0] * rnorm * gm[0], f[1] * rnorm * gm[1]); o.y = pack2_bf16_rn(f[2] * rnorm * gm[2], f[3] * rnorm * gm[3]);
                            o.z = pack2_bf16_rn(f[4] * rnorm * gm[4], f[5] * rnorm * gm[5]); o.w = pack2_bf16_rn(f[6] * rnorm * gm[6], f[7] * rnorm * gm[7]);
                            Elem<bf16_t>::unpack(o, f);
                            if (ta.norm.normed_out && (blockIdx.x | blockIdx.z) == 0 && norm_k0 + kg * 8 < ke)     // this split's rows only
                                *reinterpret_cast<uint4 *>(ta.norm.normed_out + norm_k0 + kg * 8) = o;
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) As[(kg * 8 + i) * MP + m] = f[i];
                }
            }
        };
        if (MP != M) named_barrier_sync(1, kTmaConsumers);
        fetch_chunk(kb);
        if constexpr (kCanNorm) {
            if (norm_on) {
                // 1 / rms of the row from the per-tile sums of squares, added in tile order by every warp for itself
                const float v = (lane < ta.norm.ntiles) ? ld_cg(ta.norm.tile_ss + lane) : 0.f;
                float tot = 0.f;
                for (int l = 0; l < ta.norm.ntiles; ++l) tot += __shfl_sync(0xffffffffu, v, l);
                rnorm = 1.0f / sqrtf(tot / (float)ta.norm.n + ta.norm.eps);
            }
        }
        store_chunk();
        named_barrier_sync(1, kTmaConsumers);
        if (trace && tid == 0) trace[1] = global_timer_ns();
        if (n_it > ITS_PER_CHUNK) fetch_chunk(kb + KCH);

        const int rows_last = (ke - kb) - (n_it - 1) * KT;            // rows in the last stage (1..KT)
        // this thread's first row in a stage and the distance between its rows; a FRACTAL_NZ stage is a row of
        // fractal columns, each [KT rows][16 columns]: the thread's eight columns are half of one fractal row
        const uint32_t boff = ta.fractal_nz ? (uint32_t)((tx >> 1) * NZ_COL + ty * 32 + (tx & 1) * 16) : (uint32_t)(ty * TN + tx * 8) * 2;
        const uint32_t rstride = ta.fractal_nz ? (uint32_t)RG * 32u : (uint32_t)RG * TN * 2u;
        const float *a_thread = As + ty * MP;
        auto do_row = [&](const unsigned char *stage, const float *ak, int i) {
            const uint4 v = *reinterpret_cast<const uint4 *>(stage + (size_t)i * rstride);
            float b[8];
            Elem<bf16_t>::unpack(v, b);
            const float *aki = ak + i * RG * MP;
            if constexpr (M == 1) {
                const float am = aki[0];
#pragma unroll
                for (int j = 0; j < 8; ++j) acc1[j] = fmaf(am, b[j], acc1[j]);
            } else if constexpr (MP % 4 == 0) {
#pragma unroll
                for (int q = 0; q < MP / 4; ++q) {
                    const float4 a4 = *reinterpret_cast<const float4 *>(aki + 4 * q);
                    const float2 lo = make_float2(a4.x, a4.y), hi = make_float2(a4.z, a4.w);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float2 bb = make_float2(b[j], b[j]);
                        acc[2 * q][j] = __ffma2_rn(lo, bb, acc[2 * q][j]);
                        acc[2 * q + 1][j] = __ffma2_rn(hi, bb, acc[2 * q + 1][j]);
                    }
                }
            } else {
#pragma unroll
                for (int p = 0; p < MP2; ++p) {
                    const float2 am = *reinterpret_cast<const float2 *>(aki + 2 * p);
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[p][j] = __ffma2_rn(am, make_float2(b[j], b[j]), acc[p][j]);
                }
            }
        };
        int s = 0, itc = 0;
        uint32_t ph = 0;
#pragma unroll 1
        for (int it = 0; it < n_it; ++it) {
            if (itc == ITS_PER_CHUNK) {
                itc = 0;
                named_barrier_sync(1, kTmaConsumers);                 // everyone is done with the old chunk
                store_chunk();
                named_barrier_sync(1, kTmaConsumers);
                if (it + ITS_PER_CHUNK < n_it) fetch_chunk(kb + (it + ITS_PER_CHUNK) * KT);
            }
            if (!mbar_try_wait(full0 + 8 * s, ph)) mbar_wait(full0 + 8 * s, ph, &s_abort, ta.status);
            const unsigned char *stage = ring + (size_t)s * stage_stride + boff;
            const float *ak = a_thread + itc * (KT * MP);
            if (it + 1 < n_it || rows_last == KT) {
#pragma unroll
                for (int i = 0; i < RPT; ++i) do_row(stage, ak, i);
            } else {
#pragma unroll
                for (int i = 0; i < RPT; ++i)
                    if (ty + i * RG < rows_last) do_row(stage, ak, i);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * s);
            ++itc;
            if (++s == NS) { s = 0; ph ^= 1; }
        }
    }

    // ---- all 288 threads: reduce the row groups through shared memory (the ring is free now) ------
    __syncthreads();
    if (trace && tid == 0) trace[2] = global_timer_ns();
    if (s_abort) {
        // A wait expired.  Give copies that were issued a bounded chance to land before the CTA exits.
        if (tid == 0) {
            const int issued = s_issued;
            for (int it = max(0, issued - NS); it < issued; ++it)
                for (int i = 0; i < (1 << 16) && !mbar_try_wait(full0 + 8 * (it % NS), (it / NS) & 1); ++i) {}
        }
        __syncthreads();
    }
    float *red = reinterpret_cast<float *>(ring);
    const int tx = tid % TPR, ty = tid / TPR;
    TO *C = (TO *)a.C + (long)h * a.strideC;
    float *P = a.partial ? a.partial + (((size_t)h * a.ntiles + tile) * a.nsplit + split) * (size_t)(M * TN) : nullptr;
    // cluster split-K: slot [split][m][c] in the shared memory of the cluster's first CTA, behind its barriers
    float *slots = reinterpret_cast<float *>(bars + 2 * NS + 2);
    uint32_t slot0 = 0;
    if (ta.cluster_split) {
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(slot0) : "r"(smem_u32(slots + (size_t)split * (M * TN))), "r"(0));
    }
#pragma unroll
    for (int m0 = 0; m0 < M; m0 += MPASS) {
        if (m0 > 0) __syncthreads();
        if (tid < kTmaConsumers) {
#pragma unroll
            for (int mm = 0; mm < MPASS; ++mm) {
                const int m = m0 + mm;
                if (m < M) {
                    float vals[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if constexpr (M == 1) vals[j] = acc1[j];
                        else vals[j] = (m & 1) ? acc[m / 2][j].y : acc[m / 2][j].x;
                    }
                    float4 *dst = reinterpret_cast<float4 *>(red + (size_t)(ty * MPASS + mm) * TN + tx * 8);
                    dst[0] = make_float4(vals[0], vals[1], vals[2], vals[3]);
                    dst[1] = make_float4(vals[4], vals[5], vals[6], vals[7]);
                }
            }
        }
        __syncthreads();
        for (int i = tid; i < MPASS * TN; i += kTmaThreads) {
            const int mm = i / TN, c = i - mm * TN, m = m0 + mm, n = tile * TN + c;
            if (m < M && n < a.N) {
                float s = 0.f;
#pragma unroll 8
                for (int g = 0; g < RG; ++g) s += red[(size_t)(g * MPASS + mm) * TN + c];
                if (a.nsplit == 1) NM_ST(&C[(long)m * a.ldc + n], round_out<TO>(s), span_of_C<TO>(a), ta.status);
                else if (ta.cluster_split) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(slot0 + (uint32_t)(m * TN + c) * 4u), "f"(s) : "memory");
                else               NM_ST(&P[(size_t)m * TN + c], s, span_of_partials(a), ta.status);
            }
        }
    }
    if constexpr (M == 1 && sizeof(TO) == 2) {
        if (ta.tail.enabled) {
            tail_complete(a, ta.tail, &s_last, reinterpret_cast<float *>(ring), ta.trace ? ta.trace + 4 * 160 : nullptr);
            if (trace && tid == 0) trace[3] = global_timer_ns();
            return;
        }
    }
    if (ta.cluster_split) {
        // every split's sums are in the first CTA's slots once the cluster barrier completes; that CTA adds them
        // in split order and rounds once (no fence, counter or gather through L2)
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (split == 0) {
            float sq = 0.f;                                        // M = 1, TN <= 256: at most one output per thread
            for (int i = tid; i < M * TN; i += kTmaThreads) {
                const int m = i / TN, c = i - m * TN, n = tile * TN + c;
                if (n < a.N) {
                    float s = 0.f;
                    for (int sp = 0; sp < a.nsplit; ++sp) s += slots[(size_t)sp * (M * TN) + i];
                    const TO r = round_out<TO>(s);
                    NM_ST(&C[(long)m * a.ldc + n], r, span_of_C<TO>(a), ta.status);
                    if constexpr (M == 1 && sizeof(TO) == 2) { const float rv = Elem<bf16_t>::widen(r); sq = rv * rv; }
                }
            }
            if constexpr (M == 1 && sizeof(TO) == 2) {
                if (ta.tile_ss) {                                  // sum of squares of the tile's rounded outputs, fixed order
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                    float *scr = reinterpret_cast<float *>(ring);
                    if (lane == 0) scr[warp] = sq;
                    __syncthreads();
                    if (tid == 0) {
                        float t = 0.f;
                        for (int w = 0; w < kTmaThreads / 32; ++w) t += scr[w];
                        ta.tile_ss[tile] = t;
                    }
                }
            }
        }
        if (trace && tid == 0) trace[3] = global_timer_ns();
        return;
    }
    if (a.nsplit > 1) splitk_complete<M, TO>(a, tile, h, &s_last);
    if (trace && tid == 0) trace[3] = global_timer_ns();
}

template <int TPR, typename TO>
cudaError_t launch_row_tma(const CUtensorMap &tmap, const TmaArgs &ta_in, size_t smem_bytes, cudaStream_t s, bool query_only)
{
    TmaArgs ta = ta_in;
    const MatmulArgs &a = ta.base;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.ntiles, a.nsplit, a.H);
    cfg.blockDim = dim3(kTmaThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (ta.use_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (ta.cluster_split) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 1; attr[na].val.clusterDim.y = (unsigned)a.nsplit; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    switch (a.M) {
#define NM_X(m)                                                                                           \
    case m: {                                                                                             \
        auto kern = nm_row_tma_kernel<m, TPR, TO>;                                                        \
        static std::atomic<unsigned long long> configured{0};       /* per launch site, one bit per device */ \
        {                                                                                                 \
            cudaError_t e = ensure_dynamic_smem(kern, 200 * 1024, configured);                            \
            if (e != cudaSuccess) return e;                                                               \
        }                                                                                                 \
        /* clusters that would need a second wave: through the workspace instead (query_only: just say so) */ \
        const bool fits = !ta.cluster_split || clusters_fit_one_wave(kern, cfg, (unsigned)a.nsplit, (long)a.ntiles * a.H); \
        if (query_only) return fits ? cudaSuccess : cudaErrorLaunchOutOfResources;                       \
        if (!fits && !ta.tile_ss && a.partial) {     /* the per-tile sums of squares exist on the cluster path only */ \
            ta.cluster_split = 0;                                                                         \
            cfg.numAttrs = na - 1;                                                                        \
        }                                                                                                 \
        return cudaLaunchKernelEx(&cfg, kern, tmap, ta);                                                  \
    }
        NM_FOR_EACH_M(NM_X)
#undef NM_X
    default: return cudaErrorInvalidValue;
    }
}

#define NM_INSTANTIATE_TMA(TPR, TO) \
    template cudaError_t launch_row_tma<TPR, TO>(const CUtensorMap &, const TmaArgs &, size_t, cudaStream_t, bool);
#define NM_EXTERN_TMA(TPR, TO) \
    extern template cudaError_t launch_row_tma<TPR, TO>(const CUtensorMap &, const TmaArgs &, size_t, cudaStream_t, bool);

}  // namespace nm
