// Narrow product with the roles of the operands swapped, on the tensor cores (bf16 B, either layout).
//
// For M above ~8 the CUDA-core kernel is bound by fp32 FMA issue, not by HBM (8*M FMAs per 16 bytes of
// weights against 128 FMA lanes per SM).  Here the weights take the MMA's M dimension and the token
// rows its N dimension:
//     D[128 columns of C x 16 tokens] += W[k-slab x 128 columns]^T * A[16 tokens x k-slab]^T
// so one tcgen05.mma (M=128, N=16, K=16) consumes 4 KB of weights, the tensor pipe idles most of the
// time, and the kernel is back on the HBM roofline for every M <= 16.  bf16 products are exact in
// fp32 and the accumulation is fp32, as on the CUDA-core path; the result is rounded once.
//
// Per CTA: one 128-column tile and one k-range.  A producer thread streams [64 k-rows x 128 columns]
// boxes of B (two 128-byte-swizzled TMA boxes: the k-slab is the MMA's MN-major A operand as it lies)
// and the matching [16 tokens x 64 k] box of A into a ring; one thread issues four MMAs per stage and
// commits the stage back to the producer; four warps read the 128 x 16 accumulator from TMEM at the
// end and write C (or the split-K partial tile, completed by the arrival counter as in the other
// kernels).  Weights are fetched before the programmatic-launch wait, tokens after.
//
// Column-major B ([N][K], k contiguous) is the same kernel with the weight operand K-major: one
// [128 columns of C x 64 k] box per stage (128-byte swizzle), the descriptor advanced 32 bytes per k-step.
#include <type_traits>

#include "nm_matmul_kernels.cuh"
#include "nm_row_tc.cuh"
#include "nm_tcgen05.cuh"

namespace nm {

namespace {

constexpr int kTcThreads = 192;
constexpr int kBStage = kTcKT * kTcTN * 2;         // 16 KB of weights per stage

// kTok: token columns of the accumulator (the MMA's N): 16 for M <= 16, 32 or 64 for more tokens than the narrow
// range proper - the weights are still streamed once, the tokens padded to the next size.
template <typename TO, bool kCol, int kTok>
__global__ void __launch_bounds__(kTcThreads, kTok == 16 ? 4 : 2)
nm_row_tc_kernel(const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_a, const TmaArgs ta)
{
    constexpr int kAStage = kTok * kTcKT * 2;      // 2 KB of tokens per stage at 16 tokens
    constexpr int kStage = kBStage + kAStage;
    constexpr uint32_t kTmemColsTc = kTok < 32 ? 32 : kTok;
    const MatmulArgs &a = ta.base;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    unsigned char *smem = smem_raw + (base - raw_addr);
    const int NS = ta.nstage;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)NS * kStage);
    const uint32_t full_b0 = smem_u32(bars), full_a0 = smem_u32(bars + NS), empty0 = smem_u32(bars + 2 * NS),
                   bar_done = smem_u32(bars + 3 * NS);
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort, s_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tile = blockIdx.x, split = blockIdx.y, h = blockIdx.z;
    const int M = a.M;
    const int kb = split * a.kr, ke = min(a.K, kb + a.kr);
    const int n_it = ceil_div(ke - kb, kTcKT);

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < NS; ++s) { mbar_init(full_b0 + 8 * s, 1); mbar_init(full_a0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(bar_done, 1);
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(&s_tmem_base, kTmemColsTc);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    pdl_launch_dependents();
    // Split-K inside a cluster (the k-splits of a tile are the CTAs of one cluster, see cluster_split_finish): first
    // half of a cluster barrier here, its second half before the first store into a peer's shared memory.
    if (ta.cluster_split) cluster_arrive_all();
    float *slots = reinterpret_cast<float *>(bars + 3 * NS + 2);  // [split][m][128 columns], used in the first CTA of the cluster

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_descriptor(&map_b);
            tma_prefetch_descriptor(&map_a);
            const uint64_t stream = l2_policy_evict_first(), keep = l2_policy_evict_last();
            auto load_b = [&](int it, int s) {
                const uint32_t dst = base + (uint32_t)s * kStage;
                mbar_arrive_expect_tx(full_b0 + 8 * s, kBStage);
                if constexpr (kCol) {
                    tma_load_3d(dst, &map_b, kb + it * kTcKT, tile * kTcTN, h, full_b0 + 8 * s, stream);
                } else {
                    tma_load_3d(dst, &map_b, tile * kTcTN, kb + it * kTcKT, h, full_b0 + 8 * s, stream);
                    tma_load_3d(dst + kBStage / 2, &map_b, tile * kTcTN + 64, kb + it * kTcKT, h, full_b0 + 8 * s, stream);
                }
            };
            auto load_a = [&](int it, int s) {
                mbar_arrive_expect_tx(full_a0 + 8 * s, kAStage);
                tma_load_3d(base + (uint32_t)s * kStage + kBStage, &map_a, kb + it * kTcKT, 0, h, full_a0 + 8 * s, keep);
            };
            // weights do not depend on earlier kernels: fill the ring before waiting for them
            const int pre = min(NS, n_it);
            for (int it = 0; it < pre; ++it) load_b(it, it);
            pdl_wait_prior_grids();
            for (int it = 0; it < pre; ++it) load_a(it, it);
            int s = 0;
            uint32_t ph = 0;
            for (int it = NS; it < n_it; ++it) {
                if (!mbar_try_wait(empty0 + 8 * s, ph) && !mbar_wait(empty0 + 8 * s, ph, &s_abort, ta.status)) break;
                load_b(it, s);
                load_a(it, s);
                if (++s == NS) { s = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // fp16 output means fp16 operands (the optional element type); bf16 operands otherwise
            constexpr uint32_t idesc = std::is_same<TO, f16_t>::value ? instr_desc_f16(128, kTok, !kCol, false) : instr_desc(128, kTok, !kCol, false);
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < n_it; ++it) {
                if (!mbar_try_wait(full_b0 + 8 * s, ph)) mbar_wait(full_b0 + 8 * s, ph, &s_abort, ta.status);
                if (!mbar_try_wait(full_a0 + 8 * s, ph)) mbar_wait(full_a0 + 8 * s, ph, &s_abort, ta.status);
                tc_fence_after();
                const uint32_t sb = base + (uint32_t)s * kStage, sa = sb + kBStage;
#pragma unroll
                for (int kk = 0; kk < kTcKT / 16; ++kk)
                    mma_ss(tmem, kCol ? smem_desc(sb + kk * 32, 16, 1024) : smem_desc(sb + kk * 2048, kBStage / 2, 1024),
                           smem_desc(sa + kk * 32, 16, 1024), idesc, (it | kk) != 0);
                mma_commit(empty0 + 8 * s);                       // the stage is free once these MMAs have read it
                if (++s == NS) { s = 0; ph ^= 1; }
            }
            mma_commit(bar_done);
        }
    }

    // ---- epilogue: 128 accumulator rows (columns of C) x 16 tokens ------------------------------------------
    uint32_t slot0 = 0;
    if (ta.cluster_split) {
        __syncwarp();
        cluster_wait_all();
        slot0 = cluster_slot_base(slots, split, M * kTcTN);
    }
    if (warp >= 2) {
        const int quad = warp & 3, c = quad * 32 + lane;          // column of the tile held by this thread
        if (n_it > 0) {
            mbar_wait(bar_done, 0, &s_abort, ta.status);
            tc_fence_after();
        }
        uint32_t d[kTok];
#pragma unroll
        for (int j = 0; j < kTok / 16; ++j) {
            uint32_t part[16];
            tmem_ld16(tmem + ((uint32_t)(quad * 32) << 16) + 16 * j, part);
#pragma unroll
            for (int i = 0; i < 16; ++i) d[16 * j + i] = part[i];
        }
        tmem_wait_ld();
        const int n = tile * kTcTN + c;
        pdl_wait_prior_grids();                                   // nothing is written before earlier kernels are done
        if (a.nsplit == 1) {
            TO *C = (TO *)a.C + (long)h * a.strideC;
            if (n < a.N)
#pragma unroll
                for (int m = 0; m < kTok; ++m)
                    if (m < M) NM_ST(&C[(long)m * a.ldc + n], round_out<TO>(n_it > 0 ? __uint_as_float(d[m]) : 0.f), span_of_C<TO>(a), ta.status);
        } else if (ta.cluster_split) {
#pragma unroll
            for (int m = 0; m < kTok; ++m)
                if (m < M) cluster_slot_store(slot0, m * kTcTN + c, n_it > 0 ? __uint_as_float(d[m]) : 0.f);
        } else {
            float *P = a.partial + (((size_t)h * a.ntiles + tile) * a.nsplit + split) * (size_t)(M * kTcTN);
#pragma unroll
            for (int m = 0; m < kTok; ++m)
                if (m < M) NM_ST(&P[(size_t)m * kTcTN + c], n_it > 0 ? __uint_as_float(d[m]) : 0.f, span_of_partials(a), ta.status);
        }
    }
    tc_fence_before();
    if (ta.cluster_split) {
        __syncwarp();
        cluster_split_finish<TO>(a, slots, M, tile, split, h);    // cluster barrier, then the first CTA adds the slots
        __syncthreads();
    } else if (a.nsplit > 1) {
        splitk_complete_rt<TO>(a, M, tile, h, &s_last);
    } else {
        __syncthreads();
    }
    if (s_abort && tid == 0)
        for (int s = 0; s < NS && s < n_it; ++s)
            for (int i = 0; i < (1 << 14) && !mbar_try_wait(full_b0 + 8 * s, 0); ++i) {}
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemColsTc);
    }
}

}  // namespace

int row_tc_tokens(int M) { return M <= 16 ? 16 : (M <= 32 ? 32 : 64); }
size_t row_tc_smem_bytes(int nstage, size_t slot_bytes, int tokens)
{
    return (size_t)nstage * (kBStage + tokens * kTcKT * 2) + (3 * nstage + 1) * sizeof(uint64_t) + 16 + slot_bytes + 1024;
}

template <typename TO, bool kCol, int kTok>
static cudaError_t launch_tc(const CUtensorMap &map_b, const CUtensorMap &map_a, const TmaArgs &ta_in, cudaStream_t s)
{
    TmaArgs ta = ta_in;
    const MatmulArgs &a = ta.base;
    static std::atomic<unsigned long long> configured{0};          // per instantiation, one bit per device
    auto kern = nm_row_tc_kernel<TO, kCol, kTok>;
    {
        cudaError_t e = ensure_dynamic_smem(kern, 200 * 1024, configured);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.ntiles, a.nsplit, a.H);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = row_tc_smem_bytes(ta.nstage, ta.cluster_split ? (size_t)a.nsplit * a.M * kTcTN * sizeof(float) : 0, kTok);
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
    if (ta.cluster_split && !clusters_fit_one_wave(kern, cfg, (unsigned)a.nsplit, (long)a.ntiles * a.H)) {
        ta.cluster_split = 0;                                      // through the workspace instead (the caller provided it)
        cfg.dynamicSmemBytes = row_tc_smem_bytes(ta.nstage, 0, kTok);
        cfg.numAttrs = na - 1;                                     // the cluster attribute is the last one
    }
    return cudaLaunchKernelEx(&cfg, kern, map_b, map_a, ta);
}

// How many clusters of `cluster_size` CTAs of this kernel (ring of `nstage` stages, slots for M tokens) the GPU holds
// at once; 0 when it cannot be asked (no device).  The planner sizes the k-split with it.
template <typename TO, bool kCol, int kTok>
static int max_clusters_tc(int cluster_size, int nstage, int M)
{
    auto kern = nm_row_tc_kernel<TO, kCol, kTok>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, cluster_size, 1);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = row_tc_smem_bytes(nstage, (size_t)cluster_size * M * kTcTN * sizeof(float), kTok);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = (unsigned)cluster_size; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return max_clusters_cached(kern, cfg, (unsigned)cluster_size);
}

template <typename TO, bool kCol>
static int max_clusters_by_tokens(int cluster_size, int nstage, int M)
{
    switch (row_tc_tokens(M)) {
    case 16: return max_clusters_tc<TO, kCol, 16>(cluster_size, nstage, M);
    case 32: return max_clusters_tc<TO, kCol, 32>(cluster_size, nstage, M);
    default: return max_clusters_tc<TO, kCol, 64>(cluster_size, nstage, M);
    }
}

int row_tc_max_clusters(int cluster_size, int nstage, int M, bool col_major, bool f32_out)
{
    if (col_major) return f32_out ? max_clusters_by_tokens<float, true>(cluster_size, nstage, M) : max_clusters_by_tokens<bf16_t, true>(cluster_size, nstage, M);
    return f32_out ? max_clusters_by_tokens<float, false>(cluster_size, nstage, M) : max_clusters_by_tokens<bf16_t, false>(cluster_size, nstage, M);
}

template <typename TO, bool kCol>
static cudaError_t launch_by_tokens(const CUtensorMap &map_b, const CUtensorMap &map_a, const TmaArgs &ta, cudaStream_t s)
{
    switch (row_tc_tokens(ta.base.M)) {
    case 16: return launch_tc<TO, kCol, 16>(map_b, map_a, ta, s);
    case 32: return launch_tc<TO, kCol, 32>(map_b, map_a, ta, s);
    default: return launch_tc<TO, kCol, 64>(map_b, map_a, ta, s);
    }
}

template <typename TO>
cudaError_t launch_row_tc(const CUtensorMap &map_b, const CUtensorMap &map_a, const TmaArgs &ta, cudaStream_t s, bool col_major)
{
    return col_major ? launch_by_tokens<TO, true>(map_b, map_a, ta, s) : launch_by_tokens<TO, false>(map_b, map_a, ta, s);
}

template cudaError_t launch_row_tc<bf16_t>(const CUtensorMap &, const CUtensorMap &, const TmaArgs &, cudaStream_t, bool);
template cudaError_t launch_row_tc<float>(const CUtensorMap &, const CUtensorMap &, const TmaArgs &, cudaStream_t, bool);
template cudaError_t launch_row_tc<f16_t>(const CUtensorMap &, const CUtensorMap &, const TmaArgs &, cudaStream_t, bool);

}  // namespace nm
