// Host side of the narrow matrix product: argument checks, tiling plan, launches, C-ABI entry points.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "nm_matmul_kernels.cuh"
#include "nm_row_tma.cuh"
#include "nm_row_tc.cuh"

namespace nm {

NM_EXTERN(row, bf16_t, bf16_t)
NM_EXTERN(row, bf16_t, float)
NM_EXTERN(row, float, float)
NM_EXTERN(col, bf16_t, bf16_t)
NM_EXTERN(col, bf16_t, float)
NM_EXTERN(row, f16_t, f16_t)
NM_EXTERN(col, f16_t, f16_t)
NM_EXTERN(col, float, float)
NM_EXTERN_TMA(8, bf16_t)
NM_EXTERN_TMA(8, float)
NM_EXTERN_TMA(16, bf16_t)
NM_EXTERN_TMA(16, float)
NM_EXTERN_TMA(32, bf16_t)
NM_EXTERN_TMA(32, float)

// ---- error bookkeeping ---------------------------------------------------------------------------
static thread_local char g_cuda_error[256] = "";

int record_cuda_error(cudaError_t e, const char *where)
{
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", where, cudaGetErrorString(e));
    return NM_ERR_CUDA;
}

// ---- default workspace and tuning overrides ----------------------------------------------------------
// Process-wide settings (nm_set_*, nm_debug_set_*), guarded by a mutex.  Every entry point copies them once at its
// start into a per-thread snapshot and plans from that copy alone, so a setter running on another host thread never
// yields a plan mixed from two settings (a tile width from one, a split count from the other).
struct MatmulTuning {
    void *ws = nullptr;             // default workspace of nm_matmul / nm_matmul_batched
    size_t ws_bytes = 0;
    int force_tn = 0, force_split = 0, force_kind = -1, force_stages = 0;
    int cluster_split = 1;          // k-splits of a tile as a thread-block cluster when the plan allows
    int use_pdl = 0;
    int tc_min_m = 3;               // row-major bf16 products with M >= this (and >= 32 MB of weights) go to the swap-AB tensor-core kernel
};
static std::mutex g_tuning_mutex;
// Environment, read once when the library is loaded: NM_FORCE_KERNEL (kernel family as nm_debug_set_kernel: 0 plain-load,
// 3 TMA ring, 4 swap-AB tensor cores), NM_STAGES (ring depth), NM_TILE_N and NM_SPLITK (as nm_debug_set_plan) give the
// tuning settings their initial values; NM_LOG=1 prints the plan of every product to stderr.
static int env_int(const char *name, int fallback, int lo, int hi)
{
    const char *v = getenv(name);
    if (!v || !*v) return fallback;
    const long x = strtol(v, nullptr, 10);
    return (x < lo || x > hi) ? fallback : (int)x;
}
static MatmulTuning tuning_from_environment()
{
    MatmulTuning t;
    t.force_kind = env_int("NM_FORCE_KERNEL", -1, -1, 4);
    t.force_stages = env_int("NM_STAGES", 0, 0, 16);
    t.force_tn = env_int("NM_TILE_N", 0, 0, kMaxTileN);
    t.force_split = env_int("NM_SPLITK", 0, 0, kMaxSplit);
    return t;
}
static MatmulTuning g_tuning_shared = tuning_from_environment();
static const bool g_log_plans = env_int("NM_LOG", 0, 0, 1) != 0;
struct PlanOverride { bool active = false; int tn = 0, split = 0, stages = 0; };
static thread_local PlanOverride g_plan_override;      // a plan forced for this thread's next products only
static thread_local MatmulTuning g_t;                  // the calling thread's snapshot

static void refresh_tuning()
{
    {
        std::lock_guard<std::mutex> lock(g_tuning_mutex);
        g_t = g_tuning_shared;
    }
    if (g_plan_override.active) { g_t.force_tn = g_plan_override.tn; g_t.force_split = g_plan_override.split; g_t.force_stages = g_plan_override.stages; }
}

void set_thread_plan_override(bool active, int tile_n, int nsplit, int stages)
{
    g_plan_override.active = active; g_plan_override.tn = tile_n; g_plan_override.split = nsplit; g_plan_override.stages = stages;
}

enum PlanKind { kRowVec = 0, kColVec = 1, kGeneric = 2, kRowTma = 3, kRowTc = 4 };

struct Plan {
    PlanKind kind;
    int tn, tpr, rg, nsplit, kr, ntiles, nstage;
};

static inline int elem_size(nm_dtype d) { return d == NM_F32 ? 4 : 2; }
static inline int vec_elems(nm_dtype d) { return 16 / elem_size(d); }
static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Pick the column tile and the number of k-splits.  The stream is HBM-bound, so the plan wants
// (a) enough CTAs to cover all 148 SMs a few times over, (b) per-CTA segments of B as long and as
// contiguous as the shape allows, (c) few enough splits that the partial-sum traffic stays a few
// per cent of |B|.
// Plan for the TMA-ring kernel, from measurements on B200 (sweeps over tile width, k-splits and ring
// depth for the decode step's shapes and the M-sweep shapes):
//  * 64-column tiles unless that makes more CTAs than are resident at once (then 128, then 256 columns);
//  * about one to two CTAs per SM in total: 256 for products of 32 MB and more, 160 below that
//    (each extra split costs a partial tile and lengthens the gather), 148 when M > 8 (one resident
//    CTA per SM);
//  * k-rows per split a multiple of the stage height, so that no TMA box straddles two splits;
//  * five 16 KB stages (two resident CTAs per SM), three when there are more CTAs than that, ten
//    when M > 8.
static Plan make_tma_plan(int M, int N, int K, int H, bool chained = false)
{
    Plan p{};
    p.kind = kRowTma;
    // Large single matrices with long columns: one CTA per SM, no k-split, an 8-stage ring (128 KB in flight per
    // SM).  Measured 4-10 % faster than two smaller CTAs per SM on every shape of 50-260 MB tried (6.2-6.5 TB/s),
    // provided the tiles fill most of the machine: at M = 2 a CTA is also bound by its own FMA rate, and 112
    // CTAs were too few.
    if (M <= 2 && H == 1 && g_t.force_tn == 0 && g_t.force_split == 0 && 2.0 * K * N >= 48e6 && K >= 4096) {
        for (int t = 64; t <= 256; t *= 2) {
            const int tiles = ceil_div(N, t);
            if (tiles <= kSMs && tiles >= (M == 1 ? 100 : 120)) {
                const int kt1 = (kTmaConsumers / (t / 8)) * 4;
                p.tn = t; p.tpr = t / 8; p.rg = kTmaConsumers / p.tpr; p.nsplit = 1; p.kr = ceil_div(K, kt1) * kt1; p.ntiles = tiles;
                p.nstage = g_t.force_stages > 0 ? (g_t.force_stages < 2 ? 2 : (g_t.force_stages > 11 ? 11 : g_t.force_stages)) : 8;
                return p;
            }
        }
    }
    int tn = 64;
    const long tile_cap = (M > 8) ? kSMs : 2 * kSMs;   // a single wave of resident CTAs (two per SM, one when M > 8)
    while ((long)ceil_div(N, tn) * H > tile_cap && tn < 256) tn *= 2;
    if (g_t.force_tn == 64 || g_t.force_tn == 128 || g_t.force_tn == 256) tn = g_t.force_tn;
    const int tpr = tn / 8;
    const int kt = (kTmaConsumers / tpr) * 4;
    const int ntiles = ceil_div(N, tn);
    const long base = (long)ntiles * H;
    const double total_bytes = 2.0 * K * N * H;
    const int target = (M > 8) ? kSMs : (total_bytes < 32e6 ? 160 : 256);
    int ns = (int)((target + base / 2) / base);
    if (ns > K / 128) ns = K / 128;
    if (ns > K / (40 * M)) ns = K / (40 * M);          // partial sums stay below ~10 % of the weight bytes
    // Up to eight splits meet inside a thread-block cluster (shared memory, no fence / counter / gather through L2);
    // measured on the 7168 x 576 product: 8 splits that way 5.4 us, the 14 this rule would take otherwise 7.3 us.
    if (g_t.cluster_split && M <= 8 && ns > 8) ns = 8;
    if (g_t.force_split > 0) ns = g_t.force_split;
    if (ns > kMaxSplit) ns = kMaxSplit;
    if (ns < 1) ns = 1;
    if (base > kNumCounters) ns = 1;
    int kr = ceil_div(ceil_div(K, ns), kt) * kt;
    if (g_t.force_split > 0) kr = ceil_div(ceil_div(K, ns), 8) * 8;      // forced plans keep the requested split count
    ns = ceil_div(K, kr);
    p.tn = tn; p.tpr = tpr; p.rg = kTmaConsumers / tpr; p.nsplit = ns; p.kr = kr; p.ntiles = ntiles;
    const long ctas = base * ns;
    int nstage = (M > 8) ? 10 : (ctas > 2 * kSMs ? 3 : 5);
    if (chained && M <= 2 && g_t.force_split == 0 && g_t.force_tn == 0) {
        // Launched programmatically inside a chain of kernels (the decode step): the CTAs are resident, and fill
        // their rings, while the previous kernel drains, so a deep ring is prefetch for free; and every split-K
        // gather at the end is a dependent round trip through L2 on the chain's critical path.  Measured in the
        // step: at most one CTA per SM with an 8-stage ring, no split once there are about 100 tiles.
        const int ns_c = base >= 96 ? 1 : (int)((kSMs * 9 / 10 + base / 2) / base);
        int ns2 = ns_c < 1 ? 1 : ns_c;
        if (ns2 > K / 128) ns2 = K / 128 > 0 ? K / 128 : 1;
        if (ns2 > kMaxSplit) ns2 = kMaxSplit;
        if (base * ns2 <= kSMs && base <= kNumCounters) {
            kr = ceil_div(ceil_div(K, ns2), kt) * kt;
            p.kr = kr; p.nsplit = ceil_div(K, kr);
            nstage = 8;
        }
    }
    if (g_t.force_stages > 0) nstage = g_t.force_stages;
    if (nstage < 2) nstage = 2;
    if (nstage > 11) nstage = 11;
    p.nstage = nstage;
    return p;
}

// Plan for the swap-AB tensor-core kernel: 128-column tiles, k-rows per split a multiple of the 64-row
// stage, about two CTAs per SM in total, five 18 KB stages.
static Plan make_tc_plan(int M, int N, int K, int H, bool col_major = false, bool f32_out = false)
{
    Plan p{};
    p.kind = kRowTc;
    p.tn = kTcTN; p.tpr = 0; p.rg = 0;
    p.ntiles = ceil_div(N, kTcTN);
    const long base = (long)p.ntiles * H;
    // one CTA per SM measured best for this kernel (its ring alone keeps 90 KB in flight per SM)
    int ns = (int)((kSMs + base / 2) / base);
    if (ns > K / 128) ns = K / 128;
    if (M <= NM_MAX_M) { if (ns > K / (40 * M)) ns = K / (40 * M); }     // partial sums stay below ~10 % of the weight bytes
    else if (ns > K / (8 * M)) ns = K / (8 * M);        // 17-64 tokens: up to ~40 %, or too few CTAs are left (small matrices)
    // Up to eight splits meet inside a cluster (64 KB of slots at M = 16) - when all the clusters are resident at
    // once: the CTAs of a cluster need SMs of one GPC, so fewer CTAs fit as clusters than one by one (15 clusters of
    // eight, 26 of five, 45 of three with one CTA per SM).  Take the largest split count whose clusters fit.
    // On matrices of 100 MB and more the streaming time dominates and fewer CTAs cost more than the gather saves
    // (235 MB at M = 16: 43.0 us as 168 CTAs through the workspace, 44.9 us as 56 clusters of two): no reduction there.
    if (g_t.cluster_split && g_t.force_split == 0 && ns >= 2 && 2.0 * K * N * H < 100e6 && M <= NM_MAX_M) {
        for (int c = ns < 8 ? ns : 8; c >= 2; --c)
            if (base <= row_tc_max_clusters(c, 5, M, col_major, f32_out)) { ns = c; break; }
    }
    if (g_t.force_split > 0) ns = g_t.force_split;
    if (ns > kMaxSplit) ns = kMaxSplit;
    if (ns < 1) ns = 1;
    if (base > kNumCounters) ns = 1;
    const int kr = ceil_div(ceil_div(K, ns), kTcKT) * kTcKT;
    p.kr = kr;
    p.nsplit = ceil_div(K, kr);
    // one CTA per SM on a large matrix: a deeper ring (measured +1.5 to 3 %); otherwise 90 KB, two CTAs fit an SM
    int nstage = (base * p.nsplit <= kSMs && 2.0 * K * N * H >= 48e6) ? 7 : 5;
    if (M > 16 && base * p.nsplit > kSMs) nstage = (M > 32) ? 4 : 5;      // 24 / 20 KB stages: two CTAs still share an SM
    const int its = ceil_div(kr, kTcKT);                // a ring deeper than the CTA's k-range only costs shared memory
    if (nstage > its) nstage = its;
    if (g_t.force_stages > 0) nstage = g_t.force_stages;
    if (nstage < 2) nstage = 2;
    if (nstage > 10) nstage = 10;
    p.nstage = nstage;
    return p;
}

static Plan make_plan(int M, int N, int K, int H, nm_dtype dtype, nm_layout layout, bool vec_ok, bool tma_ok, bool chained = false)
{
    // fp16 (the optional element type): the tensor-core kernel takes it, the TMA ring kernel (bf16 unpacking, fused bf16
    // stages) does not; its CUDA-core kernels pay a conversion per element, so the tensor cores take over from 8 MB on at every M
    const bool ring_ok = tma_ok && dtype != NM_F16;
    Plan p{};
    const int V = vec_elems(dtype);
    if (layout == NM_FRACTAL_NZ) {
        // fractal storage goes through the TMA ring kernel whatever M: its tiled copies read the fractals in place
        p = make_tma_plan(M, N, K, H, chained);
        const int kt = (kTmaConsumers / p.tpr) * 4;
        if (p.kr % kt) {                                   // forced split counts: whole stages per split all the same
            p.kr = ceil_div(p.kr, kt) * kt;
            p.nsplit = ceil_div(K, p.kr);
        }
        return p;
    }
    if (!vec_ok) {
        p.kind = kGeneric; p.tn = kThreads; p.ntiles = ceil_div(N, kThreads); p.nsplit = 1; p.kr = K;
        p.tpr = p.rg = 0;
        return p;
    }
    // Measured on B200: from M = 3 on, the CUDA-core kernel falls off the HBM roofline on large weight
    // matrices (fp32 FMA issue) while the tensor-core kernel stays on it; small matrices are
    // latency-bound either way and the CUDA-core kernel has the shorter fixed cost.
    // Thresholds from sweeps of both kernels over 8-34 MB matrices and the batched per-head shapes: from 16 MB
    // (8 MB when batched over heads) the tensor-core kernel wins from M = 3 on; at 8 MB in one matrix the two tie.
    const double wbytes = 2.0 * K * N * H;
    // Column-major weights: the CUDA-core column kernel is already behind at M = 2 from about 50 MB on (17 vs 14 us
    // on 75 MB).
    const int min_m = (layout == NM_COL_MAJOR && g_t.tc_min_m > 2 && g_t.tc_min_m <= NM_MAX_M) ? 2 : g_t.tc_min_m;
    // More than 16 tokens (up to 64): only the tensor-core kernel takes them, whatever the size of the matrix
    const bool tc_pays = M > NM_MAX_M || (dtype == NM_F16 && wbytes >= 8e6) ||
                         (M >= min_m && (wbytes >= 16e6 || (H > 1 && wbytes >= 8e6)) && (M >= g_t.tc_min_m || wbytes >= 48e6));
    if (tma_ok && (M > NM_MAX_M || (g_t.force_kind != kRowTma && (layout == NM_ROW_MAJOR || g_t.force_kind != kRowVec))) && (tc_pays || g_t.force_kind == kRowTc))
        return make_tc_plan(M, N, K, H, layout == NM_COL_MAJOR, dtype == NM_BF16_F32OUT);
    if (layout == NM_ROW_MAJOR && ring_ok) return make_tma_plan(M, N, K, H, chained);
    const int target = 192;                           // CTAs wanted in total (measured: 144-240 is the flat optimum)
    if (layout == NM_ROW_MAJOR) {
        p.kind = kRowVec;
        // threads per row: 8 -> 32 (128-byte to 512-byte row segments); wider when N is large
        int tpr = 8;
        const int chunks = N / V;
        if (chunks >= 32 * 64) tpr = 32;
        else if (chunks >= 16 * 24) tpr = 16;
        if (g_t.force_tn > 0) tpr = g_t.force_tn / V;
        if (tpr < 1) tpr = 1;
        if (tpr > kThreads) tpr = kThreads;
        p.tpr = tpr;
        p.tn = tpr * V;
        p.rg = kThreads / tpr;
    } else {
        p.kind = kColVec;
        p.tn = (M <= 4 ? 4 : 2) * (kThreads / 32);
        p.tpr = p.rg = 0;
    }
    p.ntiles = ceil_div(N, p.tn);
    int nsplit = 1;
    const long ctas = (long)p.ntiles * H;
    if (ctas < kSMs) nsplit = (int)((target + ctas / 2) / ctas);
    // keep at least ~64 k-rows (row kernel) / 512 k (column kernel) per split, and the partial sums
    // below ~10 % of the weight bytes
    const int min_kr = (p.kind == kRowVec) ? 2 * p.rg : 512;
    if (nsplit > K / min_kr) nsplit = K / min_kr;
    if (nsplit > K / (40 * M)) nsplit = K / (40 * M);
    if (g_t.cluster_split && M <= 8 && nsplit > 8 && 8L * M * p.tn <= kClusterSlotFloats) nsplit = 8;     // the most that meet inside a cluster
    if (g_t.force_split > 0) nsplit = g_t.force_split;
    if (nsplit > kMaxSplit) nsplit = kMaxSplit;
    if (nsplit < 1) nsplit = 1;
    if ((long)p.ntiles * H > kNumCounters) nsplit = 1;
    int kr = ceil_div(K, nsplit);
    kr = ceil_div(kr, V) * V;
    nsplit = ceil_div(K, kr);
    p.nsplit = nsplit;
    p.kr = kr;
    return p;
}

// Tensor maps of recently used weight matrices (encoding one costs about a microsecond of host time).
struct MapKey { const void *B; int N, K, H; long strideB; int tn, kt; };      // tn = box columns, kt = box rows (16 marks a token map)
struct MapEntry { MapKey key; CUtensorMap map; bool valid; long row_stride; };
static thread_local MapEntry g_maps[16];
static thread_local int g_map_next = 0;

static const CUtensorMap *get_weight_map(const void *B, int N, int K, int H, long strideB, int tn, int kt, bool swizzle128 = false,
                                         long row_stride = 0)
{
    if (row_stride == 0) row_stride = N;
    for (auto &e : g_maps) {
        const MapKey &k = e.key;
        if (e.valid && k.B == B && k.N == N && k.K == K && k.H == H && k.strideB == strideB && k.tn == tn &&
            k.kt == (swizzle128 ? -kt : kt) && e.row_stride == row_stride)
            return &e.map;
    }
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return nullptr;
    MapEntry &e = g_maps[g_map_next];
    g_map_next = (g_map_next + 1) % 16;
    e.key = MapKey{B, N, K, H, strideB, tn, swizzle128 ? -kt : kt};
    e.row_stride = row_stride;
    const cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)K, (cuuint64_t)H};
    const cuuint64_t strides[2] = {(cuuint64_t)row_stride * 2, (cuuint64_t)(H > 1 ? strideB : (long)K * row_stride) * 2};
    const cuuint32_t box[3] = {(cuuint32_t)tn, (cuuint32_t)kt, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(B), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    e.valid = (r == CUDA_SUCCESS);
    return e.valid ? &e.map : nullptr;
}

// B in 16 x 16 fractals (element (k, n) at ((n/16)*(K/16) + k/16)*256 + (k%16)*16 + n%16) as a 4-D tensor: element in
// fractal (256, contiguous), fractal row, fractal column, head.  A box of kt x tn elements - kt/16 contiguous
// fractals from each of tn/16 fractal columns - lands in shared memory as [tn/16][kt][16].  Cached with the other maps (marked by a
// negative tile width).
static const CUtensorMap *get_fractal_map(const void *B, int N, int K, int H, long strideB, int tn, int kt)
{
    for (auto &e : g_maps) {
        const MapKey &k = e.key;
        if (e.valid && k.B == B && k.N == N && k.K == K && k.H == H && k.strideB == strideB && k.tn == -tn && k.kt == kt) return &e.map;
    }
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return nullptr;
    MapEntry &e = g_maps[g_map_next];
    g_map_next = (g_map_next + 1) % 16;
    e.key = MapKey{B, N, K, H, strideB, -tn, kt};
    e.row_stride = 0;
    const cuuint64_t dims[4] = {256, (cuuint64_t)(K / 16), (cuuint64_t)(N / 16), (cuuint64_t)H};
    const cuuint64_t strides[3] = {512, (cuuint64_t)(K / 16) * 512, (cuuint64_t)(H > 1 ? strideB : (long)K * N) * 2};
    const cuuint32_t box[4] = {256, (cuuint32_t)(kt / 16), (cuuint32_t)(tn / 16), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(B), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    e.valid = (r == CUDA_SUCCESS);
    return e.valid ? &e.map : nullptr;
}

static size_t partial_floats(const Plan &p, int M, int H)
{
    return p.nsplit > 1 ? (size_t)H * p.ntiles * p.nsplit * M * p.tn : 0;
}

static int check_common(const void *A, const void *B, const void *C, int M, int N, int K, int H,
                        nm_dtype dtype, nm_layout layout)
{
    if (!A || !B || !C) return NM_ERR_INVALID_ARG;
    if (M < 1 || M > NM_MAX_M_TENSOR || N < 1 || K < 1 || H < 1) return NM_ERR_INVALID_ARG;
    if (dtype != NM_F32 && dtype != NM_BF16 && dtype != NM_BF16_F32OUT && dtype != NM_F16) return NM_ERR_UNSUPPORTED;
    if (layout != NM_ROW_MAJOR && layout != NM_COL_MAJOR && layout != NM_FRACTAL_NZ) return NM_ERR_UNSUPPORTED;
    // 16 x 16 fractals: bf16, whole fractals, and only through the TMA ring kernel (up to 16 rows)
    if (layout == NM_FRACTAL_NZ && (dtype == NM_F32 || dtype == NM_F16 || (N % 16) || (K % 16) || M > NM_MAX_M)) return NM_ERR_UNSUPPORTED;
    if (H > 65535) return NM_ERR_UNSUPPORTED;
    const uintptr_t es = (uintptr_t)elem_size(dtype);
    const uintptr_t os = (dtype == NM_BF16 || dtype == NM_F16) ? 2 : 4;
    if (((uintptr_t)A % es) || ((uintptr_t)B % es) || ((uintptr_t)C % os)) return NM_ERR_ALIGNMENT;
    return NM_OK;
}

static int matmul_impl(const void *A, const void *B, void *C, int M, int N, int K, int H,
                       long lda, long strideA, long strideB, long ldc, long strideC,
                       nm_dtype dtype, nm_layout layout, void *ws, size_t ws_bytes, cudaStream_t stream, bool pdl = false,
                       unsigned long long *trace = nullptr, const VecTail *tail = nullptr, bool *tail_taken = nullptr, bool chained = false,
                       MatmulExtras *extras = nullptr)
{
    refresh_tuning();
    if (tail_taken) *tail_taken = false;
    if (extras) { extras->tile_ss_taken = extras->norm_taken = false; extras->tile_n = 0; }
    int rc = check_common(A, B, C, M, N, K, H, dtype, layout);
    if (rc != NM_OK) return rc;
    if (lda < K || ldc < N || strideA < 0 || strideB < 0 || strideC < 0) return NM_ERR_INVALID_ARG;

    const int V = vec_elems(dtype);
    // The 16-byte paths need B aligned with rows (columns) that stay aligned, and an aligned A for
    // the column kernel (it copies A into shared memory with 16-byte loads).
    const bool b_ok = aligned16(B) && (strideB % V == 0) &&
                      (layout == NM_COL_MAJOR ? (K % V == 0) : (N % V == 0));
    const bool a_ok = aligned16(A) && (lda % V == 0) && (strideA % V == 0);
    const bool vec_ok = b_ok && (layout == NM_ROW_MAJOR || a_ok);
    // tensor maps: 16-byte aligned operands and strides, bf16.  Row-major B may take the TMA ring kernel or the
    // tensor-core kernel; column-major B only the latter (its CUDA-core path is the plain column kernel).
    bool tma_ok = b_ok && a_ok && dtype != NM_F32 && tensor_map_encoder() != nullptr && (long)N * 2 < (1L << 40) && strideB >= 0;
    if (g_t.force_kind == kRowVec && layout != NM_FRACTAL_NZ) tma_ok = false;      // the fractal storage has one kernel: nothing to force
    if (layout == NM_FRACTAL_NZ && !tma_ok) return NM_ERR_UNSUPPORTED;      // unaligned operands or no tensor-map encoder
    Plan p = make_plan(M, N, K, H, dtype, layout, vec_ok, tma_ok, chained);
    if (g_log_plans && !(extras && extras->dry_run))
        fprintf(stderr, "nm: M=%d N=%d K=%d H=%d dtype=%d layout=%d -> kernel %d (0 row, 1 column, 2 scalar, 3 TMA ring, 4 tensor cores) tile_n=%d "
                "k-splits=%d k-rows=%d tiles=%d stages=%d%s\n", M, N, K, H, (int)dtype, (int)layout, (int)p.kind, p.tn, p.nsplit, p.kr, p.ntiles, p.nstage,
                chained ? " chained" : "");
    // Copies, not pointers into the map cache: the second lookup may evict the entry the first one returned
    // (16 entries, replaced in turn), and the kernel would then get the token map in place of the weight map.
    CUtensorMap tc_map_b_copy, tc_map_a_copy;
    const CUtensorMap *tc_map_b = nullptr, *tc_map_a = nullptr;
    if (M > NM_MAX_M && p.kind != kRowTc) return NM_ERR_UNSUPPORTED;       // 17-64 tokens: bf16 operands the tensor-core kernel takes
    if (p.kind == kRowTc) {
        // weights [H][K][N] in 64x64 swizzled boxes; tokens [H][M][K] (row stride lda) in 64 x 16 swizzled boxes
        tc_map_b = (layout == NM_ROW_MAJOR) ? get_weight_map(B, N, K, H, strideB, 64, kTcKT, true)
                                            : get_weight_map(B, K, N, H, strideB, 64, kTcTN, true);     // [N][K]: 64 k x 128 columns of C
        if (tc_map_b) { tc_map_b_copy = *tc_map_b; tc_map_b = &tc_map_b_copy; }
        tc_map_a = get_weight_map(A, K, M, H, strideA, 64, row_tc_tokens(M), true, lda);
        if (tc_map_a) { tc_map_a_copy = *tc_map_a; tc_map_a = &tc_map_a_copy; }
        if (!tc_map_b || !tc_map_a) {                       // strides the encoder refuses: CUDA-core kernel
            if (M > NM_MAX_M) return NM_ERR_UNSUPPORTED;
            p = make_plan(M, N, K, H, dtype, layout, vec_ok, false, chained);
        }
    }

    MatmulArgs a{};
    a.A = A; a.B = B; a.C = C;
    a.M = M; a.N = N; a.K = K; a.H = H;
    a.lda = lda; a.strideA = strideA; a.strideB = strideB; a.ldc = ldc; a.strideC = strideC;
    a.tn = p.tn; a.tpr = p.tpr; a.rg = p.rg; a.nsplit = p.nsplit; a.kr = p.kr; a.ntiles = p.ntiles;
    a.a_vec = a_ok ? 1 : 0;
    a.status = device_status_ptr();
    a.use_pdl = (g_t.use_pdl || pdl) ? 1 : 0;
    if (p.nsplit > 1) {
        const size_t need = kCounterBytes + partial_floats(p, M, H) * sizeof(float);
        if (!ws || ws_bytes < need) return NM_ERR_WORKSPACE;
        if (!aligned16(ws)) return NM_ERR_ALIGNMENT;
        a.counters = reinterpret_cast<unsigned *>(ws);
        a.partial = reinterpret_cast<float *>(static_cast<char *>(ws) + kCounterBytes);
    }

    if (extras && extras->dry_run && p.kind != kRowTma) return NM_OK;
    if ((p.kind == kRowVec || p.kind == kColVec) && g_t.cluster_split && p.nsplit >= 2 && p.nsplit <= 8 &&
        (long)p.nsplit * M * p.tn <= kClusterSlotFloats)
        a.cluster_split = 1;
    cudaError_t e = cudaErrorInvalidValue;
    if (p.kind == kRowTc) {
        const CUtensorMap *mb = tc_map_b, *ma = tc_map_a;
        TmaArgs ta{};
        ta.base = a; ta.nstage = p.nstage; ta.use_pdl = (g_t.use_pdl || pdl) ? 1 : 0; ta.status = device_status_ptr();
        if (g_t.cluster_split && p.nsplit >= 2 && p.nsplit <= 8 && (size_t)p.nsplit * M * kTcTN * sizeof(float) <= 65536) ta.cluster_split = 1;
        const bool col = layout == NM_COL_MAJOR;
        e = (dtype == NM_BF16_F32OUT) ? launch_row_tc<float>(*mb, *ma, ta, stream, col)
            : (dtype == NM_F16)       ? launch_row_tc<f16_t>(*mb, *ma, ta, stream, col)
                                      : launch_row_tc<bf16_t>(*mb, *ma, ta, stream, col);
    } else if (p.kind == kRowTma) {
        const int kt = (kTmaConsumers / p.tpr) * 4;
        const CUtensorMap *map = (layout == NM_FRACTAL_NZ) ? get_fractal_map(B, N, K, H, strideB, p.tn, kt)
                                                           : get_weight_map(B, N, K, H, strideB, p.tn, kt);
        if (!map) return record_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
        TmaArgs ta{};
        ta.fractal_nz = (layout == NM_FRACTAL_NZ) ? 1 : 0;
        ta.base = a; ta.nstage = p.nstage; ta.use_pdl = (g_t.use_pdl || pdl) ? 1 : 0; ta.status = device_status_ptr();
        ta.trace = trace;
        if (tail && tail->enabled && M == 1 && dtype == NM_BF16 && H == 1 && ws && ws_bytes >= kCounterBytes && aligned16(ws) &&
            p.ntiles < kNumCounters - 1 && N <= 4096 && N % 4 == 0 && p.tn % 4 == 0 && ldc % 4 == 0 && ((uintptr_t)C & 7u) == 0) {
            ta.tail = *tail;
            ta.tail.counter = reinterpret_cast<unsigned *>(ws) + (kNumCounters - 1);     // the last counter is never a tile's
            if (tail_taken) *tail_taken = true;
        }
        size_t smem = (size_t)p.nstage * kt * p.tn * 2 + kAChunkFloats * sizeof(float) + 2 * p.nstage * sizeof(uint64_t);
        // Split-K inside a cluster: up to eight splits (the portable cluster size) whose partial tiles fit 16 KB of
        // the first CTA's shared memory meet there instead of in the workspace.
        const size_t slot_bytes = (size_t)p.nsplit * M * p.tn * sizeof(float);
        if (g_t.cluster_split && p.nsplit >= 2 && p.nsplit <= 8 && !ta.tail.enabled && slot_bytes <= 16384) {
            ta.cluster_split = 1;
            smem += 16 + slot_bytes;
        }
        if (extras) {
            extras->tile_n = p.tn;
            if (extras->tile_ss && ta.cluster_split && M == 1 && dtype == NM_BF16 && H == 1) {
                ta.tile_ss = extras->tile_ss;
                extras->tile_ss_taken = true;
            }
            if (extras->norm && extras->norm->enabled && M == 1 && dtype == NM_BF16 && H == 1 && extras->norm->ntiles <= 32 &&
                extras->norm->n == K && K % 8 == 0) {
                ta.norm = *extras->norm;
                extras->norm_taken = true;
            }
        }
        const bool query = extras && extras->dry_run;
        const bool f32out = (dtype == NM_BF16_F32OUT);
        if (p.tpr == 8)       e = f32out ? launch_row_tma<8, float>(*map, ta, smem, stream, query)  : launch_row_tma<8, bf16_t>(*map, ta, smem, stream, query);
        else if (p.tpr == 16) e = f32out ? launch_row_tma<16, float>(*map, ta, smem, stream, query) : launch_row_tma<16, bf16_t>(*map, ta, smem, stream, query);
        else                  e = f32out ? launch_row_tma<32, float>(*map, ta, smem, stream, query) : launch_row_tma<32, bf16_t>(*map, ta, smem, stream, query);
        if (query) {
            // dry run: what the plan would do; per-tile sums of squares only when the clusters are all resident at once
            if (e != cudaSuccess) { (void)cudaGetLastError(); extras->tile_ss_taken = false; }
            return NM_OK;
        }
    } else if (p.kind == kGeneric) {
        if (dtype == NM_F32)            e = launch_generic<float, float>(a, layout, stream);
        else if (dtype == NM_BF16)      e = launch_generic<bf16_t, bf16_t>(a, layout, stream);
        else if (dtype == NM_F16)       e = launch_generic<f16_t, f16_t>(a, layout, stream);
        else                            e = launch_generic<bf16_t, float>(a, layout, stream);
    } else if (p.kind == kRowVec) {
        if (dtype == NM_F32)            e = launch_row<float, float>(a, stream);
        else if (dtype == NM_BF16)      e = launch_row<bf16_t, bf16_t>(a, stream);
        else if (dtype == NM_F16)       e = launch_row<f16_t, f16_t>(a, stream);
        else                            e = launch_row<bf16_t, float>(a, stream);
    } else {
        if (dtype == NM_F32)            e = launch_col<float, float>(a, stream);
        else if (dtype == NM_BF16)      e = launch_col<bf16_t, bf16_t>(a, stream);
        else if (dtype == NM_F16)       e = launch_col<f16_t, f16_t>(a, stream);
        else                            e = launch_col<bf16_t, float>(a, stream);
    }
    if (e != cudaSuccess) return record_cuda_error(e, "narrow matmul launch");
    return NM_OK;
}

void matmul_row_major_split(int M, int N, int K, int H, int *k_rows_per_split, int *nsplit, bool chained)
{
    refresh_tuning();
    const Plan p = make_plan(M, N, K, H, NM_BF16, NM_ROW_MAJOR, true, true, chained);      // whichever kernel the product will take
    *k_rows_per_split = p.kr;
    *nsplit = p.nsplit;
}

// internal entry used by the decode step
int matmul_enqueue(const void *A, const void *B, void *C, int M, int N, int K, int H,
                   long lda, long strideA, long strideB, long ldc, long strideC,
                   nm_dtype dtype, nm_layout layout, void *ws, size_t ws_bytes, cudaStream_t stream, bool programmatic_launch,
                   unsigned long long *trace, const VecTail *tail, bool *tail_taken, bool chained, MatmulExtras *extras)
{
    return matmul_impl(A, B, C, M, N, K, H, lda, strideA, strideB, ldc, strideC, dtype, layout, ws, ws_bytes, stream,
                       programmatic_launch, trace, tail, tail_taken, chained, extras);
}

}  // namespace nm

using namespace nm;

extern "C" {
#pragma GCC visibility push(default)

int nm_version(void) { return 100; }

const char *nm_status_string(int status)
{
    switch (status) {
    case NM_OK: return "ok";
    case NM_ERR_INVALID_ARG: return "invalid argument";
    case NM_ERR_UNSUPPORTED: return "unsupported dtype, layout or dimension";
    case NM_ERR_ALIGNMENT: return "pointer not aligned";
    case NM_ERR_WORKSPACE: return "workspace missing or too small";
    case NM_ERR_CUDA: return "CUDA error";
    case NM_ERR_TIMEOUT: return "bounded device-side wait expired";
    case NM_ERR_TOO_LARGE: return "problem too large for the built-in scratch of nm_matmul_static";
    case NM_ERR_BOUNDS: return "debug build: an access outside its operand was caught and skipped";
    default: return "unknown status";
    }
}

const char *nm_last_cuda_error(void) { return g_cuda_error; }

size_t nm_matmul_workspace_bytes(int M, int N, int K, int H, nm_dtype dtype, nm_layout layout_B)
{
    (void)K; (void)dtype; (void)layout_B;
    if (M < 1 || N < 1 || H < 1) return 0;
    // Upper bound over every plan the library may choose: at most kMaxSplit partial tiles of at
    // most (N rounded up to a tile) x M floats per head, plus the counters.
    const size_t npad = (size_t)N + kMaxTileN;
    return kCounterBytes + (size_t)kMaxSplit * (size_t)M * npad * (size_t)H * sizeof(float);
}

int nm_workspace_init(void *workspace, size_t bytes, nm_stream stream)
{
    if (!workspace || bytes < kCounterBytes) return NM_ERR_WORKSPACE;
    NM_CUDA_TRY(cudaMemsetAsync(workspace, 0, bytes, (cudaStream_t)stream));
    return NM_OK;
}

int nm_set_workspace(void *workspace, size_t bytes)
{
    if (workspace) {
        if (bytes < kCounterBytes) return NM_ERR_WORKSPACE;
        NM_CUDA_TRY(cudaMemset(workspace, 0, kCounterBytes));
    }
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    g_tuning_shared.ws = workspace; g_tuning_shared.ws_bytes = workspace ? bytes : 0;
    return NM_OK;
}

int nm_matmul(const void *A, const void *B, void *C, int M, int N, int K,
              nm_dtype dtype, nm_layout layout_B, nm_stream stream)
{
    refresh_tuning();
    return matmul_impl(A, B, C, M, N, K, 1, K, 0, 0, N, 0, dtype, layout_B, g_t.ws, g_t.ws_bytes, (cudaStream_t)stream);
}

int nm_matmul_ws(const void *A, const void *B, void *C, int M, int N, int K,
                 nm_dtype dtype, nm_layout layout_B, void *workspace, size_t workspace_bytes, nm_stream stream)
{
    return matmul_impl(A, B, C, M, N, K, 1, K, 0, 0, N, 0, dtype, layout_B, workspace, workspace_bytes, (cudaStream_t)stream);
}

int nm_matmul_batched(const void *A, const void *B, void *C, int M, int N, int K, int H,
                      long lda, long strideA, long strideB, long ldc, long strideC,
                      nm_dtype dtype, nm_layout layout_B, nm_stream stream)
{
    refresh_tuning();
    return matmul_impl(A, B, C, M, N, K, H, lda, strideA, strideB, ldc, strideC, dtype, layout_B, g_t.ws, g_t.ws_bytes, (cudaStream_t)stream);
}

int nm_matmul_batched_ws(const void *A, const void *B, void *C, int M, int N, int K, int H,
                         long lda, long strideA, long strideB, long ldc, long strideC,
                         nm_dtype dtype, nm_layout layout_B, void *workspace, size_t workspace_bytes, nm_stream stream)
{
    return matmul_impl(A, B, C, M, N, K, H, lda, strideA, strideB, ldc, strideC, dtype, layout_B, workspace, workspace_bytes, (cudaStream_t)stream);
}

int nm_matmul_host(const void *A_host, const void *B, void *C_host, void *A_staging, void *C_staging,
                   int M, int N, int K, nm_dtype dtype, nm_layout layout_B,
                   void *workspace, size_t workspace_bytes, nm_stream stream)
{
    if (!A_host || !C_host || !A_staging || !C_staging) return NM_ERR_INVALID_ARG;
    int rc = check_common(A_staging, B, C_staging, M, N, K, 1, dtype, layout_B);
    if (rc != NM_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t a_bytes = (size_t)M * K * elem_size(dtype);
    const size_t c_bytes = (size_t)M * N * ((dtype == NM_BF16 || dtype == NM_F16) ? 2 : 4);
    NM_CUDA_TRY(cudaMemcpyAsync(A_staging, A_host, a_bytes, cudaMemcpyHostToDevice, s));
    rc = matmul_impl(A_staging, B, C_staging, M, N, K, 1, K, 0, 0, N, 0, dtype, layout_B, workspace, workspace_bytes, s);
    if (rc != NM_OK) return rc;
    NM_CUDA_TRY(cudaMemcpyAsync(C_host, C_staging, c_bytes, cudaMemcpyDeviceToHost, s));
    return NM_OK;
}

/* Tuning override for sweeps: columns per tile (row-major kernel) and k-splits; 0 = heuristic. */
int nm_debug_set_plan(int tile_n, int nsplit)
{
    if (tile_n < 0 || nsplit < 0 || tile_n > kMaxTileN || nsplit > kMaxSplit) return NM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    g_tuning_shared.force_tn = tile_n; g_tuning_shared.force_split = nsplit;
    return NM_OK;
}

int nm_debug_set_cluster_split(int enable)
{
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    g_tuning_shared.cluster_split = enable ? 1 : 0;
    return NM_OK;
}

/* Smallest M that goes to the swap-AB tensor-core kernel (row-major bf16 B); 17 keeps every M on CUDA cores. */
int nm_set_tensor_core_min_m(int m)
{
    if (m < 1 || m > NM_MAX_M + 1) return NM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    g_tuning_shared.tc_min_m = m;
    return NM_OK;
}

/* Force the kernel family (-1 heuristic, 0 plain row-major kernel instead of the TMA ring) and the ring depth. */
int nm_debug_set_kernel(int kind, int stages)
{
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    g_tuning_shared.force_kind = kind; g_tuning_shared.force_stages = stages;
    return NM_OK;
}

int nm_set_programmatic_launch(int enable)
{
    std::lock_guard<std::mutex> lock(g_tuning_mutex);
    g_tuning_shared.use_pdl = enable ? 1 : 0;
    return NM_OK;
}

/* Reports the plan the library would use: out[0..5] = kind, tile_n, nsplit, k-rows per split, tiles, CTAs. */
int nm_debug_get_plan(int M, int N, int K, int H, nm_dtype dtype, nm_layout layout_B, int vec_ok, int *out)
{
    if (!out) return NM_ERR_INVALID_ARG;
    refresh_tuning();
    Plan p = make_plan(M, N, K, H, dtype, layout_B, vec_ok != 0,
                       vec_ok != 0 && dtype != NM_F32 && g_t.force_kind != kRowVec);
    out[0] = p.kind; out[1] = p.tn; out[2] = p.nsplit; out[3] = p.kr; out[4] = p.ntiles;
    out[5] = p.ntiles * p.nsplit * H;
    return NM_OK;
}

#pragma GCC visibility pop
}  // extern "C"
