// Shared device/host helpers for the nm kernels (sm_100a only).
#pragma once
#include <atomic>
#include <cstdio>
#include <cstdlib>

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/nm.h"
#include "../../include/nm_debug.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "nm kernels are written for sm_100a"
#endif

namespace nm {

struct VecTail;

constexpr int kSMs = 148;                 // B200: 2 dies x 74 SMs
constexpr int kMaxSplit = 64;             // upper bound on k-splits (sizes the workspace)
constexpr int kMaxTileN = 2048;           // upper bound on columns per CTA tile
constexpr size_t kCounterBytes = NM_WS_COUNTER_BYTES;
constexpr int kNumCounters = int(kCounterBytes / sizeof(unsigned));

// Records a CUDA failure for nm_last_cuda_error() and maps it to NM_ERR_CUDA.
int record_cuda_error(cudaError_t e, const char *where);

#define NM_CUDA_TRY(expr)                                                        \
    do {                                                                         \
        cudaError_t _e = (expr);                                                 \
        if (_e != cudaSuccess) return ::nm::record_cuda_error(_e, #expr);        \
    } while (0)

// ---- element traits -------------------------------------------------------------------------

struct bf16_t { uint16_t bits; };

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;        // elements per 16-byte load
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[4]) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float widen(float x) { return x; }
};
template <> struct Elem<bf16_t> {
    static constexpr int kVec = 8;
    // bf16 is the upper half of an fp32: widening is a shift (exact).
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[8]) {
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    __device__ static __forceinline__ float widen(bf16_t x) { return __uint_as_float(uint32_t(x.bits) << 16); }
};

// fp16 (IEEE binary16), the optional element type: widening is a conversion instruction (exact).
struct f16_t { uint16_t bits; };
template <> struct Elem<f16_t> {
    static constexpr int kVec = 8;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&f)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 p = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            f[2 * i] = p.x; f[2 * i + 1] = p.y;
        }
    }
    __device__ static __forceinline__ float widen(f16_t x) { return __half2float(__ushort_as_half(x.bits)); }
};

// Output rounding: one round-to-nearest-even step from the fp32 sum.
template <typename T> __device__ __forceinline__ T round_out(float x);
template <> __device__ __forceinline__ float round_out<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16_t round_out<bf16_t>(float x) {
    bf16_t r; r.bits = __bfloat16_as_ushort(__float2bfloat16_rn(x)); return r;
}
template <> __device__ __forceinline__ f16_t round_out<f16_t>(float x) {
    f16_t r; r.bits = __half_as_ushort(__float2half_rn(x)); return r;
}

// 16-byte streaming load: read-only path, no L1 allocation (each weight byte is used once).
__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// ---- debug build (-DNM_BOUNDS_CHECK, libnm_check.so) -----------------------------------------------------------
// Every hand-indexed global access of the narrow-product kernels names the operand it belongs to; the debug build
// checks the address against that operand's extent first.  An access outside it raises kStatusOutOfBounds in the
// device status word (nm_check_status then returns NM_ERR_BOUNDS) and is SKIPPED - a load yields zeros, a store does
// nothing - so nothing faults and nothing traps.  (The tiled TMA copies need no such build: the copy engine clips them
// to the tensor map's extents.)  In the normal build the macros are the bare access.
constexpr unsigned kStatusOutOfBounds = 2u;
struct Span { const char *lo, *hi; };                              // [lo, hi)
__host__ __device__ __forceinline__ Span make_span(const void *base, size_t bytes)
{
    return Span{static_cast<const char *>(base), static_cast<const char *>(base) + bytes};
}
#ifdef NM_BOUNDS_CHECK
__device__ __forceinline__ bool nm_inside(const void *p, size_t n, Span s, unsigned *status)
{
    const char *c = static_cast<const char *>(p);
    const bool ok = c >= s.lo && c + n <= s.hi;
    if (!ok && status) atomicOr(status, kStatusOutOfBounds);
    return ok;
}
#define NM_LD_STREAM16(p, span, st) (::nm::nm_inside((p), 16, (span), (st)) ? ::nm::ld_stream16(p) : make_uint4(0u, 0u, 0u, 0u))
#define NM_LDG16(p, span, st) (::nm::nm_inside((p), 16, (span), (st)) ? __ldg(p) : make_uint4(0u, 0u, 0u, 0u))
template <typename T> __device__ __forceinline__ T nm_checked_load(const T *p, Span s, unsigned *status)
{
    return nm_inside(p, sizeof(T), s, status) ? *p : T{};
}
#define NM_LD(p, span, st) ::nm::nm_checked_load((p), (span), (st))
#define NM_LD_CG(p, span, st) (::nm::nm_inside((p), sizeof(float), (span), (st)) ? ::nm::ld_cg(p) : 0.f)
#define NM_ST(p, v, span, st) do { if (::nm::nm_inside((p), sizeof(*(p)), (span), (st))) *(p) = (v); } while (0)
#else
#define NM_LD_STREAM16(p, span, st) ::nm::ld_stream16(p)
#define NM_LDG16(p, span, st) __ldg(p)
#define NM_LD(p, span, st) (*(p))
#define NM_LD_CG(p, span, st) ::nm::ld_cg(p)
#define NM_ST(p, v, span, st) (*(p) = (v))
#endif

// Load that bypasses L1 (data written by other SMs in the same launch).
__device__ __forceinline__ float ld_cg(const float *p) { return __ldcg(p); }

// Validates, plans and enqueues one (batched) narrow product; `ws` may be null when the plan does
// not split K.  With programmatic_launch the kernel may begin (and prefetch B) before the previous
// kernel in the stream has finished; it still waits for it before reading A or writing anything.
// `tail`: vector stages to run when the product's last tile completes (see VecTail); only the TMA ring kernel
// takes it (M = 1, bf16 output) - *tail_taken says whether it did, the caller launches them itself otherwise.
// `chained`: the launch is one link of a programmatic chain of kernels (the decode step); the planner then
// prefers one CTA per SM with a deep ring and fewer k-splits.  Defined in nm_matmul.cu.
// `extras` (optional): per-tile sums of squares of the outputs (only the TMA ring kernel with its k-splits in a
// cluster writes them, M = 1, bf16) and RMSNorm of the token row on load (TMA ring kernel, M = 1, bf16); the
// *_taken flags and tile_n report what the plan does; with dry_run nothing is launched.
struct MatmulExtras {
    float *tile_ss = nullptr;
    const struct RowNorm *norm = nullptr;
    bool dry_run = false;
    bool tile_ss_taken = false, norm_taken = false;
    int tile_n = 0;
};
int matmul_enqueue(const void *A, const void *B, void *C, int M, int N, int K, int H,
                   long lda, long strideA, long strideB, long ldc, long strideC,
                   nm_dtype dtype, nm_layout layout, void *ws, size_t ws_bytes, cudaStream_t stream,
                   bool programmatic_launch = false, unsigned long long *trace = nullptr, const struct VecTail *tail = nullptr,
                   bool *tail_taken = nullptr, bool chained = false, MatmulExtras *extras = nullptr);

// A plan (tile width, k-splits, ring depth; zeros = planner) forced for the CALLING THREAD's next products only; it
// overrides the process-wide nm_debug_set_plan / nm_debug_set_kernel values while active.  The decode step uses it to
// force one of its products without touching what other host threads see.
void set_thread_plan_override(bool active, int tile_n, int nsplit, int stages);

// How the row-major bf16 product K x N (H heads) at this M will be split: k-rows per split and splits.
void matmul_row_major_split(int M, int N, int K, int H, int *k_rows_per_split, int *nsplit, bool chained = false);

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) is a per-device setting: remember per launch site which devices
// have it (one bit per device ordinal), so that a process using several GPUs configures the kernel on each of them.
// Two threads racing on the first call both set the (idempotent) attribute.
template <typename Kern>
cudaError_t ensure_dynamic_smem(Kern kern, int bytes, std::atomic<unsigned long long> &done_mask)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const unsigned long long bit = (dev >= 0 && dev < 64) ? (1ull << dev) : 0ull;
    if (bit && (done_mask.load(std::memory_order_acquire) & bit)) return cudaSuccess;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess && bit) done_mask.fetch_or(bit, std::memory_order_release);
    return e;
}

__host__ __device__ constexpr int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Whether all `clusters` clusters of a launch configured in `cfg` (cluster dimension among its attributes) can be
// resident at once.  The CTAs of a cluster need SMs of one GPC at the same time, so a grid that fits the machine
// CTA by CTA may still need a second wave as clusters; the split-K-in-a-cluster paths fall back to the workspace
// then.  Answers are cached per (kernel, shared memory, cluster size).
template <typename Kern>
int max_clusters_cached(Kern kern, const cudaLaunchConfig_t &cfg, unsigned cluster_size)
{
    struct Entry { const void *f; size_t smem; unsigned cs; int n; };
    static thread_local Entry cache[32];
    static thread_local int next = 0;
    const void *f = reinterpret_cast<const void *>(kern);
    for (const Entry &e : cache)
        if (e.f == f && e.smem == cfg.dynamicSmemBytes && e.cs == cluster_size) return e.n;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }   // not cached: ask again next time
    cache[next] = Entry{f, cfg.dynamicSmemBytes, cluster_size, n};
    next = (next + 1) % 32;
    return n;
}
template <typename Kern>
bool clusters_fit_one_wave(Kern kern, const cudaLaunchConfig_t &cfg, unsigned cluster_size, long clusters)
{
    return max_clusters_cached(kern, cfg, cluster_size) >= clusters;
}

}  // namespace nm
