// Single-token MLA decode step: the vector-side stages (RMSNorm, RoPE, cache-row write), the merge
// of the attention splits, and the host orchestration that overlaps the CUDA-core narrow products
// with the tensor-core attention pass.
#include <algorithm>
#include <cmath>
#include <mutex>

#include "nm_async.cuh"
#include "nm_mla.cuh"
#include "nm_matmul_kernels.cuh"

namespace nm {

// Tuning state of the decode step (nm_debug_set_*): process-wide and guarded by a mutex; every entry point plans from a
// per-thread snapshot taken once at its start, so a setter on another host thread cannot change a step half way.
struct StepTuning {
    int attn_impl = 0;          // 0: tensor-core kernel when the shape allows, 1: CUDA-core kernel, 2 / 3: force 128 / 64 heads per CTA,
                                // 4: force the wide-tile kernel
    int wide_tile = 0, wide_splits = 0, wide_cluster = 0;      // wide-tile kernel: forced rows per tile, row runs, cluster size (0 = planner)
    int kv_beside_attention = 0; // two-stream schedule: the KV chain starts when the attention operand is ready, beside the tensor-core pass
    int step_plan[3][3] = {};   // forced (tile_n, nsplit, stages) of the down-projection, W_UQR and W_O products (0 = planner)
    int host_direct_out = 1;    // host-operand step: store the result straight into device-addressable host memory
    int batch_tc_min_t = 3;     // batch decode: tokens from which the per-head products go to the tensor cores
    int fused_tails = 1;        // 0: RMSNorm / RoPE / cache write as kernels of their own; 1: folded into the products (default);
                                // 2: as 1, but only in the form where the product's last CTA runs them
    int step_pdl = 1;           // chain the kernels of the decode step with programmatic dependent launch
    int fused_heads = 1;        // per-head stages fused with their vector stage (q_finish, uv_merge) when the dims allow
    int uv_pdl = 1;             // launch uv_merge programmatically
    int prefetch_uv = 1;        // include W_UV in the L2 prefetch
    int prefetch_mb = 40;       // MB of W_O pulled into L2 beside the attention pass (plus all of W_UV); 0 = off
};
static std::mutex g_step_mutex;
static StepTuning g_step_shared;
static thread_local StepTuning g_s;                   // the calling thread's snapshot
static void refresh_step_tuning()
{
    std::lock_guard<std::mutex> lock(g_step_mutex);
    g_s = g_step_shared;
}
template <typename F> static int set_step_tuning(F f)
{
    std::lock_guard<std::mutex> lock(g_step_mutex);
    f(g_step_shared);
    return NM_OK;
}
// Cache rows (over all sequences of a call) from which the 128-head kernel is the faster one: it loads every row
// into two CTAs instead of four, which decides once a CTA has many tiles to go through; below, the 64-head
// kernel's shorter prologue and merge win (measured: 16384 rows 94.8 vs 97.3 us per step, 65536 rows 164 vs 158)
constexpr long kAttn128HeadRows = 65536;
constexpr int kAttnWideMinRows = 6144;     // single sequence: cache rows from which the wide-tile kernel takes over
constexpr int kSMsAttn = 148;
static bool attention_64_heads(long total_rows) { return g_s.attn_impl == 3 || (g_s.attn_impl != 2 && total_rows < kAttn128HeadRows); }

// ---- small vector kernels ---------------------------------------------------------------------------

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t f32_to_bf16_bits(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }

__device__ __forceinline__ float block_sum(float v, float *scratch /* >= 32 floats */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nwarp; ++w) t += scratch[w];      // same order in every thread
    return t;
}

// y = x * rsqrt(mean(x^2) + eps) * gamma, one CTA, everything in fp32, one rounding to bf16.
// x and gamma are fetched with 16-byte loads where alignment allows, all issued before the sum.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ gamma,
                                                      uint16_t *__restrict__ y, int n, float eps)
{
    __shared__ float scratch[32];
    pdl_wait_prior_grids();
    const bool vec = (n % 8 == 0) && n <= 8 * 256 * 4 && ((((uintptr_t)x | (uintptr_t)gamma | (uintptr_t)y) & 15u) == 0);
    if (vec) {
        constexpr int kMaxPerThread = 4;
        uint4 xv[kMaxPerThread], gv[kMaxPerThread];
        const int nv = n / 8;
#pragma unroll
        for (int j = 0; j < kMaxPerThread; ++j) {
            const int i = threadIdx.x + j * 256;
            if (i < nv) { xv[j] = reinterpret_cast<const uint4 *>(x)[i]; gv[j] = __ldg(reinterpret_cast<const uint4 *>(gamma) + i); }
        }
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxPerThread; ++j)
            if (threadIdx.x + j * 256 < nv) {
                float f[8];
                Elem<bf16_t>::unpack(xv[j], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
            }
        ss = block_sum(ss, scratch);
        const float r = 1.0f / sqrtf(ss / (float)n + eps);
#pragma unroll
        for (int j = 0; j < kMaxPerThread; ++j) {
            const int i = threadIdx.x + j * 256;
            if (i < nv) {
                float f[8], g[8];
                Elem<bf16_t>::unpack(xv[j], f);
                Elem<bf16_t>::unpack(gv[j], g);
                uint32_t o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    o[e] = (uint32_t)f32_to_bf16_bits(f[2 * e] * r * g[2 * e]) | ((uint32_t)f32_to_bf16_bits(f[2 * e + 1] * r * g[2 * e + 1]) << 16);
                reinterpret_cast<uint4 *>(y)[i] = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
        return;
    }
    float ss = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float v = bf16_bits_to_f32(x[i]);
        ss = fmaf(v, v, ss);
    }
    ss = block_sum(ss, scratch);
    const float r = 1.0f / sqrtf(ss / (float)n + eps);
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        y[i] = f32_to_bf16_bits(bf16_bits_to_f32(x[i]) * r * bf16_bits_to_f32(gamma[i]));
}

// Interleaved-pair rotary embedding on n_vec vectors of `dim` bf16 elements.
__global__ void __launch_bounds__(256) rope_kernel(const uint16_t *__restrict__ x, uint16_t *__restrict__ y, int n_vec, int dim,
                                                   long x_stride, long y_stride, const float *__restrict__ cs)
{
    pdl_wait_prior_grids();
    const int half = dim / 2;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_vec * half) return;
    const int v = idx / half, i = idx - v * half;
    const float c = cs[2 * i], s = cs[2 * i + 1];
    const float x0 = bf16_bits_to_f32(x[v * x_stride + 2 * i]), x1 = bf16_bits_to_f32(x[v * x_stride + 2 * i + 1]);
    y[v * y_stride + 2 * i] = f32_to_bf16_bits(x0 * c - x1 * s);
    y[v * y_stride + 2 * i + 1] = f32_to_bf16_bits(x0 * s + x1 * c);
}

// (cos, sin) of pos * base^(-2i/dim), evaluated in fp64 so that large positions keep their phase.
__global__ void rope_table_kernel(float *table, long pos_begin, int n_pos, int dim, double base)
{
    const int half = dim / 2;
    const long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long)n_pos * half) return;
    const long p = idx / half;
    const int i = (int)(idx - p * half);
    const double ang = (double)(pos_begin + p) * pow(base, -2.0 * (double)i / (double)dim);
    double s, c;
    sincos(ang, &s, &c);
    table[p * dim + 2 * i] = (float)c;
    table[p * dim + 2 * i + 1] = (float)s;
}

// The consumers of MatMul 2 in one kernel: RMSNorm of the latent part, RoPE of the key part,
// both rounded to bf16 and written into the cache row.  dc <= 512 elements per 256 threads x 2.
__global__ void __launch_bounds__(256) kv_finish_kernel(const uint16_t *__restrict__ ckr, const uint16_t *__restrict__ gamma,
                                                        const float *__restrict__ cs, uint16_t *__restrict__ cache_row,
                                                        int dc, int dr, float eps)
{
    __shared__ float scratch[32];
    pdl_wait_prior_grids();
    const int i0 = 2 * threadIdx.x;                                // two latent elements per thread
    float x0 = 0.f, x1 = 0.f, g0 = 0.f, g1 = 0.f;
    if (i0 < dc) {
        const uint32_t xv = *reinterpret_cast<const uint32_t *>(ckr + i0), gv = *reinterpret_cast<const uint32_t *>(gamma + i0);
        x0 = __uint_as_float(xv << 16); x1 = __uint_as_float(xv & 0xffff0000u);
        g0 = __uint_as_float(gv << 16); g1 = __uint_as_float(gv & 0xffff0000u);
    }
    float r0v = 0.f, r1v = 0.f, c = 0.f, sn = 0.f;
    if (threadIdx.x < dr / 2) {
        const uint32_t rv = *reinterpret_cast<const uint32_t *>(ckr + dc + i0);
        r0v = __uint_as_float(rv << 16); r1v = __uint_as_float(rv & 0xffff0000u);
        c = cs[i0]; sn = cs[i0 + 1];
    }
    const float ss = block_sum(fmaf(x0, x0, x1 * x1), scratch);
    const float r = 1.0f / sqrtf(ss / (float)dc + eps);
    if (i0 < dc)
        *reinterpret_cast<uint32_t *>(cache_row + i0) = (uint32_t)f32_to_bf16_bits(x0 * r * g0) | ((uint32_t)f32_to_bf16_bits(x1 * r * g1) << 16);
    if (threadIdx.x < dr / 2)
        *reinterpret_cast<uint32_t *>(cache_row + dc + i0) =
            (uint32_t)f32_to_bf16_bits(r0v * c - r1v * sn) | ((uint32_t)f32_to_bf16_bits(r0v * sn + r1v * c) << 16);
}

// ---- attention over a split of the rows on CUDA cores (kept for sequence splits the tensor-core
//      kernel does not take: fewer rows than one MMA tile) -------------------------------------------------
//
// grid (nsplit, H), 4 warps.  Each warp walks rows r0+warp, r0+warp+4, ... with its own online-softmax
// state; lane l owns latent columns [16l, 16l+16) and rope columns [2l, 2l+2).
__global__ void __launch_bounds__(128) attn_partial_simt_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                                AttnPartials part, int n_rows, int rows_per_split,
                                                                int dc, int dr, float scale)
{
    const int sp = blockIdx.x, h = blockIdx.y, H = gridDim.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int dkv = dc + dr;
    __shared__ float sm_m[4], sm_l[4];
    __shared__ float sm_o[4][512];
    pdl_wait_prior_grids();
    float q[18];
    {
        const uint16_t *qh = Q + (size_t)h * dkv;
#pragma unroll
        for (int i = 0; i < 16; ++i) q[i] = bf16_bits_to_f32(qh[lane * 16 + i]) * scale;
        q[16] = bf16_bits_to_f32(qh[dc + 2 * lane]) * scale;
        q[17] = bf16_bits_to_f32(qh[dc + 2 * lane + 1]) * scale;
    }
    const int r0 = sp * rows_per_split, r1 = min(n_rows, r0 + rows_per_split);
    float m = -INFINITY, l = 0.f, o[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) o[i] = 0.f;
    for (int j = r0 + warp; j < r1; j += 4) {
        const uint16_t *row = cache + (size_t)j * dkv;
        const uint4 v0 = *reinterpret_cast<const uint4 *>(row + lane * 16);
        const uint4 v1 = *reinterpret_cast<const uint4 *>(row + lane * 16 + 8);
        const uint32_t vr = *reinterpret_cast<const uint32_t *>(row + dc + 2 * lane);
        float c[16];
        float f[8];
        Elem<bf16_t>::unpack(v0, f);
#pragma unroll
        for (int i = 0; i < 8; ++i) c[i] = f[i];
        Elem<bf16_t>::unpack(v1, f);
#pragma unroll
        for (int i = 0; i < 8; ++i) c[8 + i] = f[i];
        float s = q[16] * __uint_as_float(vr << 16) + q[17] * __uint_as_float(vr & 0xffff0000u);
#pragma unroll
        for (int i = 0; i < 16; ++i) s = fmaf(q[i], c[i], s);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        const float mn = fmaxf(m, s);
        const float corr = __expf(m - mn), p = __expf(s - mn);
        l = l * corr + p;
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = fmaf(p, c[i], o[i] * corr);
        m = mn;
    }
    if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; }
#pragma unroll
    for (int i = 0; i < 16; ++i) sm_o[warp][lane * 16 + i] = o[i];
    __syncthreads();
    float M4 = fmaxf(fmaxf(sm_m[0], sm_m[1]), fmaxf(sm_m[2], sm_m[3]));
    float w[4], L = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) { w[k] = (sm_m[k] == -INFINITY) ? 0.f : __expf(sm_m[k] - M4); L += w[k] * sm_l[k]; }
    float *Od = part.O + ((size_t)sp * H + h) * dc;
    for (int cidx = threadIdx.x; cidx < dc; cidx += blockDim.x)
        Od[cidx] = w[0] * sm_o[0][cidx] + w[1] * sm_o[1][cidx] + w[2] * sm_o[2][cidx] + w[3] * sm_o[3][cidx];
    if (threadIdx.x == 0) {
        part.ml[((size_t)sp * H + h) * 2] = M4;
        part.ml[((size_t)sp * H + h) * 2 + 1] = L;
    }
}

// ---- merge of the splits (and of the row the step has just written) --------------------------------------
//
// One CTA per head.  Partial (m, l, O) of split s means: o = O / l with scores shifted by m.  The
// extra row contributes a single score.  Result: sum_s e^{m_s - M} O_s + e^{s_x - M} c_x over
// sum_s e^{m_s - M} l_s + e^{s_x - M}.
constexpr int kCombineThreads = 512;      // 4 groups of 128 threads; each group takes every 4th split

__global__ void __launch_bounds__(kCombineThreads) attn_combine_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                                       AttnPartials part, int nsplit, long extra_row, int dc, int dr,
                                                                       float scale, uint16_t *__restrict__ o_bf16, float *__restrict__ o_f32)
{
    const int h = blockIdx.x, H = gridDim.x, dkv = dc + dr;
    const int grp = threadIdx.x >> 7, t = threadIdx.x & 127;
    __shared__ float scratch[32];
    __shared__ float sm[kMaxAttnSplits], sl[kMaxAttnSplits], sw[kMaxAttnSplits];
    __shared__ float4 red[3][128];
    pdl_wait_prior_grids();
    // every split's (m, l) in one round of loads
    for (int s = threadIdx.x; s < nsplit; s += blockDim.x) {
        const float2 v = __ldcg(reinterpret_cast<const float2 *>(part.ml + ((size_t)s * H + h) * 2));
        sm[s] = v.x; sl[s] = v.y;
    }
    // first batch of partial rows goes out before anything that needs the weights
    const int c = 4 * t;                                           // dc == 512: four columns per thread
    const float *src = part.O + (size_t)h * dc + c;
    constexpr int kBatch = 8;
    float4 v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
        const int s = grp + 4 * u;
        v[u] = (s < nsplit) ? __ldcg(reinterpret_cast<const float4 *>(src + (size_t)s * H * dc)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float sx = -INFINITY;
    if (extra_row >= 0) {
        const uint16_t *qh = Q + (size_t)h * dkv, *row = cache + (size_t)extra_row * dkv;
        float acc = 0.f;
        for (int i = threadIdx.x; i < dkv; i += blockDim.x) acc = fmaf(bf16_bits_to_f32(qh[i]), bf16_bits_to_f32(row[i]), acc);
        sx = block_sum(acc, scratch) * scale;
    } else {
        __syncthreads();
    }
    float Mx = sx;
    for (int s = 0; s < nsplit; ++s) Mx = fmaxf(Mx, sm[s]);
    const float wx = (extra_row >= 0) ? __expf(sx - Mx) : 0.f;
    float L = wx;
    for (int s = 0; s < nsplit; ++s) {                             // same order in every thread
        const float w = (sm[s] == -INFINITY) ? 0.f : __expf(sm[s] - Mx);
        if (threadIdx.x == 0) sw[s] = w;
        L = fmaf(w, sl[s], L);
    }
    __syncthreads();
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (grp == 0 && extra_row >= 0) {
        const uint2 rv = *reinterpret_cast<const uint2 *>(cache + (size_t)extra_row * dkv + c);
        acc = make_float4(wx * __uint_as_float(rv.x << 16), wx * __uint_as_float(rv.x & 0xffff0000u),
                          wx * __uint_as_float(rv.y << 16), wx * __uint_as_float(rv.y & 0xffff0000u));
    }
    for (int s0 = 0; s0 < nsplit; s0 += 4 * kBatch) {
        if (s0 > 0) {
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int s = s0 + grp + 4 * u;
                v[u] = (s < nsplit) ? __ldcg(reinterpret_cast<const float4 *>(src + (size_t)s * H * dc)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int s = s0 + grp + 4 * u;
            const float w = (s < nsplit) ? sw[s] : 0.f;
            acc.x = fmaf(w, v[u].x, acc.x); acc.y = fmaf(w, v[u].y, acc.y);
            acc.z = fmaf(w, v[u].z, acc.z); acc.w = fmaf(w, v[u].w, acc.w);
        }
    }
    if (grp > 0) red[grp - 1][t] = acc;
    __syncthreads();
    if (grp == 0) {
#pragma unroll
        for (int g = 0; g < 3; ++g) {                              // fixed order: deterministic
            const float4 r = red[g][t];
            acc.x += r.x; acc.y += r.y; acc.z += r.z; acc.w += r.w;
        }
        const float inv = 1.0f / L;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        if (o_f32) *reinterpret_cast<float4 *>(o_f32 + (size_t)h * dc + c) = acc;
        if (o_bf16)
            *reinterpret_cast<uint2 *>(o_bf16 + (size_t)h * dc + c) =
                make_uint2((uint32_t)f32_to_bf16_bits(acc.x) | ((uint32_t)f32_to_bf16_bits(acc.y) << 16),
                           (uint32_t)f32_to_bf16_bits(acc.z) | ((uint32_t)f32_to_bf16_bits(acc.w) << 16));
    }
}

// The token row of the host-operand step: n 16-byte vectors from device-addressable host memory into the staging row.
// One CTA: all loads go out at once (one trip over the host link), the kernels chained behind it start meanwhile.
__device__ __forceinline__ uint4 ld_host16(const uint4 *p)        // the host may have rewritten the row since the last launch
{
    uint4 v;
    asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__global__ void __launch_bounds__(256) token_fetch_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int n)
{
    pdl_launch_dependents();
    uint4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int i = (int)threadIdx.x + u * 256;
        v[u] = (i < n) ? ld_host16(src + i) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int i = (int)threadIdx.x + u * 256;
        if (i < n) dst[i] = v[u];
    }
    for (int i = (int)threadIdx.x + 1024; i < n; i += 256) dst[i] = ld_host16(src + i);
}

// ---- host -------------------------------------------------------------------------------------------

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

AttnPlan plan_attention(const void *Q, const void *cache, int H, int n_rows, int kv_lora)
{
    AttnPlan p{};
    (void)kv_lora;
    // The tensor-core kernels take 128 heads and 16-byte aligned operands (TMA); both passes of an
    // attention call derive the same answer from the same arguments.
    const bool tc_ok = g_s.attn_impl != 1 && H == 128 && n_rows > 0 && (((uintptr_t)Q | (uintptr_t)cache) & 15u) == 0 &&
                       tensor_map_encoder() != nullptr;
    // Wide tiles (nm_attn_wide.cu) from kAttnWideMinRows cache rows on: measured per step 83.2 vs 93.2 us at 16384 rows, level
    // at 4096 (78.2 vs 77.7) and below, where the pass is all fixed cost (waiting for Q, the merge) in either kernel.
    if (tc_ok && (g_s.attn_impl == 4 || (g_s.attn_impl == 0 && n_rows >= kAttnWideMinRows))) {
        // One tile per row run as long as at most 64 runs (128 CTAs) cover the rows: the tile is as wide as that takes,
        // and the runs of a cluster merge on chip so that the final merge reads at most 16 partials per head.
        int R = g_s.wide_tile;
        const int max_runs = g_s.wide_splits > 0 ? std::min(g_s.wide_splits, 64) : 64;
        if (R != 64 && R != 128 && R != 256) R = (n_rows <= 64 * max_runs) ? 64 : (n_rows <= 128 * max_runs ? 128 : 256);
        const int tiles = ceil_div(n_rows, R);
        const int nsplit = std::min(tiles, max_runs);
        p.tensor_core = 3;
        p.tile_rows = R;
        p.rows_per_split = ceil_div(tiles, nsplit) * R;
        p.nsplit = ceil_div(n_rows, p.rows_per_split);
        int cl = g_s.wide_cluster;
        if (cl != 1 && cl != 2 && cl != 4) cl = p.nsplit > 32 ? 4 : (p.nsplit > 16 ? 2 : 1);
        p.cluster = cl;
        p.npartial = ceil_div(p.nsplit, cl);
        return p;
    }
    const int tiles = ceil_div(n_rows > 0 ? n_rows : 0, kAttnTileRows);
    p.tensor_core = !tc_ok ? 0 : (attention_64_heads(n_rows) ? 2 : 1);
    // one wave of the 148 SMs: 64 splits x 2 column halves (128 heads per CTA), or 32 splits x 2 column halves x 2
    // head halves (64 heads per CTA)
    const int split_target = (p.tensor_core == 2) ? 32 : 64;
    int nsplit = tiles < split_target ? tiles : split_target;
    if (nsplit < 1) nsplit = (n_rows > 0) ? 1 : 0;
    p.rows_per_split = nsplit ? ceil_div(tiles, nsplit) * kAttnTileRows : 0;
    p.nsplit = p.rows_per_split ? ceil_div(n_rows, p.rows_per_split) : 0;
    p.npartial = p.tensor_core ? ceil_div(p.nsplit, kAttnCluster) : p.nsplit;
    return p;
}

static size_t attention_ws_bytes(int H, int kv_lora)
{
    return align_up((size_t)kMaxAttnSplits * H * 2 * sizeof(float), 256) + (size_t)kMaxAttnSplits * H * kv_lora * sizeof(float);
}

static AttnPartials carve_partials(void *ws, int H)
{
    AttnPartials part;
    part.ml = static_cast<float *>(ws);
    part.O = reinterpret_cast<float *>(static_cast<char *>(ws) + align_up((size_t)kMaxAttnSplits * H * 2 * sizeof(float), 256));
    return part;
}

template <typename... Args>
static cudaError_t launch_pdl(void (*kern)(Args...), dim3 grid, dim3 block, cudaStream_t s, bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

static int attention_partial(const void *Q, const void *cache, int H, int n_rows, int dc, int dr, float scale,
                             void *ws, size_t ws_bytes, cudaStream_t s, bool pdl = false, L2Prefetch prefetch = L2Prefetch{})
{
    if (!Q || !cache || !ws) return NM_ERR_INVALID_ARG;
    if (H < 1 || n_rows < 0 || dc != 512 || dr != 64) return NM_ERR_UNSUPPORTED;
    if (ws_bytes < attention_ws_bytes(H, dc)) return NM_ERR_WORKSPACE;
    if (n_rows == 0) return NM_OK;
    const AttnPlan p = plan_attention(Q, cache, H, n_rows, dc);
    AttnPartials part = carve_partials(ws, H);
    if (p.tensor_core == 3)
        return attention_partial_wide(Q, 1, &cache, &n_rows, &p.rows_per_split, p.nsplit, p.tile_rows, p.cluster, part, 0, scale, s, pdl, prefetch);
    if (p.tensor_core == 2)
        return attention_partial_tc64(Q, 1, &cache, &n_rows, &p.rows_per_split, p.nsplit, kAttnCluster, part, 0, scale, s, pdl, prefetch);
    if (p.tensor_core) return attention_partial_tc(Q, cache, part, p, n_rows, scale, s, pdl, prefetch);
    cudaError_t e = launch_pdl(attn_partial_simt_kernel, dim3(p.nsplit, H), dim3(128), s, pdl, static_cast<const uint16_t *>(Q),
                               static_cast<const uint16_t *>(cache), part, n_rows, p.rows_per_split, dc, dr, scale);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention (CUDA cores) launch");
}

static int attention_combine(const void *Q, const void *cache, void *o_bf16, float *o_f32, int H, int n_rows, long extra_row,
                             int dc, int dr, float scale, void *ws, size_t ws_bytes, cudaStream_t s, bool pdl = false)
{
    if (!Q || !cache || !ws || (!o_bf16 && !o_f32)) return NM_ERR_INVALID_ARG;
    if (H < 1 || n_rows < 0 || dc != 512 || dr != 64) return NM_ERR_UNSUPPORTED;
    if (n_rows == 0 && extra_row < 0) return NM_ERR_INVALID_ARG;
    if (ws_bytes < attention_ws_bytes(H, dc)) return NM_ERR_WORKSPACE;
    const AttnPlan p = plan_attention(Q, cache, H, n_rows, dc);
    cudaError_t e = launch_pdl(attn_combine_kernel, dim3(H), dim3(kCombineThreads), s, pdl, static_cast<const uint16_t *>(Q),
                               static_cast<const uint16_t *>(cache), carve_partials(ws, H), p.npartial, extra_row, dc, dr, scale,
                               static_cast<uint16_t *>(o_bf16), o_f32);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention combine launch");
}

// Workspace of the decode step: [main-stream matmul workspace][side-stream matmul workspace]
// [attention partials][intermediates].  Each matmul workspace is [64 KB counters][partials].
struct StepLayout {
    size_t main_ws, main_ws_bytes, side_ws, side_ws_bytes, attn, attn_bytes;
    size_t c_q, c_qn, q, q_full, ckr, o_lat, o, x_down, tile_ss, total;
};

static StepLayout step_layout(const nm_mla_params *p)
{
    StepLayout L{};
    const int dq = p->nope + p->rope, dkv = p->kv_lora + p->rope;
    size_t main_need = 0;
    auto upd = [&](int N, int K, int H) {
        const size_t b = nm_matmul_workspace_bytes(1, N, K, H, NM_BF16, NM_ROW_MAJOR);
        if (b > main_need) main_need = b;
    };
    upd(p->q_lora, p->d, 1); upd(p->q_lora + dkv, p->d, 1); upd(p->H * dq, p->q_lora, 1); upd(p->kv_lora, p->nope, p->H); upd(p->v, p->kv_lora, p->H);
    upd(p->d, p->H * p->v, 1);
    size_t off = 0;
    L.main_ws = off; L.main_ws_bytes = main_need; off += align_up(main_need, 256);
    L.side_ws = off; L.side_ws_bytes = nm_matmul_workspace_bytes(1, dkv, p->d, 1, NM_BF16, NM_ROW_MAJOR);
    off += align_up(L.side_ws_bytes, 256);
    L.attn = off; L.attn_bytes = attention_ws_bytes(p->H, p->kv_lora); off += align_up(L.attn_bytes, 256);
    auto take = [&](size_t elems) { size_t o = off; off += align_up(elems * 2, 256); return o; };
    L.c_q = take(p->q_lora); L.c_qn = take(p->q_lora); L.q = take((size_t)p->H * dq); L.q_full = take((size_t)p->H * dkv);
    L.ckr = take(dkv); L.o_lat = take((size_t)p->H * p->kv_lora); L.o = take((size_t)p->H * p->v);
    L.x_down = take((size_t)p->q_lora + dkv);
    L.tile_ss = take(2 * (size_t)(ceil_div(p->q_lora + dkv, 64) + 64));     // one float per 64-column tile of the fused down-projection
    L.total = off;
    return L;
}

static int check_params(const nm_mla_params *p)
{
    if (!p) return NM_ERR_INVALID_ARG;
    if (!p->h || !p->gamma_q || !p->W_UQR || !p->gamma_kv || !p->W_UK || !p->W_UV || !p->rope_cos_sin || !p->kv_cache || !p->workspace)
        return NM_ERR_INVALID_ARG;
    if (!p->W_DQKV && (!p->W_DQ || !p->W_DKVKR)) return NM_ERR_INVALID_ARG;
    if (p->W_O && !p->out) return NM_ERR_INVALID_ARG;
    if (p->d < 1 || p->q_lora < 1 || p->H < 1 || p->nope < 1 || p->v < 1 || p->seq_len < 1) return NM_ERR_INVALID_ARG;
    if (p->kv_lora != 512 || p->rope != 64) return NM_ERR_UNSUPPORTED;
    if (p->q_lora > 16384) return NM_ERR_UNSUPPORTED;
    if (p->layout_dense != NM_ROW_MAJOR && p->layout_dense != NM_COL_MAJOR && p->layout_dense != NM_FRACTAL_NZ) return NM_ERR_UNSUPPORTED;
    return NM_OK;
}

// Tuning aid: slice of the trace buffer (see set_attention_trace) for one product of the step.
static unsigned long long *trace_at(size_t offset) { return attention_trace() ? attention_trace() + offset : nullptr; }

// Tuning aid: a forced plan around one product of the step.
struct ScopedPlan {
    bool on;
    explicit ScopedPlan(const int (&f)[3]) : on(f[0] || f[1] || f[2]) { if (on) set_thread_plan_override(true, f[0], f[1], f[2]); }
    ~ScopedPlan() { if (on) set_thread_plan_override(false, 0, 0, 0); }
};

#define NM_TRY(expr) do { int _rc = (expr); if (_rc != NM_OK) return _rc; } while (0)
#define NM_LAUNCH_CHECK(what) do { cudaError_t _e = cudaGetLastError(); if (_e != cudaSuccess) return record_cuda_error(_e, what); } while (0)

// Events used to fork the KV chain onto the side stream and join it again (created once per thread).
struct StepEvents { cudaEvent_t fork = nullptr, join = nullptr; };
static thread_local StepEvents g_events;

static int step_impl(const nm_mla_params *p, cudaStream_t ms, cudaStream_t ss)
{
    refresh_step_tuning();
    NM_TRY(check_params(p));
    const StepLayout L = step_layout(p);
    if (p->workspace_bytes < L.total) return NM_ERR_WORKSPACE;
    if (((uintptr_t)p->workspace & 255u) != 0) return NM_ERR_ALIGNMENT;
    char *ws = static_cast<char *>(p->workspace);
    const int d = p->d, ql = p->q_lora, dc = p->kv_lora, dr = p->rope, dn = p->nope, dv = p->v, H = p->H;
    const int dq = dn + dr, dkv = dc + dr;
    const long pos = (long)p->seq_len - 1;
    const nm_layout lay = (nm_layout)p->layout_dense;
    auto buf = [&](void *user, size_t off) { return user ? user : static_cast<void *>(ws + off); };
    uint16_t *c_q = (uint16_t *)buf(p->c_q, L.c_q), *c_qn = (uint16_t *)buf(p->c_qn, L.c_qn), *q = (uint16_t *)buf(p->q, L.q);
    uint16_t *q_full = (uint16_t *)buf(p->q_full, L.q_full), *ckr = (uint16_t *)buf(p->ckr, L.ckr);
    uint16_t *o_lat = (uint16_t *)buf(p->o_lat, L.o_lat), *o = (uint16_t *)buf(p->o, L.o);
    uint16_t *cache = static_cast<uint16_t *>(p->kv_cache);
    void *mws = ws + L.main_ws, *sws = ws + L.side_ws, *aws = ws + L.attn;
    const bool forked = (ss != ms) && !(p->W_DQKV && p->layout_dense != NM_COL_MAJOR && down_finish_applies(p->q_lora, p->kv_lora, p->rope));
    if (forked && !g_events.fork) {
        NM_CUDA_TRY(cudaEventCreateWithFlags(&g_events.fork, cudaEventDisableTiming));
        NM_CUDA_TRY(cudaEventCreateWithFlags(&g_events.join, cudaEventDisableTiming));
    }

    // Programmatic dependent launch inside the step: every kernel after the first on its stream may
    // start (and, for the products, prefetch its weights) while its predecessor drains; each waits
    // for the predecessor before it reads activations or writes.  The first kernel on each stream
    // keeps the ordinary dependency on whatever the caller enqueued before the step.
    const bool pdl = g_s.step_pdl != 0;
#define NM_LAUNCH(kern, grid, block, stream, ...)                                             \
    do {                                                                                      \
        cudaError_t _e = launch_pdl(kern, dim3(grid), dim3(block), stream, pdl, __VA_ARGS__); \
        if (_e != cudaSuccess) return record_cuda_error(_e, #kern);                           \
    } while (0)

    // The vector stages behind the down-projections (RMSNorm of the query latent; RMSNorm, RoPE and the cache-row
    // write of the KV part) run inside the product that feeds them, in the CTA that completes its last tile,
    // when that product is the TMA ring kernel; otherwise as kernels of their own.
    const bool tails_ok = g_s.fused_tails && down_finish_applies(ql, dc, dr);
    VecTail tq{}, tkv{};
    tq.enabled = 1; tq.q_lora = ql; tq.eps = p->rms_eps; tq.gamma_q = (const uint16_t *)p->gamma_q; tq.c_qn = c_qn;
    tkv.enabled = 1; tkv.kv_off = 0; tkv.dc = dc; tkv.rope = dr; tkv.eps = p->rms_eps; tkv.gamma_kv = (const uint16_t *)p->gamma_kv;
    tkv.cos_sin = p->rope_cos_sin; tkv.cache_row = cache + (size_t)pos * dkv;
    bool taken = false;
    // The KV chain of the two-stream schedule: the paper's MatMul 2 (h * (W_DKV | W_KR)) with RMSNorm, RoPE and the cache-row
    // write in its completion, on the side stream.  Forked at the start of the step it shares the machine with the first
    // product of the Q chain; forked when the attention operand is ready (kv_beside_attention) it is a narrow CUDA-core
    // product running on the SMs the attention pass leaves free while the tensor cores work - the paper's schedule
    // (vector units beside the cube unit), and legal because the pass attends the OLD rows only: the new row joins in the merge.
    const bool kv_late = forked && g_s.kv_beside_attention;
    auto enqueue_kv_chain = [&]() -> int {
        bool kv_taken = false;
        if (forked) {
            NM_CUDA_TRY(cudaEventRecord(g_events.fork, ms));
            NM_CUDA_TRY(cudaStreamWaitEvent(ss, g_events.fork, 0));
        }
        NM_TRY(matmul_enqueue(p->h, p->W_DKVKR, ckr, 1, dkv, d, 1, d, 0, 0, dkv, 0, NM_BF16, lay, sws, L.side_ws_bytes, ss, false, nullptr,
                              tails_ok ? &tkv : nullptr, &kv_taken, false));
        if (!kv_taken)
            NM_LAUNCH(kv_finish_kernel, 1, 256, ss, (const uint16_t *)ckr, (const uint16_t *)p->gamma_kv, p->rope_cos_sin,
                      cache + (size_t)pos * dkv, dc, dr, p->rms_eps);
        if (forked) NM_CUDA_TRY(cudaEventRecord(g_events.join, ss));
        return NM_OK;
    };
    const bool fused_down = p->W_DQKV && lay != NM_COL_MAJOR && down_finish_applies(ql, dc, dr);      // row-major or fractal storage
    // Where the plans allow: the k-splits of the fused down-projection meet inside clusters, each
    // tile leaves the sum of squares of its outputs, the W_UQR product applies RMSNorm to its token row while
    // loading it, and the KV consumers ride in an extra CTA of the per-head query kernel - the down-projection then
    // ends without a grid-wide gather, which cost it 4 us at the head of the step's critical path.
    bool split_norm = false;
    RowNorm rn{};
    KvFinish kvf{};
    float *tile_ss = reinterpret_cast<float *>(ws + L.tile_ss);
    if (fused_down && tails_ok && g_s.fused_tails == 1 && g_s.fused_heads && head_kernels_apply(H, dn, dr, dc, dv)) {
        uint16_t *x_down = reinterpret_cast<uint16_t *>(ws + L.x_down);
        MatmulExtras ex_d, ex_u;
        ex_d.tile_ss = tile_ss; ex_d.dry_run = true;
        {
            ScopedPlan sp(g_s.step_plan[0]);
            NM_TRY(matmul_enqueue(p->h, p->W_DQKV, x_down, 1, ql + dkv, d, 1, d, 0, 0, ql + dkv, 0, NM_BF16, lay, mws,
                                  L.main_ws_bytes, ms, false, nullptr, nullptr, nullptr, true, &ex_d));
        }
        if (ex_d.tile_ss_taken && ex_d.tile_n > 0 && ql % ex_d.tile_n == 0 && ql / ex_d.tile_n <= 32) {
            rn.enabled = 1; rn.n = ql; rn.ntiles = ql / ex_d.tile_n; rn.eps = p->rms_eps; rn.tile_ss = tile_ss;
            rn.gamma = (const uint16_t *)p->gamma_q; rn.normed_out = c_qn;
            ex_u.norm = &rn; ex_u.dry_run = true;
            ScopedPlan sp(g_s.step_plan[1]);
            NM_TRY(matmul_enqueue(x_down, p->W_UQR, q, 1, H * dq, ql, 1, ql, 0, 0, H * dq, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms, false,
                                  nullptr, nullptr, nullptr, true, &ex_u));
            split_norm = ex_u.norm_taken;
        }
    }
    if (split_norm) {
        uint16_t *x_down = reinterpret_cast<uint16_t *>(ws + L.x_down);
        MatmulExtras ex_d;
        ex_d.tile_ss = tile_ss;
        {
            ScopedPlan sp(g_s.step_plan[0]);
            NM_TRY(matmul_enqueue(p->h, p->W_DQKV, x_down, 1, ql + dkv, d, 1, d, 0, 0, ql + dkv, 0, NM_BF16, lay, mws,
                                  L.main_ws_bytes, ms, pdl && p->programmatic_entry, trace_at(2048), nullptr, nullptr, true, &ex_d));
        }
        if (!ex_d.tile_ss_taken) return NM_ERR_UNSUPPORTED;        // the dry run said otherwise
        kvf.enabled = 1; kvf.ckr = x_down + ql; kvf.gamma = (const uint16_t *)p->gamma_kv; kvf.cos_sin = p->rope_cos_sin;
        kvf.cache_row = cache + (size_t)pos * dkv; kvf.dc = dc; kvf.rope = dr; kvf.eps = p->rms_eps;
        if (p->c_q) NM_CUDA_TRY(cudaMemcpyAsync(p->c_q, x_down, (size_t)ql * 2, cudaMemcpyDeviceToDevice, ms));
        if (p->ckr) NM_CUDA_TRY(cudaMemcpyAsync(p->ckr, x_down + ql, (size_t)dkv * 2, cudaMemcpyDeviceToDevice, ms));
    } else if (fused_down) {
        // ---- one product for all three down-projections, h * (W_DQ | W_DKV | W_KR) (Eq. 3 extended by W_DQ),
        //      with both vector stages in its completion: no side stream, an unbroken programmatic chain
        uint16_t *x_down = reinterpret_cast<uint16_t *>(ws + L.x_down);
        VecTail both = tq;
        both.kv_off = ql; both.dc = dc; both.rope = dr; both.gamma_kv = tkv.gamma_kv; both.cos_sin = tkv.cos_sin; both.cache_row = tkv.cache_row;
        ScopedPlan sp(g_s.step_plan[0]);
        NM_TRY(matmul_enqueue(p->h, p->W_DQKV, x_down, 1, ql + dkv, d, 1, d, 0, 0, ql + dkv, 0, NM_BF16, lay, mws,
                              L.main_ws_bytes, ms, pdl && p->programmatic_entry, trace_at(2048), tails_ok ? &both : nullptr, &taken, true));
        if (!taken)
            NM_TRY(launch_down_finish(x_down, p->gamma_q, p->gamma_kv, p->rope_cos_sin, c_qn, cache + (size_t)pos * dkv, ql, dc, dr,
                                      p->rms_eps, ms, pdl));
        if (p->c_q) NM_CUDA_TRY(cudaMemcpyAsync(p->c_q, x_down, (size_t)ql * 2, cudaMemcpyDeviceToDevice, ms));
        if (p->ckr) NM_CUDA_TRY(cudaMemcpyAsync(p->ckr, x_down + ql, (size_t)dkv * 2, cudaMemcpyDeviceToDevice, ms));
    } else {
        // ---- KV chain (the paper's MatMul 2 and its consumers) on the side stream, forked at the start so that
        //      it shares the machine with the first product of the Q chain and is long done when the merge
        //      needs the new cache row -------------------------------------------------------------------------
        if (!kv_late) NM_TRY(enqueue_kv_chain());

        // ---- Q chain, main stream ----------------------------------------------------------------------------
        NM_TRY(matmul_enqueue(p->h, p->W_DQ, c_q, 1, ql, d, 1, d, 0, 0, ql, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms,
                              pdl && (!forked || p->programmatic_entry), nullptr, tails_ok ? &tq : nullptr, &taken, !forked));
        if (!taken) NM_LAUNCH(rmsnorm_kernel, 1, 256, ms, (const uint16_t *)c_q, (const uint16_t *)p->gamma_q, c_qn, ql, p->rms_eps);
    }
    {
        ScopedPlan sp(g_s.step_plan[1]);
        MatmulExtras ex_u;
        ex_u.norm = &rn;
        const uint16_t *a_row = split_norm ? reinterpret_cast<const uint16_t *>(ws + L.x_down) : c_qn;
        NM_TRY(matmul_enqueue(a_row, p->W_UQR, q, 1, H * dq, ql, 1, ql, 0, 0, H * dq, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms, pdl, trace_at(4096),
                              nullptr, nullptr, true, split_norm ? &ex_u : nullptr));
        if (split_norm && !ex_u.norm_taken) return NM_ERR_UNSUPPORTED;
    }
    const bool fused = g_s.fused_heads && head_kernels_apply(H, dn, dr, dc, dv);
    if (fused) {
        // RoPE of the rope part and q_lat[h] = q[h, :nope] * W_UK[h] in one kernel, one CTA per head
        NM_TRY(launch_q_finish(q, p->W_UK, p->rope_cos_sin, q_full, H, dr, ms, pdl, kvf));
    } else {
        NM_LAUNCH(rope_kernel, ceil_div(H * dr / 2, 256), 256, ms, (const uint16_t *)(q + dn), q_full + dc, H, dr, (long)dq, (long)dkv,
                  p->rope_cos_sin);
        // q_lat[h] = q[h, :nope] * W_UK[h], written straight into the attention operand [H][dc+dr]
        NM_TRY(matmul_enqueue(q, p->W_UK, q_full, 1, dc, dn, H, (long)H * dq, dq, (long)dn * dc, (long)H * dkv, dkv,
                              NM_BF16, NM_ROW_MAJOR, mws, L.main_ws_bytes, ms, pdl));
    }

    // ---- beside the attention pass: W_UV and the head of every k-split of W_O are pulled into L2, so that the
    //      output-side products start from L2 instead of HBM (Data Independence: the weights do not depend on
    //      the attention result) ---------------------------------------------------------------------------------
    L2Prefetch pf{};
    if (g_s.prefetch_mb > 0 && pos > 0) {
        pf.block = (const char *)p->W_UV;
        pf.block_bytes = g_s.prefetch_uv ? (long)H * dc * dv * 2 : 0;
        if (p->W_O && lay == NM_ROW_MAJOR) {
            int kr = 0, ns = 1;
            {
                ScopedPlan sp(g_s.step_plan[2]);
                matmul_row_major_split(1, d, H * dv, 1, &kr, &ns, true);
            }
            const long row_bytes = (long)d * 2;
            long rows = ((long)g_s.prefetch_mb << 20) / ns / row_bytes;
            if (rows > kr) rows = kr;
            pf.base = (const char *)p->W_O; pf.range_stride = (long)kr * row_bytes; pf.nranges = rows > 0 ? ns : 0;
            pf.range_bytes = rows * row_bytes;
        } else if (p->W_O && lay == NM_FRACTAL_NZ) {
            // fractal storage: every fractal column (16 columns, all K rows) is contiguous; the product starts each of
            // them at row 0, so the head of every fractal column is what it reads first
            const long K_o = (long)H * dv, cols = d / 16;
            long rows = (((long)g_s.prefetch_mb << 20) / cols / 32) / 16 * 16;
            if (rows > K_o) rows = K_o;
            pf.base = (const char *)p->W_O; pf.range_stride = K_o * 32; pf.nranges = rows > 0 ? (int)cols : 0;
            pf.range_bytes = rows * 32;
        }
    }

    if (kv_late) NM_TRY(enqueue_kv_chain());       // from here on the side stream runs beside the attention pass
    // ---- attention over the old rows (tensor cores), main stream; the new row joins in the merge -----------
    // When the merge kernel is launched programmatically it sits beside the attention CTAs from their start and
    // issues the prefetch itself (its threads are idle until the attention result exists); otherwise a warp of
    // the attention kernel does.
    const bool uv_early = fused && pdl && !forked && g_s.uv_pdl;
    NM_TRY(attention_partial(q_full, cache, H, (int)pos, dc, dr, p->softmax_scale, aws, L.attn_bytes, ms, pdl, uv_early ? L2Prefetch{} : pf));
    // The merge needs the cache row the KV chain wrote (two-stream schedule): the join sits right before it, where
    // it breaks only the merge's programmatic launch.
    if (forked) NM_CUDA_TRY(cudaStreamWaitEvent(ms, g_events.join, 0));
    if (fused) {
        // merge of the attention partials (+ the new row) and o[h] = o_lat[h] * W_UV[h] in one kernel
        const AttnPlan ap = plan_attention(q_full, cache, H, (int)pos, dc);
        NM_TRY(launch_uv_merge(q_full, cache, carve_partials(aws, H), ap.npartial, pos, dr, p->softmax_scale, p->W_UV, o_lat,
                               p->o_lat_f32, o, H, ms, uv_early, uv_early ? pf : L2Prefetch{}));
    } else {
        NM_TRY(attention_combine(q_full, cache, o_lat, p->o_lat_f32, H, (int)pos, pos, dc, dr, p->softmax_scale, aws, L.attn_bytes, ms,
                                 pdl && !forked));
        NM_TRY(matmul_enqueue(o_lat, p->W_UV, o, 1, dv, dc, H, (long)H * dc, dc, (long)dc * dv, (long)H * dv, dv,
                              NM_BF16, NM_ROW_MAJOR, mws, L.main_ws_bytes, ms, pdl));
    }
    if (p->W_O) {
        if (p->event_before_wo) NM_CUDA_TRY(cudaEventRecord((cudaEvent_t)p->event_before_wo, ms));
        ScopedPlan sp(g_s.step_plan[2]);
        NM_TRY(matmul_enqueue(o, p->W_O, p->out, 1, d, H * dv, 1, (long)H * dv, 0, 0, d, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms,
                              pdl && !p->event_before_wo, trace_at(6144), nullptr, nullptr, true));
        if (p->event_after_wo) NM_CUDA_TRY(cudaEventRecord((cudaEvent_t)p->event_after_wo, ms));
    }
#undef NM_LAUNCH
    return NM_OK;
}

// ---- small-batch decode: T independent sequences, one new token each ------------------------------------------
struct BatchLayout {
    size_t mws, mws_bytes, attn_ml, attn_o, x_down, c_qn, q, q_full, o_lat, o, total;
    int slot_stride;
};

static BatchLayout batch_layout(const nm_mla_params *p, int T)
{
    BatchLayout L{};
    const int dq = p->nope + p->rope, dkv = p->kv_lora + p->rope, H = p->H;
    size_t need = 0;
    auto upd = [&](int N, int K) {
        const size_t b = nm_matmul_workspace_bytes(T, N, K, 1, NM_BF16, NM_ROW_MAJOR);
        if (b > need) need = b;
    };
    upd(p->q_lora + dkv, p->d); upd(p->q_lora, p->d); upd(dkv, p->d); upd(H * dq, p->q_lora); upd(p->d, H * p->v);
    size_t off = 0;
    L.mws = off; L.mws_bytes = need; off += align_up(need, 256);
    L.slot_stride = 16;                                            // at most 64 splits in clusters of four per sequence
    L.attn_ml = off; off += align_up((size_t)T * L.slot_stride * H * 2 * sizeof(float), 256);
    L.attn_o = off; off += align_up((size_t)T * L.slot_stride * H * p->kv_lora * sizeof(float), 256);
    auto take = [&](size_t elems) { size_t o = off; off += align_up(elems * 2, 256); return o; };
    L.x_down = take((size_t)T * (p->q_lora + dkv)); L.c_qn = take((size_t)T * p->q_lora); L.q = take((size_t)T * H * dq);
    L.q_full = take((size_t)T * H * dkv); L.o_lat = take((size_t)T * H * p->kv_lora); L.o = take((size_t)T * H * p->v);
    L.total = off;
    return L;
}

static int batch_check(const nm_mla_params *p, const nm_mla_batch *b)
{
    if (!p || !b) return NM_ERR_INVALID_ARG;
    if (b->T < 1 || !b->seq_lens || !b->h || !b->rope_cos_sin || !b->kv_cache) return NM_ERR_INVALID_ARG;
    if (b->T > kMaxBatch) return NM_ERR_UNSUPPORTED;
    if (!p->gamma_q || !p->W_UQR || !p->gamma_kv || !p->W_UK || !p->W_UV || !p->workspace) return NM_ERR_INVALID_ARG;
    if (!p->W_DQKV && (!p->W_DQ || !p->W_DKVKR)) return NM_ERR_INVALID_ARG;
    if (p->W_O && !b->out) return NM_ERR_INVALID_ARG;
    if (p->d < 1 || p->q_lora < 1 || p->H < 1) return NM_ERR_INVALID_ARG;
    if (p->kv_lora != 512 || p->rope != 64 || p->nope != 128 || p->v != 128 || p->H != 128) return NM_ERR_UNSUPPORTED;
    if (!down_finish_applies(p->q_lora, p->kv_lora, p->rope)) return NM_ERR_UNSUPPORTED;
    if (p->layout_dense != NM_ROW_MAJOR && p->layout_dense != NM_COL_MAJOR) return NM_ERR_UNSUPPORTED;
    const long row = p->kv_lora + p->rope;
    for (int t = 0; t < b->T; ++t) {
        if (b->seq_lens[t] < 1) return NM_ERR_INVALID_ARG;
        if (b->T > 1 && b->cache_stride < (long)b->seq_lens[t] * row) return NM_ERR_INVALID_ARG;
    }
    if (b->cache_stride % 8 != 0) return NM_ERR_ALIGNMENT;           // every sequence's cache stays 16-byte aligned
    return NM_OK;
}

static int batch_impl(const nm_mla_params *p, const nm_mla_batch *b, cudaStream_t ms)
{
    refresh_step_tuning();
    NM_TRY(batch_check(p, b));
    const int T = b->T;
    const BatchLayout L = batch_layout(p, T);
    if (p->workspace_bytes < L.total) return NM_ERR_WORKSPACE;
    if (((uintptr_t)p->workspace & 255u) != 0) return NM_ERR_ALIGNMENT;
    char *ws = static_cast<char *>(p->workspace);
    const int d = p->d, ql = p->q_lora, dc = p->kv_lora, dr = p->rope, dn = p->nope, dv = p->v, H = p->H;
    const int dq = dn + dr, dkv = dc + dr;
    const nm_layout lay = (nm_layout)p->layout_dense;
    uint16_t *x_down = (uint16_t *)(ws + L.x_down), *c_qn = (uint16_t *)(ws + L.c_qn), *q = (uint16_t *)(ws + L.q);
    uint16_t *q_full = (uint16_t *)(ws + L.q_full), *o_lat = (uint16_t *)(ws + L.o_lat), *o = (uint16_t *)(ws + L.o);
    uint16_t *cache = static_cast<uint16_t *>(b->kv_cache);
    void *mws = ws + L.mws;
    const bool pdl = g_s.step_pdl != 0;

    // split plan of the attention pass: the same number of splits for every sequence, about 128 CTAs in all
    long total_rows = 0;
    for (int t = 0; t < T; ++t) total_rows += b->seq_lens[t];
    // 64 heads per CTA (four CTAs per split) while the batch is short enough.  Every sequence gets the same number of
    // splits; all clusters are resident at once (clusters do not straddle GPCs: fewer fit than SMs / size).  Of the split counts that fit, the one with the fewest tiles per
    // CTA on the longest sequence is taken - among equals the one divisible by four, then by two (the splits merged on
    // chip form a cluster of 4, 2 or 1), then the smallest; at most 16 partials per sequence reach the final merge.
    const bool tc64 = attention_64_heads(total_rows) && T * 4 <= kSMsAttn;
    int nsplit = (64 / T) / kAttnCluster * kAttnCluster, cluster = kAttnCluster, ragged_tiles = 0;
    if (nsplit < kAttnCluster) nsplit = kAttnCluster;
    if (tc64) {
        int max_rows = 1;
        for (int t = 0; t < T; ++t) max_rows = std::max(max_rows, b->seq_lens[t] - 1);
        const int max_tiles = ceil_div(max_rows, kAttnTileRows), fit = std::min(32, kSMsAttn / (4 * T));
        int best = 1, best_tiles = max_tiles, best_cl = 1;
        for (int ns = 1; ns <= fit; ++ns) {
            const int cl = ns % 4 == 0 ? 4 : (ns % 2 == 0 ? 2 : 1), tiles = ceil_div(max_tiles, ns);
            if (ns / cl > L.slot_stride) continue;
            int cap = attention_tc64_max_clusters(cl);
            if (cap <= 0) cap = 128 / cl;                              // the query failed: a count that always fits
            if ((long)T * 4 * (ns / cl) > cap) continue;               // a second wave of clusters costs more than it saves
            if (tiles < best_tiles || (tiles == best_tiles && cl > best_cl)) { best = ns; best_tiles = tiles; best_cl = cl; }
        }
        nsplit = best; cluster = best_cl;
        // Sequences of unequal length: the same ROWS per split for every sequence instead (a short sequence then takes
        // few CTAs, the surplus CTAs of its grid row find no rows and leave at once - which only costs nothing when no
        // cluster peer waits for them, so without the on-chip merge).  Taken when it shortens the longest run of tiles.
        for (int tau = std::max(1, ceil_div(max_tiles, L.slot_stride)); tau < best_tiles; ++tau) {
            long ctas = 0;
            for (int t = 0; t < T; ++t) ctas += 4L * ceil_div(std::max(0, b->seq_lens[t] - 1), tau * kAttnTileRows);
            if (ctas <= kSMsAttn) { ragged_tiles = tau; nsplit = ceil_div(max_tiles, tau); cluster = 1; break; }
        }
    }
    // The wide-tile kernel (all heads per CTA, two CTAs per row run): every sequence gets the same number of runs, as many as
    // keep the whole batch in one wave of CTAs (at most 16: the partial slots of a sequence); a run goes through its rows
    // in tiles as wide as its share of the longest sequence needs.  Runs stand alone (no on-chip merge), so the surplus
    // CTAs of a short sequence leave at once.
    const bool wide = (g_s.attn_impl == 0 || g_s.attn_impl == 4) && T * 2 <= kSMsAttn;
    int wide_tile = 64;
    if (wide) {
        int max_rows = 1;
        for (int t = 0; t < T; ++t) max_rows = std::max(max_rows, b->seq_lens[t] - 1);
        const int runs_cap = std::max(1, std::min(L.slot_stride, kSMsAttn / (2 * T)));
        const int share = ceil_div(max_rows, runs_cap);
        wide_tile = g_s.wide_tile == 64 || g_s.wide_tile == 128 || g_s.wide_tile == 256 ? g_s.wide_tile : (share <= 64 ? 64 : (share <= 128 ? 128 : 256));
        nsplit = std::min(runs_cap, ceil_div(max_rows, wide_tile));
        cluster = 1; ragged_tiles = 0;
    }
    BatchRows rows{};
    rows.slot_stride = L.slot_stride;
    const void *caches[kMaxBatch];
    int n_rows[kMaxBatch], rps[kMaxBatch];
    bool any_rows = false;
    for (int t = 0; t < T; ++t) {
        const long base = (long)t * b->cache_stride;
        caches[t] = cache + base;
        n_rows[t] = b->seq_lens[t] - 1;
        rows.new_row[t] = base + (long)n_rows[t] * dkv;
        const int tile_rows = wide ? wide_tile : kAttnTileRows;
        const int tiles = ceil_div(n_rows[t], tile_rows);
        rps[t] = ragged_tiles ? ragged_tiles * kAttnTileRows : (tiles > 0 ? ceil_div(tiles, nsplit) * tile_rows : tile_rows);
        rows.npart[t] = n_rows[t] > 0 ? ceil_div(ceil_div(n_rows[t], rps[t]), cluster) : 0;
        any_rows |= n_rows[t] > 0;
    }

    // ---- down-projections of all T tokens: the weights are streamed once ---------------------------------------
    // The first product may start (and fill its ring with weights) under whatever the caller enqueued before the step
    // when the caller says so (programmatic_entry: back-to-back steps or layers, static weights), as in the single-token step.
    const bool entry_pdl = pdl && p->programmatic_entry;
    if (p->W_DQKV && lay == NM_ROW_MAJOR) {
        NM_TRY(matmul_enqueue(b->h, p->W_DQKV, x_down, T, ql + dkv, d, 1, d, 0, 0, ql + dkv, 0, NM_BF16, NM_ROW_MAJOR, mws, L.mws_bytes, ms,
                              entry_pdl, nullptr, nullptr, nullptr, true));
    } else {
        NM_TRY(matmul_enqueue(b->h, p->W_DQ, x_down, T, ql, d, 1, d, 0, 0, ql + dkv, 0, NM_BF16, lay, mws, L.mws_bytes, ms,
                              entry_pdl, nullptr, nullptr, nullptr, true));
        NM_TRY(matmul_enqueue(b->h, p->W_DKVKR, x_down + ql, T, dkv, d, 1, d, 0, 0, ql + dkv, 0, NM_BF16, lay, mws, L.mws_bytes, ms,
                              pdl, nullptr, nullptr, nullptr, true));
    }
    NM_TRY(launch_down_finish_batch(x_down, p->gamma_q, p->gamma_kv, b->rope_cos_sin, c_qn, cache, rows, T, ql, dc, dr, p->rms_eps, ms, pdl));
    NM_TRY(matmul_enqueue(c_qn, p->W_UQR, q, T, H * dq, ql, 1, ql, 0, 0, H * dq, 0, NM_BF16, lay, mws, L.mws_bytes, ms, pdl, nullptr, nullptr,
                          nullptr, true));
    // From three tokens on the per-head products (128 x 512 and 512 x 128 per head and token) go to the batched swap-AB
    // tensor-core kernel, with RoPE and the merge as small kernels of their own: in the fused per-head kernels one
    // CTA per head walks every token and is bound by fp32 FMA issue and by its chain of L2 round trips (measured at
    // 4096 rows: 108 vs 112 us at T = 3, 114 vs 115 at T = 4, 133 vs 139 at T = 6, 183 vs 204 at T = 16; level at T = 2).
    const bool per_head_tc = T >= g_s.batch_tc_min_t || !g_s.fused_heads;
    if (per_head_tc) {
        NM_TRY(launch_rope_batch(q, b->rope_cos_sin, q_full, H, dn, dc, dr, T, ms, pdl));
        NM_TRY(matmul_enqueue(q, p->W_UK, q_full, T, dc, dn, H, (long)H * dq, dq, (long)dn * dc, (long)H * dkv, dkv, NM_BF16, NM_ROW_MAJOR,
                              mws, L.mws_bytes, ms, pdl));
    } else {
        NM_TRY(launch_q_finish_batch(q, p->W_UK, b->rope_cos_sin, q_full, H, dr, T, ms, pdl));
    }
    AttnPartials part;
    part.ml = reinterpret_cast<float *>(ws + L.attn_ml);
    part.O = reinterpret_cast<float *>(ws + L.attn_o);
    if (any_rows) {
        if (tensor_map_encoder() == nullptr) return NM_ERR_UNSUPPORTED;
        // beside the attention pass (a spare warp of its CTAs): W_UV and the head of every k-split of W_O into L2, as in
        // the single-token step
        L2Prefetch pf{};
        if (g_s.prefetch_mb > 0) {
            pf.block = (const char *)p->W_UV;
            pf.block_bytes = g_s.prefetch_uv ? (long)H * dc * dv * 2 : 0;
            if (p->W_O && lay == NM_ROW_MAJOR) {
                int kr = 0, ns = 1;
                matmul_row_major_split(T, d, H * dv, 1, &kr, &ns, true);
                const long row_bytes = (long)d * 2;
                long prows = ((long)g_s.prefetch_mb << 20) / ns / row_bytes;
                if (prows > kr) prows = kr;
                pf.base = (const char *)p->W_O; pf.range_stride = (long)kr * row_bytes; pf.nranges = prows > 0 ? ns : 0;
                pf.range_bytes = prows * row_bytes;
            }
        }
        if (wide)
            NM_TRY(attention_partial_wide(q_full, T, caches, n_rows, rps, nsplit, wide_tile, 1, part, L.slot_stride, p->softmax_scale, ms, pdl, pf));
        else if (tc64)
            NM_TRY(attention_partial_tc64(q_full, T, caches, n_rows, rps, nsplit, cluster, part, L.slot_stride, p->softmax_scale, ms, pdl, pf));
        else
            NM_TRY(attention_partial_tc_batch(q_full, T, caches, n_rows, rps, nsplit, part, L.slot_stride, p->softmax_scale, ms, pdl, pf));
    }
    if (per_head_tc) {
        NM_TRY(launch_attn_merge_batch(q_full, cache, part, rows, T, dr, p->softmax_scale, o_lat, H, ms, pdl));
        NM_TRY(matmul_enqueue(o_lat, p->W_UV, o, T, dv, dc, H, (long)H * dc, dc, (long)dc * dv, (long)H * dv, dv, NM_BF16, NM_ROW_MAJOR,
                              mws, L.mws_bytes, ms, pdl));
    } else {
        NM_TRY(launch_uv_merge_batch(q_full, cache, part, rows, T, dr, p->softmax_scale, p->W_UV, o_lat, o, H, ms, pdl));
    }
    if (p->W_O)
        NM_TRY(matmul_enqueue(o, p->W_O, b->out, T, d, H * dv, 1, (long)H * dv, 0, 0, d, 0, NM_BF16, lay, mws, L.mws_bytes, ms, pdl, nullptr,
                              nullptr, nullptr, true));
    if (b->o_lat) NM_CUDA_TRY(cudaMemcpyAsync(b->o_lat, o_lat, (size_t)T * H * dc * 2, cudaMemcpyDeviceToDevice, ms));
    if (b->o) NM_CUDA_TRY(cudaMemcpyAsync(b->o, o, (size_t)T * H * dv * 2, cudaMemcpyDeviceToDevice, ms));
    if (b->q_full) NM_CUDA_TRY(cudaMemcpyAsync(b->q_full, q_full, (size_t)T * H * dkv * 2, cudaMemcpyDeviceToDevice, ms));
    // stage outputs of the query side and the raw KV product, token by token out of the [T][q_lora + kv_lora + rope] rows
    if (b->c_q) NM_CUDA_TRY(cudaMemcpy2DAsync(b->c_q, (size_t)ql * 2, x_down, (size_t)(ql + dkv) * 2, (size_t)ql * 2, T, cudaMemcpyDeviceToDevice, ms));
    if (b->ckr) NM_CUDA_TRY(cudaMemcpy2DAsync(b->ckr, (size_t)dkv * 2, x_down + ql, (size_t)(ql + dkv) * 2, (size_t)dkv * 2, T, cudaMemcpyDeviceToDevice, ms));
    if (b->c_qn) NM_CUDA_TRY(cudaMemcpyAsync(b->c_qn, c_qn, (size_t)T * ql * 2, cudaMemcpyDeviceToDevice, ms));
    if (b->q) NM_CUDA_TRY(cudaMemcpyAsync(b->q, q, (size_t)T * H * dq * 2, cudaMemcpyDeviceToDevice, ms));
    return NM_OK;
}

}  // namespace nm

using namespace nm;

extern "C" {
#pragma GCC visibility push(default)

int nm_rmsnorm(const void *x, const void *gamma, void *y, int n, float eps, nm_stream stream)
{
    if (!x || !gamma || !y || n < 1) return NM_ERR_INVALID_ARG;
    if (n > 16384) return NM_ERR_UNSUPPORTED;
    rmsnorm_kernel<<<1, 256, 0, (cudaStream_t)stream>>>((const uint16_t *)x, (const uint16_t *)gamma, (uint16_t *)y, n, eps);
    NM_LAUNCH_CHECK("rmsnorm launch");
    return NM_OK;
}

int nm_rope(const void *x, void *y, int n_vec, int dim, long x_stride, long y_stride, const float *cos_sin, nm_stream stream)
{
    if (!x || !y || !cos_sin || n_vec < 1 || dim < 2 || (dim & 1) || x_stride < dim || y_stride < dim) return NM_ERR_INVALID_ARG;
    rope_kernel<<<ceil_div(n_vec * (dim / 2), 256), 256, 0, (cudaStream_t)stream>>>((const uint16_t *)x, (uint16_t *)y, n_vec, dim,
                                                                                 x_stride, y_stride, cos_sin);
    NM_LAUNCH_CHECK("rope launch");
    return NM_OK;
}

int nm_rope_table(float *table, long pos_begin, int n_pos, int dim, double base, nm_stream stream)
{
    if (!table || n_pos < 1 || dim < 2 || (dim & 1) || pos_begin < 0 || !(base > 0)) return NM_ERR_INVALID_ARG;
    const long total = (long)n_pos * (dim / 2);
    rope_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(table, pos_begin, n_pos, dim, base);
    NM_LAUNCH_CHECK("rope table launch");
    return NM_OK;
}

size_t nm_mla_attention_workspace_bytes(int H, int n_rows, int kv_lora)
{
    (void)n_rows;
    if (H < 1 || kv_lora < 1) return 0;
    return attention_ws_bytes(H, kv_lora);
}

int nm_mla_attention_partial(const void *Q, const void *kv_cache, int H, int n_rows, int kv_lora, int rope, float scale,
                             void *workspace, size_t workspace_bytes, nm_stream stream)
{
    refresh_step_tuning();
    return attention_partial(Q, kv_cache, H, n_rows, kv_lora, rope, scale, workspace, workspace_bytes, (cudaStream_t)stream);
}

int nm_mla_attention_combine(const void *Q, const void *kv_cache, void *o_bf16, float *o_f32, int H, int n_rows, long extra_row,
                             int kv_lora, int rope, float scale, void *workspace, size_t workspace_bytes, nm_stream stream)
{
    refresh_step_tuning();
    return attention_combine(Q, kv_cache, o_bf16, o_f32, H, n_rows, extra_row, kv_lora, rope, scale, workspace, workspace_bytes,
                             (cudaStream_t)stream);
}

int nm_mla_attention(const void *Q, const void *kv_cache, void *o_bf16, float *o_f32, int H, int n_rows, long extra_row,
                     int kv_lora, int rope, float scale, void *workspace, size_t workspace_bytes, nm_stream stream)
{
    refresh_step_tuning();
    NM_TRY(attention_partial(Q, kv_cache, H, n_rows, kv_lora, rope, scale, workspace, workspace_bytes, (cudaStream_t)stream));
    return attention_combine(Q, kv_cache, o_bf16, o_f32, H, n_rows, extra_row, kv_lora, rope, scale, workspace, workspace_bytes,
                             (cudaStream_t)stream);
}

size_t nm_mla_workspace_bytes(const nm_mla_params *p)
{
    if (!p || p->H < 1 || p->d < 1 || p->q_lora < 1) return 0;
    return step_layout(p).total;
}

size_t nm_mla_batch_workspace_bytes(const nm_mla_params *p, int T)
{
    if (!p || T < 1 || T > kMaxBatch) return 0;
    const size_t batch = batch_layout(p, T).total;
    if (T == 1) {                                                  // a batch of one runs the single-token step
        const size_t single = step_layout(p).total;
        return single > batch ? single : batch;
    }
    return batch;
}

int nm_mla_decode_batch(const nm_mla_params *p, const nm_mla_batch *b, nm_stream main_stream)
{
    // One sequence: the single-token step (its completion stages, prefetch and chaining are tuned for exactly that);
    // the batch fields map onto its parameters one to one.
    if (p && b && b->T == 1 && b->seq_lens && b->seq_lens[0] >= 1 && b->h && b->rope_cos_sin && b->kv_cache && p->workspace &&
        p->workspace_bytes >= step_layout(p).total) {
        nm_mla_params q = *p;
        q.seq_len = b->seq_lens[0];
        q.h = b->h; q.rope_cos_sin = b->rope_cos_sin; q.kv_cache = b->kv_cache; q.out = b->out;
        q.q_full = b->q_full; q.o_lat = b->o_lat; q.o = b->o;
        q.c_q = b->c_q; q.c_qn = b->c_qn; q.q = b->q; q.ckr = b->ckr; q.o_lat_f32 = nullptr;
        q.event_before_wo = nullptr; q.event_after_wo = nullptr; q.programmatic_entry = 0;
        if (!q.W_O) q.out = nullptr;
        return step_impl(&q, (cudaStream_t)main_stream, (cudaStream_t)main_stream);
    }
    return batch_impl(p, b, (cudaStream_t)main_stream);
}

int nm_mla_decode_step(const nm_mla_params *p, nm_stream main_stream, nm_stream side_stream)
{
    return step_impl(p, (cudaStream_t)main_stream, (cudaStream_t)side_stream);
}

int nm_mla_decode_step_host(const nm_mla_params *p, const void *h_host, void *out_host, void *h_staging, void *out_staging,
                            nm_stream main_stream, nm_stream side_stream)
{
    refresh_step_tuning();
    if (!p || !h_host || !out_host || !h_staging || !out_staging || !p->W_O) return NM_ERR_INVALID_ARG;
    nm_mla_params q = *p;
    q.h = h_staging;
    q.out = out_staging;
    // Pinned (or registered) host memory that the device can address: the W_O product stores its 14 KB result straight
    // into it - still a device-to-host transfer, but without a copy operation (and its scheduling gap) after the
    // last kernel.  The token row keeps its copy: 132 CTAs reading it over the host link would cost more.
    void *out_direct = nullptr;
    if (g_s.host_direct_out) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, out_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer &&
            ((uintptr_t)attr.devicePointer & 15u) == 0)
            out_direct = attr.devicePointer;
        else
            (void)cudaGetLastError();
    }
    if (out_direct) q.out = out_direct;
    NM_TRY(check_params(&q));
    cudaStream_t ms = (cudaStream_t)main_stream;
    // The token: when the device can address the host buffer, ONE small CTA fetches the 14 KB over the host link into the staging
    // row, and the step's first product is launched programmatically behind it - its CTAs become resident and fill their rings
    // with weights while the token is on its way (a copy operation in front of the product would be a full dependency).
    const void *h_direct = nullptr;
    if (g_s.host_direct_out && g_s.step_pdl && (p->d % 8) == 0 && ((uintptr_t)h_staging & 15u) == 0) {
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, h_host) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer &&
            ((uintptr_t)attr.devicePointer & 15u) == 0)
            h_direct = attr.devicePointer;
        else
            (void)cudaGetLastError();
    }
    if (h_direct) {
        token_fetch_kernel<<<1, 256, 0, ms>>>(static_cast<const uint4 *>(h_direct), static_cast<uint4 *>(h_staging), p->d / 8);
        NM_LAUNCH_CHECK("token fetch");
        q.programmatic_entry = 1;                                  // behind our own kernel, which writes nothing the prologue reads
    } else {
        NM_CUDA_TRY(cudaMemcpyAsync(h_staging, h_host, (size_t)p->d * 2, cudaMemcpyHostToDevice, ms));
    }
    NM_TRY(step_impl(&q, ms, (cudaStream_t)side_stream));
    if (!out_direct) NM_CUDA_TRY(cudaMemcpyAsync(out_host, out_staging, (size_t)p->d * 2, cudaMemcpyDeviceToHost, ms));
    return NM_OK;
}

int nm_debug_set_batch_per_head_min_tokens(int tokens)
{
    if (tokens < 1 || tokens > kMaxBatch + 1) return NM_ERR_INVALID_ARG;
    return set_step_tuning([&](StepTuning &t) { t.batch_tc_min_t = tokens; });
}

int nm_debug_set_step_plan(int which, int tile_n, int nsplit, int stages)
{
    if (which < 0 || which > 2) return NM_ERR_INVALID_ARG;
    return set_step_tuning([&](StepTuning &t) { t.step_plan[which][0] = tile_n; t.step_plan[which][1] = nsplit; t.step_plan[which][2] = stages; });
}

/* 1 (default): RMSNorm / RoPE / cache-row write run inside the completion of the down-projection products; 0: as
 * kernels of their own. */
int nm_debug_set_step_tails(int enable)
{
    return set_step_tuning([&](StepTuning &t) { t.fused_tails = enable < 0 ? 0 : (enable > 2 ? 2 : enable); });
}

int nm_debug_set_step_knobs(int uv_pdl, int prefetch_uv)
{
    return set_step_tuning([&](StepTuning &t) { t.uv_pdl = uv_pdl ? 1 : 0; t.prefetch_uv = prefetch_uv ? 1 : 0; });
}

/* 1 (default): RoPE + W_UK and merge + W_UV run as fused per-head kernels; 0: separate kernels. */
int nm_debug_set_step_fusion(int enable)
{
    return set_step_tuning([&](StepTuning &t) { t.fused_heads = enable ? 1 : 0; });
}

/* Device buffer of 12 uint64 that receives phase timestamps of the attention kernel (NULL = off). */
int nm_debug_set_attention_trace(void *device_buffer)
{
    set_attention_trace(static_cast<unsigned long long *>(device_buffer));
    return NM_OK;
}

/* MB of W_O the decode step prefetches into L2 beside the attention pass (0 turns the prefetch off). */
int nm_debug_set_step_prefetch(int megabytes)
{
    if (megabytes < 0 || megabytes > 100) return NM_ERR_INVALID_ARG;
    return set_step_tuning([&](StepTuning &t) { t.prefetch_mb = megabytes; });
}

/* Chain the kernels of the decode step with programmatic dependent launch (default on). */
int nm_debug_set_step_pdl(int enable)
{
    return set_step_tuning([&](StepTuning &t) { t.step_pdl = enable ? 1 : 0; });
}

/* Two-stream schedule of the decode step (separate W_DQ and W_DKV|W_KR, a side stream): 0 (default) the KV chain is forked at
 * the start of the step, beside the first product of the Q chain; 1 it is forked when the attention operand is ready and runs
 * beside the tensor-core pass. */
int nm_debug_set_step_kv_beside_attention(int enable)
{
    return set_step_tuning([&](StepTuning &t) { t.kv_beside_attention = enable ? 1 : 0; });
}

int nm_debug_set_attention_wide(int tile_rows, int max_runs, int cluster)
{
    if (tile_rows < 0 || max_runs < 0 || max_runs > 64 || cluster < 0 || cluster > 4) return NM_ERR_INVALID_ARG;
    return set_step_tuning([&](StepTuning &t) { t.wide_tile = tile_rows; t.wide_splits = max_runs; t.wide_cluster = cluster; });
}

/* 0: tensor-core attention when the shape allows (default); 1: CUDA-core attention kernel; 2 / 3: the older tensor-core
 * kernels with 128 / 64 heads per CTA whatever the length; 4: the wide-tile kernel. */
int nm_debug_set_attention(int impl)
{
    return set_step_tuning([&](StepTuning &t) { t.attn_impl = impl; });
}

#pragma GCC visibility pop
}
