// Per-head stages of the single-token decode step, one CTA per head, each fused with the small vector
// stage that feeds it (the paper's point that RMSNorm / RoPE-like consumers should start right where
// the narrow product ends, MLA Operator Optimization section):
//
//   q_finish_kernel   q_rope[h] = RoPE(q[h, nope:]),  q_lat[h] = q[h, :nope] * W_UK[h]      (128 -> 512)
//   uv_merge_kernel   o_lat[h]  = merge of the attention partials (+ the new cache row),
//                     o[h]      = bf16(o_lat[h]) * W_UV[h]                                   (512 -> 128)
//
// Both stream the head's 128 KB of weights with 32 independent 16-byte read-only loads per thread,
// the first batches issued before the programmatic-launch wait (weights do not depend on earlier
// kernels), accumulate in fp32, reduce the row groups through shared memory and round once to bf16.
#include "nm_async.cuh"
#include "nm_mla.cuh"

namespace nm {

namespace {

constexpr int kHeadThreads = 256;

__device__ __forceinline__ float bf16_to_f32(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t f32_to_bf16(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }

__device__ __forceinline__ float block_sum_256(float v, float *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kHeadThreads / 32; ++w) t += scratch[w];
    return t;
}

// y[0..N) = x[0..K) * W[K][N] (row-major bf16), x in shared memory as fp32.  256 threads: N/8 column
// groups x (2048/N) row groups, 32 rows per thread.  `w` holds this thread's 32 weight vectors, loaded
// by the caller (so that the loads can be issued before the inputs exist).
template <int K, int N>
struct HeadMatvec {
    static constexpr int kColGroups = N / 8;
    static constexpr int kRowGroups = kHeadThreads / kColGroups;
    static constexpr int kRowsPerThread = K / kRowGroups;
    static_assert(kRowsPerThread == 32, "shapes of the absorbed MLA products: 128x512 and 512x128");

    __device__ static __forceinline__ void load(const uint16_t *__restrict__ W, uint4 (&w)[32], int first, int count)
    {
        const int tx = threadIdx.x % kColGroups, ty = threadIdx.x / kColGroups;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i >= first && i < first + count) w[i] = ld_stream16(W + (size_t)(ty + i * kRowGroups) * N + tx * 8);
    }

    // returns in `out8` the 8 column sums of this thread's column group when ty == 0 (others: unspecified)
    __device__ static __forceinline__ void run(const uint4 (&w)[32], const float *x_s, float *red /* kRowGroups*N floats */, float (&out8)[8])
    {
        const int tx = threadIdx.x % kColGroups, ty = threadIdx.x / kColGroups;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            float b[8];
            Elem<bf16_t>::unpack(w[i], b);
            const float a = x_s[ty + i * kRowGroups];
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = fmaf(a, b[j], acc[j]);
        }
        float4 *dst = reinterpret_cast<float4 *>(red + (size_t)ty * N + tx * 8);
        dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
        __syncthreads();
        if (ty == 0) {
#pragma unroll
            for (int j = 0; j < 8; ++j) out8[j] = 0.f;
            for (int g = 0; g < kRowGroups; ++g) {                 // fixed order: deterministic
                const float4 *src = reinterpret_cast<const float4 *>(red + (size_t)g * N + tx * 8);
                const float4 v0 = src[0], v1 = src[1];
                out8[0] += v0.x; out8[1] += v0.y; out8[2] += v0.z; out8[3] += v0.w;
                out8[4] += v1.x; out8[5] += v1.y; out8[6] += v1.z; out8[7] += v1.w;
            }
        }
    }
};

__device__ __forceinline__ uint4 pack8_bf16(const float (&v)[8])
{
    return make_uint4((uint32_t)f32_to_bf16(v[0]) | ((uint32_t)f32_to_bf16(v[1]) << 16),
                      (uint32_t)f32_to_bf16(v[2]) | ((uint32_t)f32_to_bf16(v[3]) << 16),
                      (uint32_t)f32_to_bf16(v[4]) | ((uint32_t)f32_to_bf16(v[5]) << 16),
                      (uint32_t)f32_to_bf16(v[6]) | ((uint32_t)f32_to_bf16(v[7]) << 16));
}

// q: [H][nope+rope] bf16; W_UK: [H][nope][dc]; q_full: [H][dc+rope] (q_lat | q_rope).  nope = 128, dc = 512.
__global__ void __launch_bounds__(kHeadThreads) q_finish_kernel(const uint16_t *__restrict__ q, const uint16_t *__restrict__ W_UK,
                                                                const float *__restrict__ cs, uint16_t *__restrict__ q_full, int rope,
                                                                const KvFinish kv)
{
    constexpr int K = 128, N = 512;
    using MV = HeadMatvec<K, N>;
    __shared__ __align__(16) float x_s[K];
    __shared__ __align__(16) float red[MV::kRowGroups * N];
    if (kv.enabled && blockIdx.x == gridDim.x - 1) {
        // the extra CTA: RMSNorm of the KV latent, RoPE of the key part, both into the new cache row (dc <= 512)
        pdl_launch_dependents();
        pdl_wait_prior_grids();
        const int i0 = 2 * threadIdx.x;
        float x0 = 0.f, x1 = 0.f, g0 = 0.f, g1 = 0.f, r0 = 0.f, r1 = 0.f, c = 0.f, sn = 0.f;
        if (i0 < kv.dc) {
            const uint32_t xv = *reinterpret_cast<const uint32_t *>(kv.ckr + i0), gv = *reinterpret_cast<const uint32_t *>(kv.gamma + i0);
            x0 = __uint_as_float(xv << 16); x1 = __uint_as_float(xv & 0xffff0000u);
            g0 = __uint_as_float(gv << 16); g1 = __uint_as_float(gv & 0xffff0000u);
        }
        if (i0 < kv.rope) {
            const uint32_t rv = *reinterpret_cast<const uint32_t *>(kv.ckr + kv.dc + i0);
            r0 = __uint_as_float(rv << 16); r1 = __uint_as_float(rv & 0xffff0000u);
            c = kv.cos_sin[i0]; sn = kv.cos_sin[i0 + 1];
        }
        const float ss = block_sum_256(fmaf(x0, x0, x1 * x1), red);
        const float r = 1.0f / sqrtf(ss / (float)kv.dc + kv.eps);
        if (i0 < kv.dc)
            *reinterpret_cast<uint32_t *>(kv.cache_row + i0) = (uint32_t)f32_to_bf16(x0 * r * g0) | ((uint32_t)f32_to_bf16(x1 * r * g1) << 16);
        if (i0 < kv.rope)
            *reinterpret_cast<uint32_t *>(kv.cache_row + kv.dc + i0) =
                (uint32_t)f32_to_bf16(r0 * c - r1 * sn) | ((uint32_t)f32_to_bf16(r0 * sn + r1 * c) << 16);
        return;
    }
    const int h = blockIdx.x;
    const uint16_t *W = W_UK + (size_t)h * K * N;
    uint4 w[32];
    MV::load(W, w, 0, 32);                                        // weights first: they depend on nothing
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // q comes from the W_UQR product
    const uint16_t *qh = q + (size_t)h * (K + rope);
    if (threadIdx.x < K) x_s[threadIdx.x] = bf16_to_f32(qh[threadIdx.x]);
    if (threadIdx.x < rope / 2) {                                 // interleaved pairs, rounded to bf16
        const int i = threadIdx.x;
        const float c = cs[2 * i], s = cs[2 * i + 1];
        const float x0 = bf16_to_f32(qh[K + 2 * i]), x1 = bf16_to_f32(qh[K + 2 * i + 1]);
        uint16_t *dst = q_full + (size_t)h * (N + rope) + N + 2 * i;
        *reinterpret_cast<uint32_t *>(dst) = (uint32_t)f32_to_bf16(x0 * c - x1 * s) | ((uint32_t)f32_to_bf16(x0 * s + x1 * c) << 16);
    }
    __syncthreads();
    float out8[8];
    MV::run(w, x_s, red, out8);
    if (threadIdx.x / MV::kColGroups == 0)
        *reinterpret_cast<uint4 *>(q_full + (size_t)h * (N + rope) + (threadIdx.x % MV::kColGroups) * 8) = pack8_bf16(out8);
}

// Merge of the attention partials (see attn_combine_kernel for the algebra) followed by W_UV.
// dc = 512, dv = 128.
//
// Sized to share an SM with a CTA of the attention kernel that precedes it (which holds nearly all of the
// shared memory and under half of the registers; the register file is split over the four schedulers, two
// warps of each kernel per scheduler, so the two kernels' registers per thread must add up to 256 or less): under 8 KB of shared memory, at most 128 registers per
// thread.  Launched programmatically, it is therefore resident - with half of the head's 128 KB
// of weights already in registers - when the attention result arrives; the rest (an L2 hit after its own
// prefetch) is fetched once the partial rows have left their registers.
// kUvPre weight vectors per thread are loaded before the inputs exist; the partial rows are requested kBatch at a time
// (one L2 round trip per batch): 16 and 16 for up to 16 partials, 8 and 32 beyond (the registers are the same).
constexpr int kUvMaxParts = 64;                                    // partials per head the merge takes (the planner never makes more)
template <int kUvPre, int kBatch>
__global__ void __launch_bounds__(kHeadThreads, 2) uv_merge_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                                   AttnPartials part, int npart, long extra_row, int rope, float scale,
                                                                   const uint16_t *__restrict__ W_UV, uint16_t *__restrict__ o_lat_bf16,
                                                                   float *__restrict__ o_lat_f32, uint16_t *__restrict__ o, const L2Prefetch pf,
                                                                   unsigned long long *trace)
{
#define UV_TRACE(i) do { if (trace && tid == 0 && (blockIdx.x == 0 || blockIdx.x == 77)) trace[1100 + (blockIdx.x ? 16 : 0) + (i)] = global_timer_ns(); } while (0)
    constexpr int K = 512, N = 128;
    constexpr int kColGroups = N / 8, kRowGroups = kHeadThreads / kColGroups;        // 16 x 16; 32 rows per thread
    __shared__ __align__(16) float x_s[K];
    __shared__ __align__(16) float red[(kRowGroups / 2) * N];      // row groups 2j and 2j+1 sit in one warp: added by shuffle
    __shared__ float scratch[32];
    __shared__ float sm[kUvMaxParts], sl[kUvMaxParts], sw[kUvMaxParts];
    const int h = blockIdx.x, H = gridDim.x, dkv = K + rope, tid = threadIdx.x;
    const int tx = tid % kColGroups, ty = tid / kColGroups;
    const uint16_t *W = W_UV + (size_t)h * K * N + (size_t)ty * N + tx * 8;          // row ty + i*kRowGroups for i = 0..31
    UV_TRACE(0);
    uint4 w[kUvPre];
#pragma unroll
    for (int i = 0; i < kUvPre; ++i) w[i] = ld_stream16(W + (size_t)i * kRowGroups * N);
    pdl_launch_dependents();
    // While the attention kernel (which needs little HBM bandwidth) runs, this grid is resident and idle:
    // it pulls into L2 the rest of its own weights and the ranges of the next product's weights it was
    // given (the head of every k-split of W_O) - they do not depend on the attention result.  The request
    // stalls its thread while the queue is full; nothing here is waiting for these threads yet.
    if (pf.nranges >= 0) {
        constexpr long kChunk = 4096;
        if (tid < (K - kUvPre * kRowGroups) * N * 2 / kChunk)       // rows kUvPre*16.. of this head: contiguous
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"((const char *)(W_UV + (size_t)h * K * N + (size_t)kUvPre * kRowGroups * N) + tid * kChunk),
                         "r"((uint32_t)kChunk) : "memory");
        const long chunks_per_range = (pf.range_bytes + kChunk - 1) / kChunk, total = chunks_per_range * pf.nranges;
        for (long i = (long)h * kHeadThreads + tid; i < total; i += (long)H * kHeadThreads) {
            const long r = i / chunks_per_range, off = (i - r * chunks_per_range) * kChunk;
            const long n = min(kChunk, pf.range_bytes - off) & ~15L;
            if (n > 0) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(pf.base + r * pf.range_stride + off), "r"((uint32_t)n) : "memory");
        }
    }
    UV_TRACE(1);
    pdl_wait_prior_grids();                                       // partials come from the attention kernel
    UV_TRACE(2);
    // Everything the merge needs is asked for at once, so that one L2 round trip covers it: the partial rows
    // of up to 16 parts (two columns per thread), the (m, l) pairs, and the operands of the new row's score.
    const int c = 2 * tid;
    const float *src = part.O + (size_t)h * K + c;
    float2 v[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
        v[u] = (u < npart) ? __ldcg(reinterpret_cast<const float2 *>(src + (size_t)u * H * K)) : make_float2(0.f, 0.f);
    for (int s = tid; s < npart; s += kHeadThreads) {
        const float2 ml = __ldcg(reinterpret_cast<const float2 *>(part.ml + ((size_t)s * H + h) * 2));
        sm[s] = ml.x; sl[s] = ml.y;
    }
    float sx = -INFINITY;
    if (extra_row >= 0) {
        float dot = 0.f;
        if (tid < dkv / 8) {                                       // dkv = 576: 72 threads, eight elements each
            float qf[8], rf[8];
            Elem<bf16_t>::unpack(__ldcg(reinterpret_cast<const uint4 *>(Q + (size_t)h * dkv) + tid), qf);
            Elem<bf16_t>::unpack(__ldcg(reinterpret_cast<const uint4 *>(cache + (size_t)extra_row * dkv) + tid), rf);
#pragma unroll
            for (int e = 0; e < 8; ++e) dot = fmaf(qf[e], rf[e], dot);
        }
        sx = block_sum_256(dot, scratch) * scale;
    } else {
        __syncthreads();
    }
    UV_TRACE(3);
    // weights of the parts: exp(m_s - max), the new row's exp(sx - max), and the normaliser L.  Up to 32 parts
    // (the tensor-core pass makes at most 16) are handled by one warp with shuffles in a fixed order.
    if (npart <= 32) {
        if (tid < 32) {
            const float m = (tid < npart) ? sm[tid] : -INFINITY, l = (tid < npart) ? sl[tid] : 0.f;
            float Mx = fmaxf(m, sx);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) Mx = fmaxf(Mx, __shfl_xor_sync(0xffffffffu, Mx, o));
            const float wgt = (m == -INFINITY) ? 0.f : __expf(m - Mx);
            float L = wgt * l;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
            const float wx = (extra_row >= 0) ? __expf(sx - Mx) : 0.f;
            sw[tid] = wgt;
            if (tid == 0) { scratch[16] = wx; scratch[17] = L + wx; }
        }
    } else if (tid == 0) {
        float Mx = sx;
        for (int s = 0; s < npart; ++s) Mx = fmaxf(Mx, sm[s]);
        const float wx = (extra_row >= 0) ? __expf(sx - Mx) : 0.f;
        float L = wx;
        for (int s = 0; s < npart; ++s) {
            const float wgt = (sm[s] == -INFINITY) ? 0.f : __expf(sm[s] - Mx);
            sw[s] = wgt;
            L = fmaf(wgt, sl[s], L);
        }
        scratch[16] = wx; scratch[17] = L;
    }
    __syncthreads();
    const float wx = scratch[16], L = scratch[17];
    float2 acc = make_float2(0.f, 0.f);
    if (extra_row >= 0) {
        const uint32_t rv = *reinterpret_cast<const uint32_t *>(cache + (size_t)extra_row * dkv + c);
        acc = make_float2(wx * __uint_as_float(rv << 16), wx * __uint_as_float(rv & 0xffff0000u));
    }
    for (int s0 = 0; s0 < npart; s0 += kBatch) {
        if (s0 > 0) {
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                v[u] = (s0 + u < npart) ? __ldcg(reinterpret_cast<const float2 *>(src + (size_t)(s0 + u) * H * K)) : make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const float wgt = (s0 + u < npart) ? sw[s0 + u] : 0.f;
            acc.x = fmaf(wgt, v[u].x, acc.x);
            acc.y = fmaf(wgt, v[u].y, acc.y);
        }
    }
    UV_TRACE(4);
    // the second half of the weights (L2 hits) takes the registers the partial rows have left
    uint4 w2[K / kRowGroups - kUvPre];
#pragma unroll
    for (int i = 0; i < K / kRowGroups - kUvPre; ++i) w2[i] = ld_stream16(W + (size_t)(kUvPre + i) * kRowGroups * N);
    const float inv = 1.0f / L;
    const float o0 = acc.x * inv, o1 = acc.y * inv;
    const uint16_t b0 = f32_to_bf16(o0), b1 = f32_to_bf16(o1);
    if (o_lat_f32) *reinterpret_cast<float2 *>(o_lat_f32 + (size_t)h * K + c) = make_float2(o0, o1);
    if (o_lat_bf16) *reinterpret_cast<uint32_t *>(o_lat_bf16 + (size_t)h * K + c) = (uint32_t)b0 | ((uint32_t)b1 << 16);
    x_s[c] = bf16_to_f32(b0);                                      // W_UV sees the rounded o_lat, as the stage-wise definition says
    x_s[c + 1] = bf16_to_f32(b1);
    __syncthreads();

    UV_TRACE(5);
    // ---- o[h] = o_lat[h] * W_UV[h]: rows ty + i*16 ------------------------------------------------------------
    float a8[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) a8[j] = 0.f;
    auto use = [&](const uint4 &wv, int i) {
        float b[8];
        Elem<bf16_t>::unpack(wv, b);
        const float a = x_s[ty + i * kRowGroups];
#pragma unroll
        for (int j = 0; j < 8; ++j) a8[j] = fmaf(a, b[j], a8[j]);
    };
#pragma unroll
    for (int i = 0; i < kUvPre; ++i) use(w[i], i);
#pragma unroll
    for (int i = 0; i < K / kRowGroups - kUvPre; ++i) use(w2[i], kUvPre + i);
    UV_TRACE(6);
#pragma unroll
    for (int j = 0; j < 8; ++j) a8[j] += __shfl_xor_sync(0xffffffffu, a8[j], 16);     // row groups 2j + 2j+1
    if ((tid & 16) == 0) {
        float4 *dst = reinterpret_cast<float4 *>(red + (size_t)(ty >> 1) * N + tx * 8);
        dst[0] = make_float4(a8[0], a8[1], a8[2], a8[3]);
        dst[1] = make_float4(a8[4], a8[5], a8[6], a8[7]);
    }
    __syncthreads();
    if (ty == 0) {
        float out8[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) out8[j] = 0.f;
        for (int g = 0; g < kRowGroups / 2; ++g) {                 // fixed order: deterministic
            const float4 *src4 = reinterpret_cast<const float4 *>(red + (size_t)g * N + tx * 8);
            const float4 v0 = src4[0], v1 = src4[1];
            out8[0] += v0.x; out8[1] += v0.y; out8[2] += v0.z; out8[3] += v0.w;
            out8[4] += v1.x; out8[5] += v1.y; out8[6] += v1.z; out8[7] += v1.w;
        }
        *reinterpret_cast<uint4 *>(o + (size_t)h * N + tx * 8) = pack8_bf16(out8);
    }
    UV_TRACE(7);
#undef UV_TRACE
}

// The vector stages behind the fused down-projection h * (W_DQ | W_DKV | W_KR): CTA 0 normalises the
// query latent (c_qn = RMSNorm(c_q; gamma_q)), CTA 1 finishes the cache row (RMSNorm of the KV latent,
// RoPE of the key part).  x: [q_lora + dc + rope] bf16 as the product wrote it.
__global__ void __launch_bounds__(kHeadThreads) down_finish_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ gamma_q,
                                                                   const uint16_t *__restrict__ gamma_kv, const float *__restrict__ cs,
                                                                   uint16_t *__restrict__ c_qn, uint16_t *__restrict__ cache_row,
                                                                   int q_lora, int dc, int rope, float eps)
{
    __shared__ float scratch[32];
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    pdl_wait_prior_grids();
    if (blockIdx.x == 0) {
        // up to 8 elements per thread (q_lora <= 2048, multiple of 8 checked by the host)
        const int i0 = 8 * tid;
        float f[8], g[8];
        const bool on = i0 < q_lora;
        if (on) {
            Elem<bf16_t>::unpack(*reinterpret_cast<const uint4 *>(x + i0), f);
            Elem<bf16_t>::unpack(__ldg(reinterpret_cast<const uint4 *>(gamma_q + i0)), g);
        }
        float ss = 0.f;
        if (on)
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
        ss = block_sum_256(ss, scratch);
        const float r = 1.0f / sqrtf(ss / (float)q_lora + eps);
        if (on) {
            float y[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = f[e] * r * g[e];
            *reinterpret_cast<uint4 *>(c_qn + i0) = pack8_bf16(y);
        }
    } else {
        const uint16_t *ckr = x + q_lora;
        const int i0 = 2 * tid;                                    // dc <= 512
        float x0 = 0.f, x1 = 0.f, g0 = 0.f, g1 = 0.f;
        if (i0 < dc) {
            const uint32_t xv = *reinterpret_cast<const uint32_t *>(ckr + i0), gv = *reinterpret_cast<const uint32_t *>(gamma_kv + i0);
            x0 = __uint_as_float(xv << 16); x1 = __uint_as_float(xv & 0xffff0000u);
            g0 = __uint_as_float(gv << 16); g1 = __uint_as_float(gv & 0xffff0000u);
        }
        float r0v = 0.f, r1v = 0.f, c = 0.f, sn = 0.f;
        if (tid < rope / 2) {
            const uint32_t rv = *reinterpret_cast<const uint32_t *>(ckr + dc + i0);
            r0v = __uint_as_float(rv << 16); r1v = __uint_as_float(rv & 0xffff0000u);
            c = cs[i0]; sn = cs[i0 + 1];
        }
        const float ss = block_sum_256(fmaf(x0, x0, x1 * x1), scratch);
        const float r = 1.0f / sqrtf(ss / (float)dc + eps);
        if (i0 < dc)
            *reinterpret_cast<uint32_t *>(cache_row + i0) = (uint32_t)f32_to_bf16(x0 * r * g0) | ((uint32_t)f32_to_bf16(x1 * r * g1) << 16);
        if (tid < rope / 2)
            *reinterpret_cast<uint32_t *>(cache_row + dc + i0) =
                (uint32_t)f32_to_bf16(r0v * c - r1v * sn) | ((uint32_t)f32_to_bf16(r0v * sn + r1v * c) << 16);
    }
}

template <typename... Args>
cudaError_t launch_with_pdl(void (*kern)(Args...), int grid, cudaStream_t s, bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kHeadThreads); cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace

bool head_kernels_apply(int H, int nope, int rope, int dc, int dv)
{
    return H >= 1 && nope == 128 && dc == 512 && dv == 128 && rope >= 2 && rope <= 2 * kHeadThreads && (rope & 1) == 0;
}

bool down_finish_applies(int q_lora, int dc, int rope)
{
    return q_lora % 8 == 0 && q_lora <= 8 * kHeadThreads && dc % 2 == 0 && dc <= 2 * kHeadThreads && rope % 2 == 0 && rope <= dc;
}

int launch_down_finish(const void *x, const void *gamma_q, const void *gamma_kv, const float *cos_sin, void *c_qn, void *cache_row,
                       int q_lora, int dc, int rope, float eps, cudaStream_t s, bool pdl)
{
    cudaError_t e = launch_with_pdl(down_finish_kernel, 2, s, pdl, (const uint16_t *)x, (const uint16_t *)gamma_q, (const uint16_t *)gamma_kv,
                                    cos_sin, (uint16_t *)c_qn, (uint16_t *)cache_row, q_lora, dc, rope, eps);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "down_finish launch");
}

int launch_q_finish(const void *q, const void *W_UK, const float *cos_sin, void *q_full, int H, int rope, cudaStream_t s, bool pdl, KvFinish kv)
{
    if (kv.enabled && (kv.dc > 2 * kHeadThreads || kv.rope > kv.dc || (kv.dc | kv.rope) % 2)) return NM_ERR_UNSUPPORTED;
    cudaError_t e = launch_with_pdl(q_finish_kernel, H + (kv.enabled ? 1 : 0), s, pdl, (const uint16_t *)q, (const uint16_t *)W_UK, cos_sin,
                                    (uint16_t *)q_full, rope, kv);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "q_finish launch");
}

int launch_uv_merge(const void *Q, const void *cache, AttnPartials part, int npart, long extra_row, int rope, float scale,
                    const void *W_UV, void *o_lat_bf16, float *o_lat_f32, void *o, int H, cudaStream_t s, bool pdl, L2Prefetch prefetch)
{
    if (npart < 0 || npart > kUvMaxParts) return NM_ERR_UNSUPPORTED;
    if (!prefetch.base && !prefetch.block) prefetch.nranges = -1;  // no prefetch at all
    cudaError_t e = launch_with_pdl(npart > 16 ? uv_merge_kernel<8, 32> : uv_merge_kernel<16, 16>, H, s, pdl, (const uint16_t *)Q,
                                    (const uint16_t *)cache, part, npart, extra_row, rope, scale, (const uint16_t *)W_UV, (uint16_t *)o_lat_bf16,
                                    o_lat_f32, (uint16_t *)o, prefetch, attention_trace());
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "uv_merge launch");
}

}  // namespace nm
