// Vector and per-head stages of the small-batch decode step: T independent sequences, one new token each
// (the paper's "larger token" direction, Condition 5: the narrow products take M = T rows and stream the
// weights once for all of them).  Same arithmetic as the single-token kernels of nm_head_kernels.cu and
// nm_mla.cu; every CTA keeps its head's weights in registers and walks over the tokens.
#include "nm_async.cuh"
#include "nm_mla.cuh"

namespace nm {

namespace {

constexpr int kThreadsB = 256;

__device__ __forceinline__ float bf2f(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t f2bf(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ uint32_t pack2(float lo, float hi) { return (uint32_t)f2bf(lo) | ((uint32_t)f2bf(hi) << 16); }

__device__ __forceinline__ float block_sum(float v, float *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kThreadsB / 32; ++w) t += scratch[w];
    return t;
}

// RMSNorm of the query latent (CTA x = 0) and RMSNorm + RoPE + cache-row write of the KV part (CTA x = 1) of
// token blockIdx.y.  x: [T][q_lora + dc + rope] as the down-projection wrote it.
__global__ void __launch_bounds__(kThreadsB) down_finish_batch_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ gamma_q,
                                                                      const uint16_t *__restrict__ gamma_kv, const float *__restrict__ cs,
                                                                      uint16_t *__restrict__ c_qn, uint16_t *__restrict__ cache,
                                                                      const BatchRows rows, int q_lora, int dc, int rope, float eps)
{
    __shared__ float scratch[32];
    const int tid = threadIdx.x, t = blockIdx.y;
    pdl_launch_dependents();
    pdl_wait_prior_grids();
    const uint16_t *xt = x + (size_t)t * (q_lora + dc + rope);
    if (blockIdx.x == 0) {
        const int i0 = 8 * tid;
        float f[8], g[8];
        const bool on = i0 < q_lora;
        if (on) {
            Elem<bf16_t>::unpack(*reinterpret_cast<const uint4 *>(xt + i0), f);
            Elem<bf16_t>::unpack(__ldg(reinterpret_cast<const uint4 *>(gamma_q + i0)), g);
        }
        float ss = 0.f;
        if (on)
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
        ss = block_sum(ss, scratch);
        const float r = 1.0f / sqrtf(ss / (float)q_lora + eps);
        if (on) {
            uint4 o;
            o.x = pack2(f[0] * r * g[0], f[1] * r * g[1]); o.y = pack2(f[2] * r * g[2], f[3] * r * g[3]);
            o.z = pack2(f[4] * r * g[4], f[5] * r * g[5]); o.w = pack2(f[6] * r * g[6], f[7] * r * g[7]);
            *reinterpret_cast<uint4 *>(c_qn + (size_t)t * q_lora + i0) = o;
        }
    } else {
        const uint16_t *ckr = xt + q_lora;
        uint16_t *row = cache + rows.new_row[t];
        const float *cst = cs + (size_t)t * rope;
        const int i0 = 2 * tid;
        float x0 = 0.f, x1 = 0.f, g0 = 0.f, g1 = 0.f;
        if (i0 < dc) {
            const uint32_t xv = *reinterpret_cast<const uint32_t *>(ckr + i0), gv = *reinterpret_cast<const uint32_t *>(gamma_kv + i0);
            x0 = __uint_as_float(xv << 16); x1 = __uint_as_float(xv & 0xffff0000u);
            g0 = __uint_as_float(gv << 16); g1 = __uint_as_float(gv & 0xffff0000u);
        }
        float r0 = 0.f, r1 = 0.f, c = 0.f, sn = 0.f;
        if (i0 < rope) {
            const uint32_t rv = *reinterpret_cast<const uint32_t *>(ckr + dc + i0);
            r0 = __uint_as_float(rv << 16); r1 = __uint_as_float(rv & 0xffff0000u);
            c = cst[i0]; sn = cst[i0 + 1];
        }
        const float ss = block_sum(fmaf(x0, x0, x1 * x1), scratch);
        const float r = 1.0f / sqrtf(ss / (float)dc + eps);
        if (i0 < dc) *reinterpret_cast<uint32_t *>(row + i0) = pack2(x0 * r * g0, x1 * r * g1);
        if (i0 < rope) *reinterpret_cast<uint32_t *>(row + dc + i0) = pack2(r0 * c - r1 * sn, r0 * sn + r1 * c);
    }
}

constexpr int kTokGroup = 4;              // tokens whose products share one pass over the weights in registers

// For head blockIdx.x and every token t: q_rope = RoPE(q[t, h, nope:]), q_lat = q[t, h, :nope] * W_UK[h].
// q: [T][H][nope + rope]; q_full: [T][H][dc + rope] (q_lat | q_rope).  nope = 128, dc = 512.
// All tokens' inputs are fetched at once; the product runs over groups of four tokens, each thread keeping four
// accumulator sets for its 32 weight rows, so that the weights in registers are walked once per group and the
// cross-row-group sums cost two barriers per group instead of per token.
__global__ void __launch_bounds__(kThreadsB) q_finish_batch_kernel(const uint16_t *__restrict__ q, const uint16_t *__restrict__ W_UK,
                                                                   const float *__restrict__ cs, uint16_t *__restrict__ q_full, int rope, int T)
{
    constexpr int K = 128, N = 512, kColGroups = N / 8, kRowGroups = kThreadsB / kColGroups;      // 64 x 4
    __shared__ __align__(16) float x_s[kMaxBatch][K];
    __shared__ __align__(16) float red[kTokGroup][kRowGroups][N];
    const int h = blockIdx.x, H = gridDim.x, tid = threadIdx.x;
    const int tx = tid % kColGroups, ty = tid / kColGroups;
    const uint16_t *W = W_UK + (size_t)h * K * N + (size_t)ty * N + tx * 8;
    uint4 w[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = ld_stream16(W + (size_t)i * kRowGroups * N);
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // q comes from the W_UQR product
    for (int i = tid; i < T * K; i += kThreadsB) {
        const int t = i / K, k = i - t * K;
        x_s[t][k] = bf2f(q[((size_t)t * H + h) * (K + rope) + k]);
    }
    for (int i = tid; i < T * (rope / 2); i += kThreadsB) {       // interleaved pairs, rounded to bf16
        const int t = i / (rope / 2), pr = i - t * (rope / 2);
        const uint16_t *qh = q + ((size_t)t * H + h) * (K + rope) + K;
        const float c = cs[(size_t)t * rope + 2 * pr], sn = cs[(size_t)t * rope + 2 * pr + 1];
        const float x0 = bf2f(qh[2 * pr]), x1 = bf2f(qh[2 * pr + 1]);
        *reinterpret_cast<uint32_t *>(q_full + ((size_t)t * H + h) * (N + rope) + N + 2 * pr) = pack2(x0 * c - x1 * sn, x0 * sn + x1 * c);
    }
    __syncthreads();
    for (int t0 = 0; t0 < T; t0 += kTokGroup) {
        float acc[kTokGroup][8];
#pragma unroll
        for (int g = 0; g < kTokGroup; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[g][j] = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            float b[8];
            uint4 wi = w[i];
            // keeps the widening of the weights inside the group loop: hoisted out of it, the 256 widened values
            // of a thread would not fit its registers
            asm volatile("" : "+r"(wi.x), "+r"(wi.y), "+r"(wi.z), "+r"(wi.w));
            Elem<bf16_t>::unpack(wi, b);
#pragma unroll
            for (int g = 0; g < kTokGroup; ++g) {
                const float a = x_s[min(t0 + g, kMaxBatch - 1)][ty + i * kRowGroups];
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[g][j] = fmaf(a, b[j], acc[g][j]);
            }
        }
#pragma unroll
        for (int g = 0; g < kTokGroup; ++g) {
            float4 *dst = reinterpret_cast<float4 *>(&red[g][ty][tx * 8]);
            dst[0] = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
            dst[1] = make_float4(acc[g][4], acc[g][5], acc[g][6], acc[g][7]);
        }
        __syncthreads();
        // thread (ty, tx) finishes token t0 + ty: eight columns, row groups added in a fixed order
        if (t0 + ty < T) {
            float out8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) out8[j] = 0.f;
#pragma unroll
            for (int g = 0; g < kRowGroups; ++g) {
                const float4 *src = reinterpret_cast<const float4 *>(&red[ty][g][tx * 8]);
                const float4 v0 = src[0], v1 = src[1];
                out8[0] += v0.x; out8[1] += v0.y; out8[2] += v0.z; out8[3] += v0.w;
                out8[4] += v1.x; out8[5] += v1.y; out8[6] += v1.z; out8[7] += v1.w;
            }
            uint4 o;
            o.x = pack2(out8[0], out8[1]); o.y = pack2(out8[2], out8[3]); o.z = pack2(out8[4], out8[5]); o.w = pack2(out8[6], out8[7]);
            *reinterpret_cast<uint4 *>(q_full + ((size_t)(t0 + ty) * H + h) * (N + rope) + tx * 8) = o;
        }
        __syncthreads();                                           // red is reused by the next group
    }
}

// For head blockIdx.x and every token t: log-sum-exp merge of the attention partials of sequence t and of the
// row the step just wrote, o_lat rounded to bf16, then o[t, h] = o_lat[t, h] * W_UV[h].  dc = 512, dv = 128.
// Phases over all tokens at once (scores of the new rows by warps, weights by one thread per token, merge with
// all partial rows of eight tokens in flight), then the product over groups of four tokens as above.
__global__ void __launch_bounds__(kThreadsB) uv_merge_batch_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                                   AttnPartials part, const BatchRows rows, int rope, float scale,
                                                                   const uint16_t *__restrict__ W_UV, uint16_t *__restrict__ o_lat_bf16,
                                                                   uint16_t *__restrict__ o, int T)
{
    constexpr int K = 512, N = 128, kColGroups = N / 8, kRowGroups = kThreadsB / kColGroups;      // 16 x 16
    constexpr int kMaxParts = 16;                                 // 64 splits in clusters of four
    __shared__ __align__(16) uint16_t x_s[kMaxBatch][K];          // merged o_lat, already rounded to bf16
    __shared__ __align__(16) float red[kTokGroup][kRowGroups / 2][N];
    __shared__ float sm[kMaxBatch][kMaxParts], sl[kMaxBatch][kMaxParts], sw[kMaxBatch][kMaxParts];
    __shared__ float sx[kMaxBatch], swx[kMaxBatch], sinv[kMaxBatch];
    const int h = blockIdx.x, H = gridDim.x, dkv = K + rope, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tx = tid % kColGroups, ty = tid / kColGroups;
    const uint16_t *W = W_UV + (size_t)h * K * N + (size_t)ty * N + tx * 8;
    uint4 w[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = ld_stream16(W + (size_t)i * kRowGroups * N);
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // partials come from the attention kernel
    // (m, l) of every (token, part)
    for (int i = tid; i < T * kMaxParts; i += kThreadsB) {
        const int t = i / kMaxParts, s = i - t * kMaxParts;
        if (s < rows.npart[t]) {
            const float2 p = __ldcg(reinterpret_cast<const float2 *>(part.ml + (((size_t)t * rows.slot_stride + s) * H + h) * 2));
            sm[t][s] = p.x; sl[t][s] = p.y;
        }
    }
    // score of each token's new row: one warp per token, 576 elements over 32 lanes
    for (int t = warp; t < T; t += kThreadsB / 32) {
        const uint16_t *qh = Q + ((size_t)t * H + h) * dkv, *row = cache + rows.new_row[t];
        float dot = 0.f;
        for (int i = lane * 2; i < dkv; i += 64) {
            const uint32_t a = __ldcg(reinterpret_cast<const uint32_t *>(qh + i)), b = __ldcg(reinterpret_cast<const uint32_t *>(row + i));
            dot = fmaf(__uint_as_float(a << 16), __uint_as_float(b << 16), dot);
            dot = fmaf(__uint_as_float(a & 0xffff0000u), __uint_as_float(b & 0xffff0000u), dot);
        }
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o2);
        if (lane == 0) sx[t] = dot * scale;
    }
    __syncthreads();
    if (tid < T) {                                                 // weights of the parts and of the new row, normaliser
        const int t = tid, npart = rows.npart[t];
        float Mx = sx[t];
        for (int s = 0; s < npart; ++s) Mx = fmaxf(Mx, sm[t][s]);
        const float wx = __expf(sx[t] - Mx);
        float L = wx;
        for (int s = 0; s < npart; ++s) {
            const float wgt = (sm[t][s] == -INFINITY) ? 0.f : __expf(sm[t][s] - Mx);
            sw[t][s] = wgt;
            L = fmaf(wgt, sl[t][s], L);
        }
        swx[t] = wx; sinv[t] = 1.0f / L;
    }
    __syncthreads();
    // merge: two columns per thread, every token
    const int c = 2 * tid;
    for (int t = 0; t < T; ++t) {
        const int npart = rows.npart[t];
        const float *Ot = part.O + ((size_t)t * rows.slot_stride * H + h) * K + c;
        float2 v[kMaxParts];
#pragma unroll
        for (int s = 0; s < kMaxParts; ++s)
            v[s] = (s < npart) ? __ldcg(reinterpret_cast<const float2 *>(Ot + (size_t)s * H * K)) : make_float2(0.f, 0.f);
        const uint32_t rv = __ldcg(reinterpret_cast<const uint32_t *>(cache + rows.new_row[t] + c));
        float2 acc = make_float2(swx[t] * __uint_as_float(rv << 16), swx[t] * __uint_as_float(rv & 0xffff0000u));
#pragma unroll
        for (int s = 0; s < kMaxParts; ++s) {                      // part order: deterministic
            const float wgt = (s < npart) ? sw[t][s] : 0.f;
            acc.x = fmaf(wgt, v[s].x, acc.x);
            acc.y = fmaf(wgt, v[s].y, acc.y);
        }
        const uint32_t ob = pack2(acc.x * sinv[t], acc.y * sinv[t]);
        *reinterpret_cast<uint32_t *>(o_lat_bf16 + ((size_t)t * H + h) * K + c) = ob;
        *reinterpret_cast<uint32_t *>(&x_s[t][c]) = ob;            // W_UV sees the rounded o_lat, as the stage-wise definition says
    }
    __syncthreads();
    for (int t0 = 0; t0 < T; t0 += kTokGroup) {
        float acc[kTokGroup][8];
#pragma unroll
        for (int g = 0; g < kTokGroup; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[g][j] = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            float b[8];
            uint4 wi = w[i];
            // keeps the widening of the weights inside the group loop: hoisted out of it, the 256 widened values
            // of a thread would not fit its registers
            asm volatile("" : "+r"(wi.x), "+r"(wi.y), "+r"(wi.z), "+r"(wi.w));
            Elem<bf16_t>::unpack(wi, b);
#pragma unroll
            for (int g = 0; g < kTokGroup; ++g) {
                const float a = bf2f(x_s[min(t0 + g, kMaxBatch - 1)][ty + i * kRowGroups]);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[g][j] = fmaf(a, b[j], acc[g][j]);
            }
        }
#pragma unroll
        for (int g = 0; g < kTokGroup; ++g) {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[g][j] += __shfl_xor_sync(0xffffffffu, acc[g][j], 16);    // row groups 2j + 2j+1
            if ((tid & 16) == 0) {
                float4 *dst = reinterpret_cast<float4 *>(&red[g][ty >> 1][tx * 8]);
                dst[0] = make_float4(acc[g][0], acc[g][1], acc[g][2], acc[g][3]);
                dst[1] = make_float4(acc[g][4], acc[g][5], acc[g][6], acc[g][7]);
            }
        }
        __syncthreads();
        // 4 tokens x 128 columns = 512 outputs, two per thread; row-group pairs added in a fixed order
        {
            const int g = tid / 64, col = (tid % 64) * 2;
            if (t0 + g < T) {
                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                for (int r = 0; r < kRowGroups / 2; ++r) { s0 += red[g][r][col]; s1 += red[g][r][col + 1]; }
                *reinterpret_cast<uint32_t *>(o + ((size_t)(t0 + g) * H + h) * N + col) = pack2(s0, s1);
            }
        }
        __syncthreads();                                           // red is reused by the next group
    }
}

// ---- the same two stages without the per-head products, for batches large enough that those products belong on
//      the tensor cores (the batched swap-AB kernel): RoPE of every token's query heads, and the merge alone ------

// grid (T, parts): q_full[t, h, dc:] = RoPE(q[t, h, nope:]) for every head; the heads of a token are dealt to `parts` CTAs.
__global__ void __launch_bounds__(kThreadsB) rope_batch_kernel(const uint16_t *__restrict__ q, const float *__restrict__ cs,
                                                               uint16_t *__restrict__ q_full, int H, int nope, int dc, int rope)
{
    const int t = blockIdx.x, half = rope / 2;
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // q comes from the W_UQR product
    for (int i = blockIdx.y * kThreadsB + threadIdx.x; i < H * half; i += kThreadsB * gridDim.y) {
        const int h = i / half, pr = i - h * half;
        const uint32_t xv = *reinterpret_cast<const uint32_t *>(q + ((size_t)t * H + h) * (nope + rope) + nope + 2 * pr);
        const float2 c = *reinterpret_cast<const float2 *>(cs + (size_t)t * rope + 2 * pr);
        const float x0 = __uint_as_float(xv << 16), x1 = __uint_as_float(xv & 0xffff0000u);
        *reinterpret_cast<uint32_t *>(q_full + ((size_t)t * H + h) * (dc + rope) + dc + 2 * pr) = pack2(x0 * c.x - x1 * c.y, x0 * c.y + x1 * c.x);
    }
}

// grid (H, T), 128 threads: log-sum-exp merge of the attention partials of sequence t and of the row the step just
// wrote, for one head; o_lat rounded to bf16.  dc = 512: four columns per thread.
constexpr int kMergeThreads = 128;
__global__ void __launch_bounds__(kMergeThreads) attn_merge_batch_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                                         AttnPartials part, const BatchRows rows, int rope, float scale,
                                                                         uint16_t *__restrict__ o_lat_bf16)
{
    constexpr int K = 512, kMaxParts = 16, kFirst = 4;
    __shared__ float sm[kMaxParts], sl[kMaxParts], scratch[kMergeThreads / 32];
    const int h = blockIdx.x, H = gridDim.x, t = blockIdx.y, dkv = K + rope, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int npart = rows.npart[t];
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // partials come from the attention kernel
    if (tid < npart) {
        const float2 p = __ldcg(reinterpret_cast<const float2 *>(part.ml + (((size_t)t * rows.slot_stride + tid) * H + h) * 2));
        sm[tid] = p.x; sl[tid] = p.y;
    }
    // the first partial rows and the new row are requested before the score is reduced
    const int c = 4 * tid;
    const float *Ot = part.O + ((size_t)t * rows.slot_stride * H + h) * K + c;
    float4 v[kFirst];
#pragma unroll
    for (int s = 0; s < kFirst; ++s)
        v[s] = (s < npart) ? __ldcg(reinterpret_cast<const float4 *>(Ot + (size_t)s * H * K)) : make_float4(0.f, 0.f, 0.f, 0.f);
    const uint16_t *row = cache + rows.new_row[t];
    const uint2 rv = __ldcg(reinterpret_cast<const uint2 *>(row + c));
    const uint16_t *qh = Q + ((size_t)t * H + h) * dkv;
    float dot = 0.f;
    for (int i = 2 * tid; i < dkv; i += 2 * kMergeThreads) {
        const uint32_t a = __ldcg(reinterpret_cast<const uint32_t *>(qh + i)), b = __ldcg(reinterpret_cast<const uint32_t *>(row + i));
        dot = fmaf(__uint_as_float(a << 16), __uint_as_float(b << 16), dot);
        dot = fmaf(__uint_as_float(a & 0xffff0000u), __uint_as_float(b & 0xffff0000u), dot);
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o2);
    if (lane == 0) scratch[warp] = dot;
    __syncthreads();
    float sx = 0.f;
#pragma unroll
    for (int w = 0; w < kMergeThreads / 32; ++w) sx += scratch[w];
    sx *= scale;
    float Mx = sx;
    for (int s = 0; s < npart; ++s) Mx = fmaxf(Mx, sm[s]);
    const float wx = __expf(sx - Mx);
    float L = wx;
    float4 acc = make_float4(wx * __uint_as_float(rv.x << 16), wx * __uint_as_float(rv.x & 0xffff0000u),
                             wx * __uint_as_float(rv.y << 16), wx * __uint_as_float(rv.y & 0xffff0000u));
    for (int s = 0; s < npart; ++s) {                             // part order: deterministic
        const float wgt = (sm[s] == -INFINITY) ? 0.f : __expf(sm[s] - Mx);
        L = fmaf(wgt, sl[s], L);
        float4 x;
        if (s < kFirst) {
            x = v[0];
#pragma unroll
            for (int u = 1; u < kFirst; ++u) x = (s == u) ? v[u] : x;
        } else {
            x = __ldcg(reinterpret_cast<const float4 *>(Ot + (size_t)s * H * K));
        }
        acc.x = fmaf(wgt, x.x, acc.x); acc.y = fmaf(wgt, x.y, acc.y); acc.z = fmaf(wgt, x.z, acc.z); acc.w = fmaf(wgt, x.w, acc.w);
    }
    const float inv = 1.0f / L;
    *reinterpret_cast<uint2 *>(o_lat_bf16 + ((size_t)t * H + h) * K + c) = make_uint2(pack2(acc.x * inv, acc.y * inv), pack2(acc.z * inv, acc.w * inv));
}

template <typename... Args>
cudaError_t launch_b(void (*kern)(Args...), dim3 grid, cudaStream_t s, bool pdl, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = dim3(kThreadsB); cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace

int launch_down_finish_batch(const void *x, const void *gamma_q, const void *gamma_kv, const float *cos_sin, void *c_qn, void *cache,
                             const BatchRows &rows, int T, int q_lora, int dc, int rope, float eps, cudaStream_t s, bool pdl)
{
    cudaError_t e = launch_b(down_finish_batch_kernel, dim3(2, T), s, pdl, (const uint16_t *)x, (const uint16_t *)gamma_q,
                             (const uint16_t *)gamma_kv, cos_sin, (uint16_t *)c_qn, (uint16_t *)cache, rows, q_lora, dc, rope, eps);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "down_finish (batch) launch");
}

int launch_q_finish_batch(const void *q, const void *W_UK, const float *cos_sin, void *q_full, int H, int rope, int T, cudaStream_t s, bool pdl)
{
    cudaError_t e = launch_b(q_finish_batch_kernel, dim3(H), s, pdl, (const uint16_t *)q, (const uint16_t *)W_UK, cos_sin, (uint16_t *)q_full, rope, T);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "q_finish (batch) launch");
}

int launch_uv_merge_batch(const void *Q, const void *cache, AttnPartials part, const BatchRows &rows, int T, int rope, float scale,
                          const void *W_UV, void *o_lat_bf16, void *o, int H, cudaStream_t s, bool pdl)
{
    for (int t = 0; t < T; ++t)
        if (rows.npart[t] < 0 || rows.npart[t] > 16) return NM_ERR_UNSUPPORTED;
    cudaError_t e = launch_b(uv_merge_batch_kernel, dim3(H), s, pdl, (const uint16_t *)Q, (const uint16_t *)cache, part, rows, rope, scale,
                             (const uint16_t *)W_UV, (uint16_t *)o_lat_bf16, (uint16_t *)o, T);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "uv_merge (batch) launch");
}

int launch_rope_batch(const void *q, const float *cos_sin, void *q_full, int H, int nope, int dc, int rope, int T, cudaStream_t s, bool pdl)
{
    const int parts = (H * (rope / 2) + kThreadsB - 1) / kThreadsB;      // one pair per thread
    cudaError_t e = launch_b(rope_batch_kernel, dim3(T, parts < 1 ? 1 : parts), s, pdl, (const uint16_t *)q, cos_sin, (uint16_t *)q_full, H, nope, dc, rope);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "rope (batch) launch");
}

int launch_attn_merge_batch(const void *Q, const void *cache, AttnPartials part, const BatchRows &rows, int T, int rope, float scale,
                            void *o_lat_bf16, int H, cudaStream_t s, bool pdl)
{
    for (int t = 0; t < T; ++t)
        if (rows.npart[t] < 0 || rows.npart[t] > 16) return NM_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(H, T); cfg.blockDim = dim3(kMergeThreads); cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_merge_batch_kernel, (const uint16_t *)Q, (const uint16_t *)cache, part, rows, rope, scale,
                                       (uint16_t *)o_lat_bf16);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention merge (batch) launch");
}

}  // namespace nm
