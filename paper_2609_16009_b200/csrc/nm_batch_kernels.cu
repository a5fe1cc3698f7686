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

// y[0..N) = x[0..K) * W[K][N] with this thread's 32 weight vectors in `w` (rows ty + i * kRowGroups, eight
// columns from 8 tx): partial sums to shared memory, row groups added in a fixed order by the threads with
// ty == 0, which get the eight column sums in out8.
template <int K, int N>
__device__ __forceinline__ void head_matvec(const uint4 (&w)[32], const float *x_s, float *red, float (&out8)[8])
{
    constexpr int kColGroups = N / 8, kRowGroups = kThreadsB / kColGroups;
    static_assert(K / kRowGroups == 32, "128x512 or 512x128");
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
        for (int g = 0; g < kRowGroups; ++g) {
            const float4 *src = reinterpret_cast<const float4 *>(red + (size_t)g * N + tx * 8);
            const float4 v0 = src[0], v1 = src[1];
            out8[0] += v0.x; out8[1] += v0.y; out8[2] += v0.z; out8[3] += v0.w;
            out8[4] += v1.x; out8[5] += v1.y; out8[6] += v1.z; out8[7] += v1.w;
        }
    }
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

// For head blockIdx.x and every token t: q_rope = RoPE(q[t, h, nope:]), q_lat = q[t, h, :nope] * W_UK[h].
// q: [T][H][nope + rope]; q_full: [T][H][dc + rope] (q_lat | q_rope).  nope = 128, dc = 512.
__global__ void __launch_bounds__(kThreadsB) q_finish_batch_kernel(const uint16_t *__restrict__ q, const uint16_t *__restrict__ W_UK,
                                                                   const float *__restrict__ cs, uint16_t *__restrict__ q_full, int rope, int T)
{
    constexpr int K = 128, N = 512, kColGroups = N / 8, kRowGroups = kThreadsB / kColGroups;
    __shared__ __align__(16) float x_s[K];
    __shared__ __align__(16) float red[kRowGroups * N];
    const int h = blockIdx.x, H = gridDim.x, tid = threadIdx.x;
    const int tx = tid % kColGroups, ty = tid / kColGroups;
    const uint16_t *W = W_UK + (size_t)h * K * N + (size_t)ty * N + tx * 8;
    uint4 w[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = ld_stream16(W + (size_t)i * kRowGroups * N);
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // q comes from the W_UQR product
    for (int t = 0; t < T; ++t) {
        const uint16_t *qh = q + ((size_t)t * H + h) * (K + rope);
        uint16_t *dst = q_full + ((size_t)t * H + h) * (N + rope);
        if (tid < K) x_s[tid] = bf2f(qh[tid]);
        if (tid < rope / 2) {
            const float c = cs[(size_t)t * rope + 2 * tid], s = cs[(size_t)t * rope + 2 * tid + 1];
            const float x0 = bf2f(qh[K + 2 * tid]), x1 = bf2f(qh[K + 2 * tid + 1]);
            *reinterpret_cast<uint32_t *>(dst + N + 2 * tid) = pack2(x0 * c - x1 * s, x0 * s + x1 * c);
        }
        __syncthreads();
        float out8[8];
        head_matvec<K, N>(w, x_s, red, out8);
        if (ty == 0) {
            uint4 o;
            o.x = pack2(out8[0], out8[1]); o.y = pack2(out8[2], out8[3]); o.z = pack2(out8[4], out8[5]); o.w = pack2(out8[6], out8[7]);
            *reinterpret_cast<uint4 *>(dst + tx * 8) = o;
        }
        __syncthreads();                                           // x_s and red are reused by the next token
    }
}

// For head blockIdx.x and every token t: log-sum-exp merge of the attention partials of sequence t and of the
// row the step just wrote, o_lat rounded to bf16, then o[t, h] = o_lat[t, h] * W_UV[h].  dc = 512, dv = 128.
__global__ void __launch_bounds__(kThreadsB) uv_merge_batch_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                                   AttnPartials part, const BatchRows rows, int rope, float scale,
                                                                   const uint16_t *__restrict__ W_UV, uint16_t *__restrict__ o_lat_bf16,
                                                                   uint16_t *__restrict__ o, int T)
{
    constexpr int K = 512, N = 128, kColGroups = N / 8, kRowGroups = kThreadsB / kColGroups;
    constexpr int kMaxParts = 64;
    __shared__ __align__(16) float x_s[K];
    __shared__ __align__(16) float red[kRowGroups * N];
    __shared__ float scratch[32];
    __shared__ float sm[kMaxParts], sl[kMaxParts], sw[kMaxParts];
    const int h = blockIdx.x, H = gridDim.x, dkv = K + rope, tid = threadIdx.x;
    const int tx = tid % kColGroups, ty = tid / kColGroups;
    const uint16_t *W = W_UV + (size_t)h * K * N + (size_t)ty * N + tx * 8;
    uint4 w[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = ld_stream16(W + (size_t)i * kRowGroups * N);
    pdl_launch_dependents();
    pdl_wait_prior_grids();                                       // partials come from the attention kernel
    const int c = 2 * tid;
    for (int t = 0; t < T; ++t) {
        const int npart = rows.npart[t];
        const float *ml = part.ml + (size_t)t * rows.slot_stride * H * 2;
        const float *Ot = part.O + (size_t)t * rows.slot_stride * H * K + (size_t)h * K + c;
        const uint16_t *new_row = cache + rows.new_row[t];
        constexpr int kBatch = 8;
        float2 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u)
            v[u] = (u < npart) ? __ldcg(reinterpret_cast<const float2 *>(Ot + (size_t)u * H * K)) : make_float2(0.f, 0.f);
        for (int s = tid; s < npart; s += kThreadsB) {
            const float2 p = __ldcg(reinterpret_cast<const float2 *>(ml + ((size_t)s * H + h) * 2));
            sm[s] = p.x; sl[s] = p.y;
        }
        // score of the new row: q . row over all 576 elements
        float dot = 0.f;
        if (tid < dkv / 8) {
            float qf[8], rf[8];
            Elem<bf16_t>::unpack(__ldcg(reinterpret_cast<const uint4 *>(Q + ((size_t)t * H + h) * dkv) + tid), qf);
            Elem<bf16_t>::unpack(__ldcg(reinterpret_cast<const uint4 *>(new_row) + tid), rf);
#pragma unroll
            for (int e = 0; e < 8; ++e) dot = fmaf(qf[e], rf[e], dot);
        }
        const float sx = block_sum(dot, scratch) * scale;
        float Mx = sx;
        for (int s = 0; s < npart; ++s) Mx = fmaxf(Mx, sm[s]);
        const float wx = __expf(sx - Mx);
        float L = wx;
        for (int s = 0; s < npart; ++s) {                          // same order in every thread
            const float wgt = (sm[s] == -INFINITY) ? 0.f : __expf(sm[s] - Mx);
            if (tid == 0) sw[s] = wgt;
            L = fmaf(wgt, sl[s], L);
        }
        __syncthreads();
        const uint32_t rv = *reinterpret_cast<const uint32_t *>(new_row + c);
        float2 acc = make_float2(wx * __uint_as_float(rv << 16), wx * __uint_as_float(rv & 0xffff0000u));
        for (int s0 = 0; s0 < npart; s0 += kBatch) {
            if (s0 > 0) {
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
                    v[u] = (s0 + u < npart) ? __ldcg(reinterpret_cast<const float2 *>(Ot + (size_t)(s0 + u) * H * K)) : make_float2(0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const float wgt = (s0 + u < npart) ? sw[s0 + u] : 0.f;
                acc.x = fmaf(wgt, v[u].x, acc.x);
                acc.y = fmaf(wgt, v[u].y, acc.y);
            }
        }
        const float inv = 1.0f / L;
        const uint16_t b0 = f2bf(acc.x * inv), b1 = f2bf(acc.y * inv);
        *reinterpret_cast<uint32_t *>(o_lat_bf16 + ((size_t)t * H + h) * K + c) = (uint32_t)b0 | ((uint32_t)b1 << 16);
        x_s[c] = bf2f(b0);                                         // W_UV sees the rounded o_lat, as the stage-wise definition says
        x_s[c + 1] = bf2f(b1);
        __syncthreads();
        float out8[8];
        head_matvec<K, N>(w, x_s, red, out8);
        if (ty == 0) {
            uint4 ov;
            ov.x = pack2(out8[0], out8[1]); ov.y = pack2(out8[2], out8[3]); ov.z = pack2(out8[4], out8[5]); ov.w = pack2(out8[6], out8[7]);
            *reinterpret_cast<uint4 *>(o + ((size_t)t * H + h) * N + tx * 8) = ov;
        }
        __syncthreads();                                           // shared buffers are reused by the next token
    }
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
        if (rows.npart[t] < 0 || rows.npart[t] > 64) return NM_ERR_UNSUPPORTED;
    cudaError_t e = launch_b(uv_merge_batch_kernel, dim3(H), s, pdl, (const uint16_t *)Q, (const uint16_t *)cache, part, rows, rope, scale,
                             (const uint16_t *)W_UV, (uint16_t *)o_lat_bf16, (uint16_t *)o, T);
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "uv_merge (batch) launch");
}

}  // namespace nm
