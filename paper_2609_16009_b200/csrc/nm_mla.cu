// Single-token MLA decode step: the vector-side stages (RMSNorm, RoPE, cache-row write), the merge
// of the attention splits, and the host orchestration that overlaps the CUDA-core narrow products
// with the tensor-core attention pass.
#include <cmath>

#include "nm_async.cuh"
#include "nm_mla.cuh"

namespace nm {

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
__global__ void __launch_bounds__(256) rmsnorm_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ gamma,
                                                      uint16_t *__restrict__ y, int n, float eps)
{
    __shared__ float scratch[32];
    pdl_wait_prior_grids();
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
// both rounded to bf16 and written into the cache row.
__global__ void __launch_bounds__(256) kv_finish_kernel(const uint16_t *__restrict__ ckr, const uint16_t *__restrict__ gamma,
                                                        const float *__restrict__ cs, uint16_t *__restrict__ cache_row,
                                                        int dc, int dr, float eps)
{
    __shared__ float scratch[32];
    pdl_wait_prior_grids();
    float ss = 0.f;
    for (int i = threadIdx.x; i < dc; i += blockDim.x) {
        const float v = bf16_bits_to_f32(ckr[i]);
        ss = fmaf(v, v, ss);
    }
    ss = block_sum(ss, scratch);
    const float r = 1.0f / sqrtf(ss / (float)dc + eps);
    for (int i = threadIdx.x; i < dc; i += blockDim.x)
        cache_row[i] = f32_to_bf16_bits(bf16_bits_to_f32(ckr[i]) * r * bf16_bits_to_f32(gamma[i]));
    for (int i = threadIdx.x; i < dr / 2; i += blockDim.x) {
        const float c = cs[2 * i], s = cs[2 * i + 1];
        const float x0 = bf16_bits_to_f32(ckr[dc + 2 * i]), x1 = bf16_bits_to_f32(ckr[dc + 2 * i + 1]);
        cache_row[dc + 2 * i] = f32_to_bf16_bits(x0 * c - x1 * s);
        cache_row[dc + 2 * i + 1] = f32_to_bf16_bits(x0 * s + x1 * c);
    }
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
__global__ void __launch_bounds__(128) attn_combine_kernel(const uint16_t *__restrict__ Q, const uint16_t *__restrict__ cache,
                                                           AttnPartials part, int nsplit, long extra_row, int dc, int dr,
                                                           float scale, uint16_t *__restrict__ o_bf16, float *__restrict__ o_f32)
{
    const int h = blockIdx.x, H = gridDim.x, dkv = dc + dr;
    __shared__ float scratch[32];
    __shared__ float sw[kMaxAttnSplits];
    pdl_wait_prior_grids();
    float sx = -INFINITY;
    if (extra_row >= 0) {
        const uint16_t *qh = Q + (size_t)h * dkv, *row = cache + (size_t)extra_row * dkv;
        float acc = 0.f;
        for (int i = threadIdx.x; i < dkv; i += blockDim.x) acc = fmaf(bf16_bits_to_f32(qh[i]), bf16_bits_to_f32(row[i]), acc);
        sx = block_sum(acc, scratch) * scale;
    }
    float Mx = sx;
    for (int s = 0; s < nsplit; ++s) Mx = fmaxf(Mx, part.ml[((size_t)s * H + h) * 2]);
    for (int s = threadIdx.x; s < nsplit; s += blockDim.x) {
        const float ms = part.ml[((size_t)s * H + h) * 2];
        sw[s] = (ms == -INFINITY) ? 0.f : __expf(ms - Mx);
    }
    __syncthreads();
    const float wx = (extra_row >= 0) ? __expf(sx - Mx) : 0.f;
    float L = wx;
    for (int s = 0; s < nsplit; ++s) L += sw[s] * part.ml[((size_t)s * H + h) * 2 + 1];
    const float inv = 1.0f / L;
    for (int c = threadIdx.x; c < dc; c += blockDim.x) {
        float acc = (extra_row >= 0) ? wx * bf16_bits_to_f32(cache[(size_t)extra_row * dkv + c]) : 0.f;
        for (int s = 0; s < nsplit; ++s) acc = fmaf(sw[s], part.O[((size_t)s * H + h) * dc + c], acc);
        const float o = acc * inv;
        if (o_f32) o_f32[(size_t)h * dc + c] = o;
        if (o_bf16) o_bf16[(size_t)h * dc + c] = f32_to_bf16_bits(o);
    }
}

// ---- host -------------------------------------------------------------------------------------------

static int g_attn_impl = 0;          // 0: tensor-core kernel when the shape allows, 1: CUDA-core kernel

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

AttnPlan plan_attention(int H, int n_rows, int kv_lora)
{
    AttnPlan p{};
    (void)H; (void)kv_lora;
    const int tiles = ceil_div(n_rows > 0 ? n_rows : 0, kAttnTileRows);
    // 64 splits x 2 column halves = 128 CTAs: one wave of the 148 SMs, leaving a few for the narrow
    // products that run beside the attention pass
    constexpr int kSplitTarget = 64;
    int nsplit = tiles < kSplitTarget ? tiles : kSplitTarget;
    if (nsplit < 1) nsplit = (n_rows > 0) ? 1 : 0;
    p.nsplit = nsplit;
    p.rows_per_split = nsplit ? ceil_div(tiles, nsplit) * kAttnTileRows : 0;
    p.nsplit = p.rows_per_split ? ceil_div(n_rows, p.rows_per_split) : 0;
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
                             void *ws, size_t ws_bytes, cudaStream_t s)
{
    if (!Q || !cache || !ws) return NM_ERR_INVALID_ARG;
    if (H < 1 || n_rows < 0 || dc != 512 || dr != 64) return NM_ERR_UNSUPPORTED;
    if (ws_bytes < attention_ws_bytes(H, dc)) return NM_ERR_WORKSPACE;
    if (n_rows == 0) return NM_OK;
    const AttnPlan p = plan_attention(H, n_rows, dc);
    AttnPartials part = carve_partials(ws, H);
    if (g_attn_impl == 0 && H == 128) {
        int rc = attention_partial_tc(Q, cache, part, p, n_rows, scale, s);
        if (rc != NM_ERR_UNSUPPORTED) return rc;
    }
    attn_partial_simt_kernel<<<dim3(p.nsplit, H), 128, 0, s>>>(static_cast<const uint16_t *>(Q), static_cast<const uint16_t *>(cache),
                                                             part, n_rows, p.rows_per_split, dc, dr, scale);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention (CUDA cores) launch");
}

static int attention_combine(const void *Q, const void *cache, void *o_bf16, float *o_f32, int H, int n_rows, long extra_row,
                             int dc, int dr, float scale, void *ws, size_t ws_bytes, cudaStream_t s)
{
    if (!Q || !cache || !ws || (!o_bf16 && !o_f32)) return NM_ERR_INVALID_ARG;
    if (H < 1 || n_rows < 0 || dc != 512 || dr != 64) return NM_ERR_UNSUPPORTED;
    if (n_rows == 0 && extra_row < 0) return NM_ERR_INVALID_ARG;
    if (ws_bytes < attention_ws_bytes(H, dc)) return NM_ERR_WORKSPACE;
    const AttnPlan p = plan_attention(H, n_rows, dc);
    attn_combine_kernel<<<H, 128, 0, s>>>(static_cast<const uint16_t *>(Q), static_cast<const uint16_t *>(cache), carve_partials(ws, H),
                                          p.nsplit, extra_row, dc, dr, scale, static_cast<uint16_t *>(o_bf16), o_f32);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? NM_OK : record_cuda_error(e, "attention combine launch");
}

// Workspace of the decode step: [main-stream matmul workspace][side-stream matmul workspace]
// [attention partials][intermediates].  Each matmul workspace is [64 KB counters][partials].
struct StepLayout {
    size_t main_ws, main_ws_bytes, side_ws, side_ws_bytes, attn, attn_bytes;
    size_t c_q, c_qn, q, q_full, ckr, o_lat, o, total;
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
    upd(p->q_lora, p->d, 1); upd(p->H * dq, p->q_lora, 1); upd(p->kv_lora, p->nope, p->H); upd(p->v, p->kv_lora, p->H);
    upd(p->d, p->H * p->v, 1);
    size_t off = 0;
    L.main_ws = off; L.main_ws_bytes = main_need; off += align_up(main_need, 256);
    L.side_ws = off; L.side_ws_bytes = nm_matmul_workspace_bytes(1, dkv, p->d, 1, NM_BF16, NM_ROW_MAJOR);
    off += align_up(L.side_ws_bytes, 256);
    L.attn = off; L.attn_bytes = attention_ws_bytes(p->H, p->kv_lora); off += align_up(L.attn_bytes, 256);
    auto take = [&](size_t elems) { size_t o = off; off += align_up(elems * 2, 256); return o; };
    L.c_q = take(p->q_lora); L.c_qn = take(p->q_lora); L.q = take((size_t)p->H * dq); L.q_full = take((size_t)p->H * dkv);
    L.ckr = take(dkv); L.o_lat = take((size_t)p->H * p->kv_lora); L.o = take((size_t)p->H * p->v);
    L.total = off;
    return L;
}

static int check_params(const nm_mla_params *p)
{
    if (!p) return NM_ERR_INVALID_ARG;
    if (!p->h || !p->W_DQ || !p->gamma_q || !p->W_UQR || !p->W_DKVKR || !p->gamma_kv || !p->W_UK || !p->W_UV ||
        !p->rope_cos_sin || !p->kv_cache || !p->workspace)
        return NM_ERR_INVALID_ARG;
    if (p->W_O && !p->out) return NM_ERR_INVALID_ARG;
    if (p->d < 1 || p->q_lora < 1 || p->H < 1 || p->nope < 1 || p->v < 1 || p->seq_len < 1) return NM_ERR_INVALID_ARG;
    if (p->kv_lora != 512 || p->rope != 64) return NM_ERR_UNSUPPORTED;
    if (p->q_lora > 16384) return NM_ERR_UNSUPPORTED;
    if (p->layout_dense != NM_ROW_MAJOR && p->layout_dense != NM_COL_MAJOR) return NM_ERR_UNSUPPORTED;
    return NM_OK;
}

#define NM_TRY(expr) do { int _rc = (expr); if (_rc != NM_OK) return _rc; } while (0)
#define NM_LAUNCH_CHECK(what) do { cudaError_t _e = cudaGetLastError(); if (_e != cudaSuccess) return record_cuda_error(_e, what); } while (0)

// Events used to fork the KV chain onto the side stream and join it again (created once per thread).
struct StepEvents { cudaEvent_t fork = nullptr, join = nullptr; };
static thread_local StepEvents g_events;

static int step_impl(const nm_mla_params *p, cudaStream_t ms, cudaStream_t ss)
{
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
    const bool forked = (ss != ms);
    if (forked && !g_events.fork) {
        NM_CUDA_TRY(cudaEventCreateWithFlags(&g_events.fork, cudaEventDisableTiming));
        NM_CUDA_TRY(cudaEventCreateWithFlags(&g_events.join, cudaEventDisableTiming));
    }

    // ---- Q chain, main stream ------------------------------------------------------------------------
    NM_TRY(matmul_enqueue(p->h, p->W_DQ, c_q, 1, ql, d, 1, d, 0, 0, ql, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms));
    rmsnorm_kernel<<<1, 256, 0, ms>>>(c_q, (const uint16_t *)p->gamma_q, c_qn, ql, p->rms_eps);
    NM_LAUNCH_CHECK("rmsnorm launch");
    NM_TRY(matmul_enqueue(c_qn, p->W_UQR, q, 1, H * dq, ql, 1, ql, 0, 0, H * dq, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms));
    rope_kernel<<<ceil_div(H * dr / 2, 256), 256, 0, ms>>>(q + dn, q_full + dc, H, dr, dq, dkv, p->rope_cos_sin);
    NM_LAUNCH_CHECK("rope launch");
    // q_lat[h] = q[h, :nope] * W_UK[h], written straight into the attention operand [H][dc+dr]
    NM_TRY(matmul_enqueue(q, p->W_UK, q_full, 1, dc, dn, H, (long)H * dq, dq, (long)dn * dc, (long)H * dkv, dkv,
                          NM_BF16, NM_ROW_MAJOR, mws, L.main_ws_bytes, ms));

    // ---- KV chain (the paper's MatMul 2 and its consumers): side stream, concurrent with the attention
    //      pass over the old rows ---------------------------------------------------------------------------
    if (forked) {
        NM_CUDA_TRY(cudaEventRecord(g_events.fork, ms));
        NM_CUDA_TRY(cudaStreamWaitEvent(ss, g_events.fork, 0));
    }
    NM_TRY(matmul_enqueue(p->h, p->W_DKVKR, ckr, 1, dkv, d, 1, d, 0, 0, dkv, 0, NM_BF16, lay, sws, L.side_ws_bytes, ss));
    kv_finish_kernel<<<1, 256, 0, ss>>>(ckr, (const uint16_t *)p->gamma_kv, p->rope_cos_sin, cache + (size_t)pos * dkv, dc, dr, p->rms_eps);
    NM_LAUNCH_CHECK("kv finish launch");
    if (forked) NM_CUDA_TRY(cudaEventRecord(g_events.join, ss));

    // ---- attention over the old rows (tensor cores), main stream; the new row joins in the merge -----------
    NM_TRY(attention_partial(q_full, cache, H, (int)pos, dc, dr, p->softmax_scale, aws, L.attn_bytes, ms));
    if (forked) NM_CUDA_TRY(cudaStreamWaitEvent(ms, g_events.join, 0));
    NM_TRY(attention_combine(q_full, cache, o_lat, p->o_lat_f32, H, (int)pos, pos, dc, dr, p->softmax_scale, aws, L.attn_bytes, ms));

    // ---- output side -----------------------------------------------------------------------------------
    NM_TRY(matmul_enqueue(o_lat, p->W_UV, o, 1, dv, dc, H, (long)H * dc, dc, (long)dc * dv, (long)H * dv, dv,
                          NM_BF16, NM_ROW_MAJOR, mws, L.main_ws_bytes, ms));
    if (p->W_O) {
        if (p->event_before_wo) NM_CUDA_TRY(cudaEventRecord((cudaEvent_t)p->event_before_wo, ms));
        NM_TRY(matmul_enqueue(o, p->W_O, p->out, 1, d, H * dv, 1, (long)H * dv, 0, 0, d, 0, NM_BF16, lay, mws, L.main_ws_bytes, ms));
        if (p->event_after_wo) NM_CUDA_TRY(cudaEventRecord((cudaEvent_t)p->event_after_wo, ms));
    }
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
    return attention_partial(Q, kv_cache, H, n_rows, kv_lora, rope, scale, workspace, workspace_bytes, (cudaStream_t)stream);
}

int nm_mla_attention_combine(const void *Q, const void *kv_cache, void *o_bf16, float *o_f32, int H, int n_rows, long extra_row,
                             int kv_lora, int rope, float scale, void *workspace, size_t workspace_bytes, nm_stream stream)
{
    return attention_combine(Q, kv_cache, o_bf16, o_f32, H, n_rows, extra_row, kv_lora, rope, scale, workspace, workspace_bytes,
                             (cudaStream_t)stream);
}

int nm_mla_attention(const void *Q, const void *kv_cache, void *o_bf16, float *o_f32, int H, int n_rows, long extra_row,
                     int kv_lora, int rope, float scale, void *workspace, size_t workspace_bytes, nm_stream stream)
{
    NM_TRY(attention_partial(Q, kv_cache, H, n_rows, kv_lora, rope, scale, workspace, workspace_bytes, (cudaStream_t)stream));
    return attention_combine(Q, kv_cache, o_bf16, o_f32, H, n_rows, extra_row, kv_lora, rope, scale, workspace, workspace_bytes,
                             (cudaStream_t)stream);
}

size_t nm_mla_workspace_bytes(const nm_mla_params *p)
{
    if (!p || p->H < 1 || p->d < 1 || p->q_lora < 1) return 0;
    return step_layout(p).total;
}

int nm_mla_decode_step(const nm_mla_params *p, nm_stream main_stream, nm_stream side_stream)
{
    return step_impl(p, (cudaStream_t)main_stream, (cudaStream_t)side_stream);
}

int nm_mla_decode_step_host(const nm_mla_params *p, const void *h_host, void *out_host, void *h_staging, void *out_staging,
                            nm_stream main_stream, nm_stream side_stream)
{
    if (!p || !h_host || !out_host || !h_staging || !out_staging || !p->W_O) return NM_ERR_INVALID_ARG;
    nm_mla_params q = *p;
    q.h = h_staging;
    q.out = out_staging;
    NM_TRY(check_params(&q));
    cudaStream_t ms = (cudaStream_t)main_stream;
    NM_CUDA_TRY(cudaMemcpyAsync(h_staging, h_host, (size_t)p->d * 2, cudaMemcpyHostToDevice, ms));
    NM_TRY(step_impl(&q, ms, (cudaStream_t)side_stream));
    NM_CUDA_TRY(cudaMemcpyAsync(out_host, out_staging, (size_t)p->d * 2, cudaMemcpyDeviceToHost, ms));
    return NM_OK;
}

/* 0: tensor-core attention when the shape allows (default); 1: CUDA-core attention kernel. */
int nm_debug_set_attention(int impl)
{
    g_attn_impl = impl;
    return NM_OK;
}

#pragma GCC visibility pop
}
