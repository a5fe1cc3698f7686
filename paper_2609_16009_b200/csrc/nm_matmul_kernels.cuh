// Narrow matrix product kernels: C[MxN] = A[MxK] * B[KxN], 1 <= M <= 16, on CUDA cores.
//
// B is streamed from HBM exactly once with 16-byte read-only loads; A is staged in shared memory;
// products accumulate in fp32 registers; K may be split over CTAs, in which case every CTA stores
// an fp32 partial tile and the last CTA to arrive at a tile sums the partials in split order
// (deterministic) and rounds once to the output type.  This is the split-K / partial-sum-buffer /
// gather structure of Algorithm 1, with the device-wide barrier replaced by an arrival counter so
// that no CTA ever waits on another.
#pragma once

#include "nm_async.cuh"
#include "nm_common.cuh"

namespace nm {

constexpr int kThreads = 256;
constexpr int kSmemFloats = 8192;         // 32 KB: A chunk during the stream, reduction buffer after

struct MatmulArgs {
    const void *A, *B;
    void *C;
    int M, N, K, H;
    long lda, strideA, strideB, ldc, strideC;
    int tn;        // columns per CTA tile
    int tpr;       // row kernel: threads per B row (tn / kVec)
    int rg;        // row kernel: row groups per CTA (kThreads / tpr)
    int nsplit;    // k-splits (gridDim.y)
    int kr;        // k-rows per split (multiple of kVec)
    int ntiles;    // column tiles (gridDim.x)
    int a_vec;     // A rows can be staged with 16-byte loads
    float *partial;
    unsigned *counters;
    int cluster_split;   // plain kernels: the k-splits of a tile form a cluster (1 x nsplit x 1) and meet in shared memory
    unsigned *status;    // device status word (the debug build reports an access outside its operand there)
    int use_pdl;         // plain kernels: launched programmatically - the first weight loads go out before the wait for earlier kernels
};

// Extents of the operands, for the debug build's checks (see NM_BOUNDS_CHECK in nm_common.cuh).
template <typename TI> __device__ __forceinline__ Span span_of_A(const MatmulArgs &a)
{
    return make_span(a.A, (size_t)((long)(a.H - 1) * a.strideA + (long)(a.M - 1) * a.lda + a.K) * sizeof(TI));
}
template <typename TI> __device__ __forceinline__ Span span_of_B(const MatmulArgs &a)
{
    return make_span(a.B, (size_t)((long)(a.H - 1) * a.strideB + (long)a.K * a.N) * sizeof(TI));
}
template <typename TO> __device__ __forceinline__ Span span_of_C(const MatmulArgs &a)
{
    return make_span(a.C, (size_t)((long)(a.H - 1) * a.strideC + (long)(a.M - 1) * a.ldc + a.N) * sizeof(TO));
}
__device__ __forceinline__ Span span_of_partials(const MatmulArgs &a)
{
    return make_span(a.partial, a.partial ? (size_t)a.H * a.ntiles * a.nsplit * (size_t)a.M * a.tn * sizeof(float) : 0);
}

// ---- split-K inside a thread-block cluster (plain kernels) ----------------------------------------------
// The k-splits of a column tile are the CTAs of one cluster.  Each stores its sums into slot [split] of the first
// CTA's shared memory; after a cluster barrier that CTA adds the slots in split order, rounds once and writes C:
// no workspace, fence, counter or gather through L2.  Every CTA arrives on the cluster barrier at its start and
// waits for it before the first remote store (all peers are running by then).
constexpr int kClusterSlotFloats = 2048;                           // 8 KB: nsplit * M * tile_n floats at most
__device__ __forceinline__ void cluster_arrive_all() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_all() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_slot_base(const float *slots, int split, int per_split)
{
    uint32_t local = (uint32_t)__cvta_generic_to_shared(slots + (size_t)split * per_split), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(0));
    return remote;
}
__device__ __forceinline__ void cluster_slot_store(uint32_t base, int i, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(base + (uint32_t)i * 4u), "f"(v) : "memory");
}
// all threads of every CTA of the cluster, after the remote stores
template <typename TO>
__device__ __forceinline__ void cluster_split_finish(const MatmulArgs &a, const float *slots, int M, int tile, int split, int h)
{
    cluster_arrive_all();
    cluster_wait_all();
    if (split != 0) return;
    TO *C = (TO *)a.C + (long)h * a.strideC;
    const int per = M * a.tn;
    for (int i = threadIdx.x; i < per; i += (int)blockDim.x) {
        const int m = i / a.tn, c = i - m * a.tn, n = tile * a.tn + c;
        if (n < a.N) {
            float s = 0.f;
            for (int sp = 0; sp < a.nsplit; ++sp) s += slots[(size_t)sp * per + i];
            NM_ST(&C[(long)m * a.ldc + n], round_out<TO>(s), span_of_C<TO>(a), a.status);
        }
    }
}

// Extra launch state of the TMA-fed kernels.
// The vector stages that consume a down-projection of the decode step, run by whichever CTA completes the
// product's last tile (a grid-wide arrival counter: nobody waits): RMSNorm of x[0, q_lora) -> c_qn, and / or
// RMSNorm of x[kv_off, kv_off + dc) and RoPE of the next `rope` elements -> cache_row.  x is the product's C.
// This is the paper's remark that the normalisation, RoPE and caching start right where MatMul 2 ends
// (MLA Operator Optimization), taken literally: no kernel boundary in between.
struct VecTail {
    int enabled;
    int q_lora, kv_off, dc, rope;          // q_lora == 0: no query part; dc == 0: no KV part
    float eps;
    const uint16_t *gamma_q, *gamma_kv;
    const float *cos_sin;                  // [rope/2][2] for the row's position
    uint16_t *c_qn, *cache_row;
    unsigned *counter;                     // zero on entry, left at zero
};

// RMSNorm applied to the token row as it is loaded (M = 1): the producer of the row left the sum of squares of each
// of its column tiles in `tile_ss`; the consumer adds them in tile order, scales the row by gamma / rms, rounds it to
// bf16 - exactly what a separate RMSNorm stage would have stored - and multiplies that.
struct RowNorm {
    int enabled;
    int n;                                 // elements of the row (= K of the product)
    int ntiles;                            // entries of tile_ss (<= 32)
    float eps;
    const float *tile_ss;
    const uint16_t *gamma;
    uint16_t *normed_out;                  // when non-null, the CTAs of column tile 0 also store the normalised row here
};

struct TmaArgs {
    MatmulArgs base;
    int nstage;            // ring depth
    int use_pdl;           // kernel was launched with programmatic stream serialization
    unsigned *status;      // device status word
    unsigned long long *trace;   // tuning aid: when non-null every CTA stores four timestamps (start, inputs ready, loop done, end)
    VecTail tail;
    int cluster_split;     // the k-splits of a tile form a thread-block cluster (1 x nsplit x 1): partial sums meet in shared memory
    int fractal_nz;        // B is stored in 16 x 16 fractals (5-D tensor map): a stage arrives as [tile_n/16][KT][16] instead of [KT][tile_n]
    float *tile_ss;        // cluster split-K, M = 1: when non-null, tile t also stores the sum of squares of its rounded outputs at [t]
    RowNorm norm;
};

// Sum over the CTA (any size up to 1024 threads, a multiple of 32), same value in every thread.
__device__ __forceinline__ float cta_sum(float v, float *scratch /* 32 floats */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += scratch[w];
    return t;
}

__device__ __forceinline__ uint32_t pack2_bf16_rn(float lo, float hi)
{
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
}

__device__ __forceinline__ unsigned long long tail_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Two sums over the CTA at once (any size up to 1024 threads, a multiple of 32), same values in every thread.
__device__ __forceinline__ float2 cta_sum2(float2 v, float *scratch /* 64 floats */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        v.x += __shfl_xor_sync(0xffffffffu, v.x, o);
        v.y += __shfl_xor_sync(0xffffffffu, v.y, o);
    }
    __syncthreads();
    if (lane == 0) { scratch[2 * warp] = v.x; scratch[2 * warp + 1] = v.y; }
    __syncthreads();
    float2 t = make_float2(0.f, 0.f);
    for (int w = 0; w < nw; ++w) { t.x += scratch[2 * w]; t.y += scratch[2 * w + 1]; }
    return t;
}

// Completion of a product that carries a VecTail (M = 1, bf16 output, one head).  One arrival counter for the
// whole grid instead of one per tile: every CTA publishes its tile (split-K: its fp32 partial tile; otherwise
// the finished bf16 columns) and arrives; the last CTA of the grid gathers every column - partials summed in
// split order, rounded once - writes C, keeps the rounded row in shared memory and runs the vector stages on
// it: RMSNorm of the first q_lora outputs, RMSNorm + RoPE + cache-row write of the outputs from kv_off on.
// Everything that crosses L2 here queues behind the next product of the chain, which is filling its ring from
// HBM at full rate at that very moment (1-3 us per dependent round trip), so there are as few of them as the
// data allows: one fence / atomic; then the constants of the vector stages and the partials of two passes of
// columns are requested together; both sums of squares share one reduction.  `xs` needs N floats (+64 of
// scratch behind them).
__device__ __forceinline__ void tail_complete(const MatmulArgs &a, const VecTail &t, int *s_last, float *xs, unsigned long long *dbg = nullptr)
{
    const int tid = threadIdx.x;
    __threadfence();
    __syncthreads();
    if (tid == 0) *s_last = (atomicAdd(t.counter, 1u) == (unsigned)(a.ntiles * a.nsplit - 1));
    __syncthreads();
    if (!*s_last) return;
    if (dbg && tid == 0) dbg[0] = tail_timer_ns();
    __threadfence();
    if (tid == 0) *t.counter = 0u;
    // constants of the vector stages (8 elements of q_lora <= 2048, 2 of dc <= 512 and of rope <= dc per thread)
    const bool q_on = t.q_lora > 0 && 8 * tid < t.q_lora;
    const bool kv_on = t.dc > 0 && 2 * tid < t.dc, rope_on = t.dc > 0 && 2 * tid < t.rope;
    uint4 gq = make_uint4(0, 0, 0, 0);
    uint32_t gkv = 0;
    float cs = 0.f, sn = 0.f;
    if (q_on) gq = __ldg(reinterpret_cast<const uint4 *>(t.gamma_q + 8 * tid));
    if (kv_on) gkv = __ldg(reinterpret_cast<const uint32_t *>(t.gamma_kv + 2 * tid));
    if (rope_on) { cs = __ldg(t.cos_sin + 2 * tid); sn = __ldg(t.cos_sin + 2 * tid + 1); }

    uint16_t *C = reinterpret_cast<uint16_t *>(a.C);
    // four consecutive columns (one 16-byte load per split) per thread and pass, two passes requested at a time;
    // N and the tile width are multiples of four (checked by the host), so the four columns lie in one tile
    const int stride = 4 * (int)blockDim.x;
    auto finish = [&](int n, float4 sum) {                         // round once, write C, keep the rounded values
        const __nv_bfloat16 b0 = __float2bfloat16_rn(sum.x), b1 = __float2bfloat16_rn(sum.y), b2 = __float2bfloat16_rn(sum.z),
                            b3 = __float2bfloat16_rn(sum.w);
        *reinterpret_cast<uint2 *>(C + n) = make_uint2((uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16),
                                                       (uint32_t)__bfloat16_as_ushort(b2) | ((uint32_t)__bfloat16_as_ushort(b3) << 16));
        *reinterpret_cast<float4 *>(xs + n) = make_float4(__bfloat162float(b0), __bfloat162float(b1), __bfloat162float(b2), __bfloat162float(b3));
    };
    for (int n0 = 4 * tid; n0 < a.N; n0 += 2 * stride) {
        const int n1 = n0 + stride;
        const bool two = n1 < a.N;
        if (a.nsplit > 1) {
            const int nb = two ? n1 : n0;                          // without a second pass its loads repeat the first's
            const int t0 = n0 / a.tn, t1 = nb / a.tn;
            const float *P0 = a.partial + (size_t)t0 * a.nsplit * a.tn + (n0 - t0 * a.tn);
            const float *P1 = a.partial + (size_t)t1 * a.nsplit * a.tn + (nb - t1 * a.tn);
            float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
            for (int sp = 0; sp < a.nsplit; sp += 4) {
                float4 v0[4], v1[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {                      // branch-free: a slot past the last split re-reads it
                    const size_t off = (size_t)min(sp + u, a.nsplit - 1) * a.tn;
                    v0[u] = __ldcg(reinterpret_cast<const float4 *>(P0 + off));
                    v1[u] = __ldcg(reinterpret_cast<const float4 *>(P1 + off));
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)                        // split order: deterministic
                    if (sp + u < a.nsplit) {
                        s0.x += v0[u].x; s0.y += v0[u].y; s0.z += v0[u].z; s0.w += v0[u].w;
                        s1.x += v1[u].x; s1.y += v1[u].y; s1.z += v1[u].z; s1.w += v1[u].w;
                    }
            }
            finish(n0, s0);
            if (two) finish(n1, s1);
        } else {
            const uint2 c0 = __ldcg(reinterpret_cast<const uint2 *>(C + n0));
            const uint2 c1 = __ldcg(reinterpret_cast<const uint2 *>(C + (two ? n1 : n0)));
            *reinterpret_cast<float4 *>(xs + n0) = make_float4(__uint_as_float(c0.x << 16), __uint_as_float(c0.x & 0xffff0000u),
                                                               __uint_as_float(c0.y << 16), __uint_as_float(c0.y & 0xffff0000u));
            if (two)
                *reinterpret_cast<float4 *>(xs + n1) = make_float4(__uint_as_float(c1.x << 16), __uint_as_float(c1.x & 0xffff0000u),
                                                                   __uint_as_float(c1.y << 16), __uint_as_float(c1.y & 0xffff0000u));
        }
    }
    if (dbg && tid == 0) dbg[1] = tail_timer_ns();
    __syncthreads();
    if (dbg && tid == 0) dbg[2] = tail_timer_ns();

    // ---- the vector stages on the rounded row --------------------------------------------------------------
    float f[8], g[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = 0.f;
    if (q_on) {
        const float4 x = *reinterpret_cast<const float4 *>(xs + 8 * tid), y = *reinterpret_cast<const float4 *>(xs + 8 * tid + 4);
        f[0] = x.x; f[1] = x.y; f[2] = x.z; f[3] = x.w; f[4] = y.x; f[5] = y.y; f[6] = y.z; f[7] = y.w;
    }
    Elem<bf16_t>::unpack(gq, g);
    const float *ckr = xs + t.kv_off;
    float x0 = 0.f, x1 = 0.f, r0 = 0.f, r1 = 0.f;
    if (kv_on) { x0 = ckr[2 * tid]; x1 = ckr[2 * tid + 1]; }
    if (rope_on) { r0 = ckr[t.dc + 2 * tid]; r1 = ckr[t.dc + 2 * tid + 1]; }
    float ssq = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) ssq = fmaf(f[e], f[e], ssq);
    const float2 ss = cta_sum2(make_float2(ssq, fmaf(x0, x0, x1 * x1)), xs + ((a.N + 31) & ~31));
    if (dbg && tid == 0) dbg[3] = tail_timer_ns();
    if (q_on) {
        const float r = 1.0f / sqrtf(ss.x / (float)t.q_lora + t.eps);
        uint4 o;
        o.x = pack2_bf16_rn(f[0] * r * g[0], f[1] * r * g[1]); o.y = pack2_bf16_rn(f[2] * r * g[2], f[3] * r * g[3]);
        o.z = pack2_bf16_rn(f[4] * r * g[4], f[5] * r * g[5]); o.w = pack2_bf16_rn(f[6] * r * g[6], f[7] * r * g[7]);
        *reinterpret_cast<uint4 *>(t.c_qn + 8 * tid) = o;
    }
    if (t.dc > 0) {
        const float r = 1.0f / sqrtf(ss.y / (float)t.dc + t.eps);
        const float g0 = __uint_as_float(gkv << 16), g1 = __uint_as_float(gkv & 0xffff0000u);
        if (kv_on) *reinterpret_cast<uint32_t *>(t.cache_row + 2 * tid) = pack2_bf16_rn(x0 * r * g0, x1 * r * g1);
        if (rope_on) *reinterpret_cast<uint32_t *>(t.cache_row + t.dc + 2 * tid) = pack2_bf16_rn(r0 * cs - r1 * sn, r0 * sn + r1 * cs);
    }
}

template <int M> struct RowCfg {
    static constexpr int kUnroll = (M <= 4) ? 8 : (M <= 8 ? 6 : 4);
    static constexpr int kMinBlocks = (M <= 2) ? 3 : (M <= 8 ? 2 : 1);
    static constexpr int kChunk = ((kSmemFloats / M) / 8) * 8;     // k-rows of A held in smem
    static constexpr int kPass = (M < 4) ? M : 4;                  // m-rows reduced per pass
};

// Sum of the nsplit partial tiles of one (head, tile), in split order, rounded once and written to C.
template <typename TO>
__device__ __forceinline__ void splitk_gather(const float *P, TO *C, int M, int tn, int nsplit, int N, int tile, long ldc,
                                              Span span_p, Span span_c, unsigned *status)
{
    (void)span_p; (void)span_c; (void)status;
    // Four outputs per thread and pass, and the partials of all four requested four splits at a time before any
    // is used: a chain of L2 round trips otherwise (M * tile_n outputs x nsplit partials, one CTA).  The inner
    // loops are free of branches - a slot past the thread's last output repeats that output's address and its
    // sum is dropped - so that the loads really are issued back to back.
    constexpr int kOut = 4;
    const int tid = threadIdx.x, total = M * tn, stride = (int)blockDim.x;
    const size_t split_stride = (size_t)M * tn;
    for (int i0 = 0; i0 < total; i0 += kOut * stride) {
        const int live = min(kOut, (total - i0 - tid + stride - 1) / stride);     // outputs this thread has in this pass
        if (live <= 0) continue;
        float s[kOut];
        const float *src[kOut];
#pragma unroll
        for (int j = 0; j < kOut; ++j) {
            src[j] = P + (i0 + min(j, live - 1) * stride + tid);
            s[j] = 0.f;
        }
        int sp = 0;
        for (; sp + 4 <= nsplit; sp += 4) {
            float v[4][kOut];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int j = 0; j < kOut; ++j) v[u][j] = NM_LD_CG(src[j] + (sp + u) * split_stride, span_p, status);
#pragma unroll
            for (int u = 0; u < 4; ++u)                            // split order: deterministic
#pragma unroll
                for (int j = 0; j < kOut; ++j) s[j] += v[u][j];
        }
        for (; sp < nsplit; ++sp) {
            float v[kOut];
#pragma unroll
            for (int j = 0; j < kOut; ++j) v[j] = NM_LD_CG(src[j] + sp * split_stride, span_p, status);
#pragma unroll
            for (int j = 0; j < kOut; ++j) s[j] += v[j];
        }
#pragma unroll
        for (int j = 0; j < kOut; ++j) {
            if (j < live) {
                const int i = i0 + j * stride + tid;
                const int m = i / tn, c = i - m * tn, n = tile * tn + c;
                if (n < N) NM_ST(&C[(long)m * ldc + n], round_out<TO>(s[j]), span_c, status);
            }
        }
    }
}

// ---- split-K completion shared by both kernels -----------------------------------------------------
//
// Called by all threads of the CTA after its partial tile has been written to `partial`.  The
// last CTA to arrive at (h, tile) reads all nsplit partial tiles in order and writes C; it then
// puts the counter back to zero, so the workspace needs no clearing between launches.
template <typename TO, bool kBatched = true>
__device__ __forceinline__ void splitk_complete_rt(const MatmulArgs &a, int M, int tile, int h, int *s_last)
{
    const int tid = threadIdx.x;
    __threadfence();
    __syncthreads();
    unsigned *cnt = a.counters + (size_t)h * a.ntiles + tile;
    if (tid == 0) {
        unsigned t = atomicAdd(cnt, 1u);
        *s_last = (t == (unsigned)(a.nsplit - 1));
    }
    __syncthreads();
    if (!*s_last) return;
    __threadfence();
    const float *P = a.partial + ((size_t)h * a.ntiles + tile) * a.nsplit * (size_t)(M * a.tn);
    TO *C = (TO *)a.C + (long)h * a.strideC;
    if constexpr (!kBatched) {                                     // few outputs per thread (M <= 2): the plain loop, and
        for (int i = tid; i < M * a.tn; i += blockDim.x) {         // nothing that would change the main loop's registers
            const int m = i / a.tn, c = i - m * a.tn, n = tile * a.tn + c;
            if (n < a.N) {
                float s = 0.f;
#pragma unroll 4
                for (int sp = 0; sp < a.nsplit; ++sp) s += NM_LD_CG(P + ((size_t)sp * M + m) * a.tn + c, span_of_partials(a), a.status);
                NM_ST(&C[(long)m * a.ldc + n], round_out<TO>(s), span_of_C<TO>(a), a.status);
            }
        }
    } else {
        splitk_gather<TO>(P, C, M, a.tn, a.nsplit, a.N, tile, a.ldc, span_of_partials(a), span_of_C<TO>(a), a.status);
    }
    if (tid == 0) *cnt = 0u;
}

template <int M, typename TO>
__device__ __forceinline__ void splitk_complete(const MatmulArgs &a, int tile, int h, int *s_last)
{
    splitk_complete_rt<TO, (M > 2)>(a, M, tile, h, s_last);
}

// ---- row-major B (n contiguous): each thread owns kVec consecutive columns ---------------------------
template <int M, typename TI>
__device__ __forceinline__ void fma_row(float (&acc)[M][Elem<TI>::kVec], const uint4 &v,
                                        const float *As /* &As[0][row] */)
{
    constexpr int V = Elem<TI>::kVec;
    float b[V];
    Elem<TI>::unpack(v, b);
#pragma unroll
    for (int m = 0; m < M; ++m) {
        const float am = As[m * RowCfg<M>::kChunk];
#pragma unroll
        for (int j = 0; j < V; ++j) acc[m][j] = fmaf(am, b[j], acc[m][j]);
    }
}

template <int M, typename TI, typename TO>
__global__ void __launch_bounds__(kThreads, RowCfg<M>::kMinBlocks) nm_row_kernel(const MatmulArgs a)
{
    using E = Elem<TI>;
    constexpr int V = E::kVec;
    constexpr int U = RowCfg<M>::kUnroll;
    constexpr int KC = RowCfg<M>::kChunk;
    constexpr int MP = RowCfg<M>::kPass;
    __shared__ __align__(16) float smem[kSmemFloats];
    __shared__ __align__(16) float s_slots[kClusterSlotFloats];
    __shared__ int s_last;
    if (a.cluster_split) cluster_arrive_all();
    pdl_launch_dependents();

    const int tid = threadIdx.x;
    const int tx = tid % a.tpr, ty = tid / a.tpr;
    const int tile = blockIdx.x, split = blockIdx.y, h = blockIdx.z;
    const int n0 = tile * a.tn + tx * V;
    const bool active = (ty < a.rg) && (n0 < a.N);
    const int kb = split * a.kr;
    const int ke = min(a.K, kb + a.kr);
    const int rg = a.rg;
    const long ldb = a.N;
    const TI *__restrict__ A = (const TI *)a.A + (long)h * a.strideA;
    const TI *__restrict__ B = (const TI *)a.B + (long)h * a.strideB;
    const Span sp_a = span_of_A<TI>(a), sp_b = span_of_B<TI>(a), sp_c = span_of_C<TO>(a), sp_p = span_of_partials(a);
    (void)sp_a; (void)sp_b; (void)sp_c; (void)sp_p;

    float acc[M][V];
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int j = 0; j < V; ++j) acc[m][j] = 0.f;

    for (int kc = kb; kc < ke; kc += KC) {
        const int klen = min(KC, ke - kc);
        const TI *bp = B + (long)kc * ldb + n0;
        // First batch of weight loads goes out before A is staged, so the two latencies overlap.
        uint4 v[U];
        int r = ty;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int rr = r + u * rg;
            v[u] = (active && rr < klen) ? NM_LD_STREAM16(bp + (long)rr * ldb, sp_b, a.status) : make_uint4(0, 0, 0, 0);
        }
        if (kc == kb) pdl_wait_prior_grids();             // weights depend on nothing; A and everything written do
        __syncthreads();                                  // readers of the previous chunk are done
        if (a.a_vec) {
            const int nv = klen / V;                      // klen is a multiple of kVec on this path
            for (int m = 0; m < M; ++m) {
                const uint4 *src = (const uint4 *)(A + (long)m * a.lda + kc);
                for (int i = tid; i < nv; i += kThreads) {
                    float f[V];
                    E::unpack(NM_LDG16(src + i, sp_a, a.status), f);
#pragma unroll
                    for (int j = 0; j < V; ++j) smem[m * KC + i * V + j] = f[j];
                }
                for (int i = nv * V + tid; i < klen; i += kThreads) smem[m * KC + i] = E::widen(NM_LD(&A[(long)m * a.lda + kc + i], sp_a, a.status));
            }
        } else {
            for (int m = 0; m < M; ++m)
                for (int i = tid; i < klen; i += kThreads) smem[m * KC + i] = E::widen(NM_LD(&A[(long)m * a.lda + kc + i], sp_a, a.status));
        }
        __syncthreads();
        if (active) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int rr = r + u * rg;
                if (rr < klen) fma_row<M, TI>(acc, v[u], smem + rr);
            }
            r += U * rg;
            for (; r + (U - 1) * rg < klen; r += U * rg) {
#pragma unroll
                for (int u = 0; u < U; ++u) v[u] = NM_LD_STREAM16(bp + (long)(r + u * rg) * ldb, sp_b, a.status);
#pragma unroll
                for (int u = 0; u < U; ++u) fma_row<M, TI>(acc, v[u], smem + r + u * rg);
            }
            for (; r < klen; r += rg) {
                const uint4 w = NM_LD_STREAM16(bp + (long)r * ldb, sp_b, a.status);
                fma_row<M, TI>(acc, w, smem + r);
            }
        }
    }

    // Reduce the rg row groups of the CTA through shared memory, MP rows of C per pass.
    float *red = smem;
    TO *C = (TO *)a.C + (long)h * a.strideC;
    float *P = a.partial ? a.partial + (((size_t)h * a.ntiles + tile) * a.nsplit + split) * (size_t)(M * a.tn) : nullptr;
    uint32_t slot0 = 0;
    if (a.cluster_split) {
        cluster_wait_all();
        slot0 = cluster_slot_base(s_slots, split, M * a.tn);
    }
#pragma unroll
    for (int m0 = 0; m0 < M; m0 += MP) {
        __syncthreads();
        if (ty < rg) {
#pragma unroll
            for (int mm = 0; mm < MP; ++mm) {
                if (m0 + mm < M) {
                    float4 *dst = (float4 *)(red + (size_t)(ty * MP + mm) * a.tn + tx * V);
#pragma unroll
                    for (int j = 0; j < V; j += 4)
                        dst[j / 4] = make_float4(acc[m0 + mm][j], acc[m0 + mm][j + 1], acc[m0 + mm][j + 2], acc[m0 + mm][j + 3]);
                }
            }
        }
        __syncthreads();
        for (int i = tid; i < MP * a.tn; i += kThreads) {
            const int mm = i / a.tn, c = i - mm * a.tn, m = m0 + mm, n = tile * a.tn + c;
            if (m < M && n < a.N) {
                float s = 0.f;
                for (int g = 0; g < rg; ++g) s += red[(size_t)(g * MP + mm) * a.tn + c];
                if (a.nsplit == 1) NM_ST(&C[(long)m * a.ldc + n], round_out<TO>(s), sp_c, a.status);
                else if (a.cluster_split) cluster_slot_store(slot0, m * a.tn + c, s);
                else               NM_ST(&P[(size_t)m * a.tn + c], s, sp_p, a.status);
            }
        }
    }
    if (a.cluster_split) { cluster_split_finish<TO>(a, s_slots, M, tile, split, h); return; }
    if (a.nsplit > 1) splitk_complete<M, TO>(a, tile, h, &s_last);
}

// ---- column-major B (k contiguous): each warp owns kCols columns, lanes stride along k ------------------
template <int M> struct ColCfg {
    static constexpr int kCols = (M <= 4) ? 4 : 2;                 // columns per warp
    static constexpr int kWarps = kThreads / 32;
    static constexpr int kTile = kCols * kWarps;                   // columns per CTA
};

template <int M, typename TI, typename TO>
__global__ void __launch_bounds__(kThreads, 2) nm_col_kernel(const MatmulArgs a)
{
    using E = Elem<TI>;
    constexpr int V = E::kVec;
    constexpr int CW = ColCfg<M>::kCols;
    constexpr int STEP = 32 * V;                                   // k covered by a warp per load
    // A chunk kept in its storage type: M x KC elements in 32 KB
    constexpr int KC = (((kSmemFloats * 4 / (int)sizeof(TI)) / M) / STEP) * STEP;
    __shared__ __align__(16) float smem[kSmemFloats];
    __shared__ __align__(16) float s_slots[kClusterSlotFloats];
    __shared__ int s_last;
    if (a.cluster_split) cluster_arrive_all();
    pdl_launch_dependents();
    uint4 *As = (uint4 *)smem;                                     // [M][KC / V] 16-byte vectors

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x, split = blockIdx.y, h = blockIdx.z;
    const int col0 = tile * a.tn + warp * CW;
    const int kb = split * a.kr;
    const int ke = min(a.K, kb + a.kr);
    const TI *__restrict__ A = (const TI *)a.A + (long)h * a.strideA;
    const TI *__restrict__ B = (const TI *)a.B + (long)h * a.strideB;
    const long ldb = a.K;
    const Span sp_a = span_of_A<TI>(a), sp_b = span_of_B<TI>(a), sp_c = span_of_C<TO>(a), sp_p = span_of_partials(a);
    (void)sp_a; (void)sp_b; (void)sp_c; (void)sp_p;

    float acc[M][CW];
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int c = 0; c < CW; ++c) acc[m][c] = 0.f;

    for (int kc = kb; kc < ke; kc += KC) {
        const int klen = min(KC, ke - kc);                         // multiple of V
        uint4 b0[CW], b1[CW];
        int kk = lane * V;
        // first two batches of weight loads go out before A is staged
#pragma unroll
        for (int c = 0; c < CW; ++c) {
            const bool okc = col0 + c < a.N;
            const TI *bp = B + (long)(col0 + c) * ldb + kc;
            b0[c] = (okc && kk < klen) ? NM_LD_STREAM16(bp + kk, sp_b, a.status) : make_uint4(0, 0, 0, 0);
            b1[c] = (okc && kk + STEP < klen) ? NM_LD_STREAM16(bp + kk + STEP, sp_b, a.status) : make_uint4(0, 0, 0, 0);
        }
        if (kc == kb) pdl_wait_prior_grids();                      // weights depend on nothing; A and everything written do
        __syncthreads();
        const int nv = klen / V;
        for (int m = 0; m < M; ++m) {
            const uint4 *src = (const uint4 *)(A + (long)m * a.lda + kc);
            for (int i = tid; i < nv; i += kThreads) As[m * (KC / V) + i] = NM_LDG16(src + i, sp_a, a.status);
        }
        __syncthreads();
        for (; kk < klen; kk += 2 * STEP) {
            const bool second = kk + STEP < klen;
            float bf0[CW][V], bf1[CW][V];
#pragma unroll
            for (int c = 0; c < CW; ++c) { E::unpack(b0[c], bf0[c]); E::unpack(b1[c], bf1[c]); }
            // next two batches
            const int kn = kk + 2 * STEP;
#pragma unroll
            for (int c = 0; c < CW; ++c) {
                const bool okc = col0 + c < a.N;
                const TI *bp = B + (long)(col0 + c) * ldb + kc;
                b0[c] = (okc && kn < klen) ? NM_LD_STREAM16(bp + kn, sp_b, a.status) : make_uint4(0, 0, 0, 0);
                b1[c] = (okc && kn + STEP < klen) ? NM_LD_STREAM16(bp + kn + STEP, sp_b, a.status) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int m = 0; m < M; ++m) {
                float af[V];
                E::unpack(As[m * (KC / V) + kk / V], af);
#pragma unroll
                for (int c = 0; c < CW; ++c)
#pragma unroll
                    for (int j = 0; j < V; ++j) acc[m][c] = fmaf(af[j], bf0[c][j], acc[m][c]);
                if (second) {
                    E::unpack(As[m * (KC / V) + (kk + STEP) / V], af);
#pragma unroll
                    for (int c = 0; c < CW; ++c)
#pragma unroll
                        for (int j = 0; j < V; ++j) acc[m][c] = fmaf(af[j], bf1[c][j], acc[m][c]);
                }
            }
        }
    }

    // butterfly over the 32 lanes; lane (m*CW + c) keeps element (m, c)
    float mine = 0.f;
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int c = 0; c < CW; ++c) {
            float s = acc[m][c];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == m * CW + c) mine = s;
        }
    uint32_t slot0 = 0;
    if (a.cluster_split) {
        cluster_wait_all();
        slot0 = cluster_slot_base(s_slots, split, M * a.tn);
    }
    if (lane < M * CW) {
        const int m = lane / CW, c = lane - m * CW, n = col0 + c;
        if (n < a.N) {
            if (a.nsplit == 1) {
                NM_ST(&((TO *)a.C + (long)h * a.strideC)[(long)m * a.ldc + n], round_out<TO>(mine), sp_c, a.status);
            } else if (a.cluster_split) {
                cluster_slot_store(slot0, m * a.tn + warp * CW + c, mine);
            } else {
                float *P = a.partial + (((size_t)h * a.ntiles + tile) * a.nsplit + split) * (size_t)(M * a.tn);
                NM_ST(&P[(size_t)m * a.tn + warp * CW + c], mine, sp_p, a.status);
            }
        }
    }
    if (a.cluster_split) { cluster_split_finish<TO>(a, s_slots, M, tile, split, h); return; }
    if (a.nsplit > 1) splitk_complete<M, TO>(a, tile, h, &s_last);
}

// ---- scalar kernel for shapes the vector paths cannot take (odd N / K, unaligned pointers) ------------------
template <typename TI, typename TO>
__global__ void __launch_bounds__(kThreads) nm_generic_kernel(const MatmulArgs a, int layout)
{
    const int n = blockIdx.x * kThreads + threadIdx.x, h = blockIdx.z;
    if (n >= a.N) return;
    const TI *__restrict__ A = (const TI *)a.A + (long)h * a.strideA;
    const TI *__restrict__ B = (const TI *)a.B + (long)h * a.strideB;
    float acc[NM_MAX_M];
#pragma unroll
    for (int m = 0; m < NM_MAX_M; ++m) acc[m] = 0.f;
    for (int k = 0; k < a.K; ++k) {
        const long ib = (layout == NM_ROW_MAJOR) ? (long)k * a.N + n : (long)n * a.K + k;
        const float b = Elem<TI>::widen(NM_LD(&B[ib], span_of_B<TI>(a), a.status));
#pragma unroll
        for (int m = 0; m < NM_MAX_M; ++m)
            if (m < a.M) acc[m] = fmaf(Elem<TI>::widen(NM_LD(&A[(long)m * a.lda + k], span_of_A<TI>(a), a.status)), b, acc[m]);
    }
    TO *C = (TO *)a.C + (long)h * a.strideC;
#pragma unroll
    for (int m = 0; m < NM_MAX_M; ++m)
        if (m < a.M) NM_ST(&C[(long)m * a.ldc + n], round_out<TO>(acc[m]), span_of_C<TO>(a), a.status);
}

// ---- launch helpers (explicitly instantiated per element type in their own translation units) ------------
#define NM_FOR_EACH_M(X) X(1) X(2) X(3) X(4) X(5) X(6) X(7) X(8) X(9) X(10) X(11) X(12) X(13) X(14) X(15) X(16)

template <typename TI, typename TO>
cudaError_t launch_row(const MatmulArgs &a, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.ntiles, a.nsplit, a.H);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = s;
    // attribute 0: programmatic launch (when asked for); the cluster attribute, when used, comes last so that it can be dropped
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (a.use_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    const int na_plain = na;
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 1; attr[na].val.clusterDim.y = (unsigned)a.nsplit; attr[na].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.cluster_split ? na + 1 : na;
    switch (a.M) {
#define NM_X(m)                                                                                          \
    case m: {                                                                                            \
        auto kern = nm_row_kernel<m, TI, TO>;                                                             \
        MatmulArgs b = a;                                                                                \
        if (b.cluster_split && b.partial && !clusters_fit_one_wave(kern, cfg, (unsigned)b.nsplit, (long)b.ntiles * b.H)) { \
            b.cluster_split = 0;       /* a second wave of clusters: through the workspace instead */      \
            cfg.numAttrs = na_plain;                                                                     \
        }                                                                                                \
        return cudaLaunchKernelEx(&cfg, kern, b);                                                        \
    }
        NM_FOR_EACH_M(NM_X)
#undef NM_X
    default: return cudaErrorInvalidValue;
    }
}

template <typename TI, typename TO>
cudaError_t launch_col(const MatmulArgs &a, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.ntiles, a.nsplit, a.H);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = s;
    // attribute 0: programmatic launch (when asked for); the cluster attribute, when used, comes last so that it can be dropped
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (a.use_pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    const int na_plain = na;
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 1; attr[na].val.clusterDim.y = (unsigned)a.nsplit; attr[na].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.cluster_split ? na + 1 : na;
    switch (a.M) {
#define NM_X(m)                                                                                          \
    case m: {                                                                                            \
        auto kern = nm_col_kernel<m, TI, TO>;                                                             \
        MatmulArgs b = a;                                                                                \
        if (b.cluster_split && b.partial && !clusters_fit_one_wave(kern, cfg, (unsigned)b.nsplit, (long)b.ntiles * b.H)) { \
            b.cluster_split = 0;       /* a second wave of clusters: through the workspace instead */      \
            cfg.numAttrs = na_plain;                                                                     \
        }                                                                                                \
        return cudaLaunchKernelEx(&cfg, kern, b);                                                        \
    }
        NM_FOR_EACH_M(NM_X)
#undef NM_X
    default: return cudaErrorInvalidValue;
    }
}

template <typename TI, typename TO>
cudaError_t launch_generic(const MatmulArgs &a, int layout, cudaStream_t s)
{
    dim3 grid(ceil_div(a.N, kThreads), 1, a.H);
    nm_generic_kernel<TI, TO><<<grid, kThreads, 0, s>>>(a, layout);
    return cudaGetLastError();
}

#define NM_INSTANTIATE(KIND, TI, TO) \
    template cudaError_t launch_##KIND<TI, TO>(const MatmulArgs &, cudaStream_t);
#define NM_EXTERN(KIND, TI, TO) \
    extern template cudaError_t launch_##KIND<TI, TO>(const MatmulArgs &, cudaStream_t);

}  // namespace nm
