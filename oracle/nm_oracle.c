/*
 * CPU oracle for the narrow matrix product and the single-token MLA decode step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * GPU library must compute.  It shares no code, header, table or helper with the
 * CUDA path; only the tests, the smoke check and the bench's CPU-baseline leg may
 * load it.  Everything accumulates in fp64 over exactly-widened inputs, in the
 * order the definition states (k increasing, j increasing), with no blocking or
 * fusion.  OpenMP only spreads independent output elements over threads.
 *
 * What each function follows:
 *   nmo_matmul*        - the problem statement C[MxN] = A[MxK] * B[KxN] (narrow-dimension
 *                        condition; Eq. 4 for the K=7168, N=576 case).
 *   nmo_rmsnorm/rope   - the vector-side consumers of MatMul 2 ("RMS, RoPE and caching
 *                        normalization", MLA Operator Optimization section).
 *   nmo_mla_attention  - absorbed multi-head latent attention over the 576-wide cache rows.
 *   nmo_mla_decode_step- the eleven-stage decode step; Eq. 1-3 give stage 5, the final cast
 *                        to bfloat16 after accumulation (Data Type Issue section) gives the
 *                        rounding point after every matmul.
 *
 * The optional fp16 element type of the product (the paper uses bf16 data; fp16 appears there only as a type pun)
 * follows the same definition with binary16 widening and one binary16 rounding; pinned by all 65536 bit patterns
 * and by roundings (ties, subnormals, overflow) against hand values and numpy's float16.
 *
 * Pins (tests, CPU only): hand-computed 1x3 * 3x2 case in both layouts; brute force
 * against int64 on all shapes <= 4; small-integer exactness at K=7168; rounding ties
 * 257 -> 256 and 259 -> 260; identity / one-hot; closed forms; linearity and the
 * concatenation property of Eq. 3; numpy float64 cross-check; the restated
 * Algorithm 2 index arithmetic; softmax / RoPE / RMSNorm invariants; absorbed ==
 * textbook MLA on a tiny instance; permutation invariance of the cache rows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { NMO_F32 = 0, NMO_BF16 = 1, NMO_F16 = 2, NMO_F64 = 3 };
enum { NMO_ROW_MAJOR = 0, NMO_COL_MAJOR = 1, NMO_FRACTAL_NZ = 2 };

/* ---- exact widening and single-step rounding ------------------------------------- */

static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;   /* bf16 is the upper half of an fp32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* fp64 -> bf16, round to nearest, ties to even, in one step (no fp32 stop on the way). */
static uint16_t f64_to_bf16(double x)
{
    if (isnan(x)) return 0x7fc0;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7f80;
    int e;
    (void)frexp(a, &e);          /* a = f * 2^e with f in [0.5, 1)  ->  floor(log2 a) = e - 1 */
    int p = e - 1;
    if (p < -126) p = -126;      /* subnormal range shares the quantum of the lowest binade */
    double quantum = ldexp(1.0, p - 7);          /* bf16 keeps 7 fraction bits */
    double r = nearbyint(a / quantum) * quantum; /* default rounding mode: ties to even */
    if (r >= ldexp(1.0, 128)) return sign | 0x7f80;
    float f = (float)r;          /* exact: r has at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return sign | (uint16_t)(u >> 16);
}

double nmo_bf16_to_f64(uint16_t b) { return bf16_to_f64(b); }
uint16_t nmo_f64_to_bf16(double x) { return f64_to_bf16(x); }

/* IEEE binary16 (the optional fp16 element type of the product): 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double f16_to_f64(uint16_t h)
{
    int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)f, -24);                       /* zero and subnormals: f * 2^-24 */
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

/* fp64 -> fp16, round to nearest, ties to even, in one step. */
static uint16_t f64_to_f16(double x)
{
    if (isnan(x)) return 0x7e00;
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7c00;
    int e;
    (void)frexp(a, &e);
    int p = e - 1;                                /* floor(log2 a) */
    if (p < -14) p = -14;                         /* subnormals share the quantum of the lowest binade, 2^-24 */
    double quantum = ldexp(1.0, p - 10);          /* fp16 keeps 10 fraction bits */
    double r = nearbyint(a / quantum) * quantum;  /* default rounding mode: ties to even */
    if (r >= 65536.0) return sign | 0x7c00;       /* past the largest finite value (65504) by half a quantum or more */
    if (r < ldexp(1.0, -14)) return sign | (uint16_t)(r / ldexp(1.0, -24));      /* subnormal or zero */
    (void)frexp(r, &e);                           /* rounding may have carried into the next binade */
    p = e - 1;
    double frac = r / ldexp(1.0, p) - 1.0;        /* in [0, 1), a multiple of 2^-10 */
    return sign | (uint16_t)((p + 15) << 10) | (uint16_t)(frac * 1024.0);
}

double nmo_f16_to_f64(uint16_t h) { return f16_to_f64(h); }
uint16_t nmo_f64_to_f16(double x) { return f64_to_f16(x); }

static double load_as_f64(const void *p, long i, int dtype)
{
    switch (dtype) {
    case NMO_F32:  return (double)((const float *)p)[i];
    case NMO_BF16: return bf16_to_f64(((const uint16_t *)p)[i]);
    case NMO_F16:  return f16_to_f64(((const uint16_t *)p)[i]);
    default:       return ((const double *)p)[i];
    }
}

static void store_rounded(void *p, long i, int dtype, double x)
{
    switch (dtype) {
    case NMO_F32:  ((float *)p)[i] = (float)x; break;          /* C cast: RNE */
    case NMO_BF16: ((uint16_t *)p)[i] = f64_to_bf16(x); break;
    case NMO_F16:  ((uint16_t *)p)[i] = f64_to_f16(x); break;
    default:       ((double *)p)[i] = x; break;
    }
}

void nmo_widen(const void *src, double *dst, long n, int dtype)
{
    for (long i = 0; i < n; ++i) dst[i] = load_as_f64(src, i, dtype);
}

void nmo_round(const double *src, void *dst, long n, int dtype)
{
    for (long i = 0; i < n; ++i) store_rounded(dst, i, dtype, src[i]);
}

/* Quantise fp64 values to the bf16 grid but keep them as fp64 ("->bf16, continue from the
 * rounded value"). */
void nmo_quantize_bf16(double *x, long n)
{
    for (long i = 0; i < n; ++i) x[i] = bf16_to_f64(f64_to_bf16(x[i]));
}

/* ---- narrow matrix product: the definition ---------------------------------------- */

/*
 * C[m,n] = sum_k A[m,k] * B[k,n], k increasing, fp64.  A is row-major MxK (element (m,k) at
 * m*lda + k); B element (k,n) sits at k*ldb + n (row-major) or n*ldb + k (column-major, i.e. an
 * [out,in] weight such as W^{DKV} in R^{d_c x d}) or at fractal_nz_index (FRACTAL_NZ; ldb unused); C64 (optional)
 * receives the unrounded sums,
 * C (optional) the sums rounded once to out_dtype, bound (optional) sum_k |a*b|.
 */
/*
 * FRACTAL_NZ, the tiling the paper's weight matrices have in memory (MLA Operator Optimization; figure of the
 * special formats): the K x N matrix is cut into 16 x 16 fractals; the fractals are ordered by columns (all
 * fractals of the first 16 columns from top to bottom, then the next 16 columns), the 256 elements inside a
 * fractal by rows.  K and N are multiples of 16.
 */
static long fractal_nz_index(int k, int n, int K)
{
    return ((long)(n / 16) * (K / 16) + k / 16) * 256 + (long)(k % 16) * 16 + n % 16;
}

void nmo_matmul_strided(const void *A, const void *B, void *C, double *C64, double *bound,
                        int M, int N, int K, long lda, long ldb, long ldc,
                        int in_dtype, int out_dtype, int layout_B, int threads)
{
#ifdef _OPENMP
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
#endif
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            double acc = 0.0, s = 0.0;
            for (int k = 0; k < K; ++k) {
                long ib;
                if (layout_B == NMO_ROW_MAJOR)      ib = (long)k * ldb + n;
                else if (layout_B == NMO_COL_MAJOR) ib = (long)n * ldb + k;
                else                                ib = fractal_nz_index(k, n, K);
                double p = load_as_f64(A, (long)m * lda + k, in_dtype) * load_as_f64(B, ib, in_dtype);
                acc += p;
                s += fabs(p);
            }
            long ic = (long)m * ldc + n;
            if (C)     store_rounded(C, ic, out_dtype, acc);
            if (C64)   C64[ic] = acc;
            if (bound) bound[ic] = s;
        }
    }
}

void nmo_matmul(const void *A, const void *B, void *C, double *C64, double *bound,
                int M, int N, int K, int in_dtype, int out_dtype, int layout_B, int threads)
{
    long ldb = (layout_B == NMO_ROW_MAJOR) ? N : K;
    nmo_matmul_strided(A, B, C, C64, bound, M, N, K, K, ldb, N, in_dtype, out_dtype, layout_B, threads);
}

/*
 * H independent products.  A(m,h,k) at m*lda + h*strideA + k; B_h at B + h*strideB, dense
 * KxN in the given layout; C(m,h,n) at m*ldc + h*strideC + n.  bound / C64 use the C indexing.
 */
void nmo_matmul_batched(const void *A, const void *B, void *C, double *C64, double *bound,
                        int M, int N, int K, int H, long lda, long strideA, long strideB,
                        long ldc, long strideC, int in_dtype, int out_dtype, int layout_B, int threads)
{
    size_t esz_in = (in_dtype == NMO_F32) ? 4 : ((in_dtype == NMO_BF16 || in_dtype == NMO_F16) ? 2 : 8);
    size_t esz_out = (out_dtype == NMO_F32) ? 4 : ((out_dtype == NMO_BF16 || out_dtype == NMO_F16) ? 2 : 8);
    long ldb = (layout_B == NMO_ROW_MAJOR) ? N : K;
    for (int h = 0; h < H; ++h) {
        const char *Ah = (const char *)A + (size_t)h * strideA * esz_in;
        const char *Bh = (const char *)B + (size_t)h * strideB * esz_in;
        char *Ch = C ? (char *)C + (size_t)h * strideC * esz_out : NULL;
        nmo_matmul_strided(Ah, Bh, Ch, C64 ? C64 + (size_t)h * strideC : NULL,
                           bound ? bound + (size_t)h * strideC : NULL,
                           M, N, K, lda, ldb, ldc, in_dtype, out_dtype, layout_B, threads);
    }
}

/* ---- vector-side stages of the decode step (fp64 in, fp64 out, no rounding inside) ---- */

/* y[i] = x[i] * rsqrt(mean(x^2) + eps) * gamma[i] */
void nmo_rmsnorm(const double *x, const double *gamma, double *y, int n, double eps)
{
    double ss = 0.0;
    for (int i = 0; i < n; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / (double)n + eps);
    for (int i = 0; i < n; ++i) y[i] = x[i] * r * gamma[i];
}

/* Interleaved-pair rotary embedding: pair (x[2i], x[2i+1]) turns by pos * base^(-2i/dim). */
void nmo_rope(const double *x, double *y, int dim, long pos, double base)
{
    for (int i = 0; i < dim / 2; ++i) {
        double ang = (double)pos * pow(base, -2.0 * (double)i / (double)dim);
        double c = cos(ang), s = sin(ang);
        double x0 = x[2 * i], x1 = x[2 * i + 1];
        y[2 * i]     = x0 * c - x1 * s;
        y[2 * i + 1] = x0 * s + x1 * c;
    }
}

/*
 * Absorbed latent attention for all heads over cache rows 0..S-1.
 * Q: H x dqk (per head: [q_lat(dv) | q_rope(dqk-dv)]); cache: S x dqk (per row: [c_kv(dv) | k_rope]).
 *   s[h,j] = scale * sum_{c<dqk} Q[h,c] * cache[j,c]
 *   p[h,:] = softmax_j(s[h,:])  (row max subtracted)
 *   o[h,c] = sum_j p[h,j] * cache[j,c],  c < dv
 * P (optional, H x S) receives the probabilities.
 */
void nmo_mla_attention(const double *Q, const double *cache, double *O, double *P,
                       int H, int S, int dqk, int dv, double scale, int threads)
{
#ifdef _OPENMP
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
#endif
    for (int h = 0; h < H; ++h) {
        double *s = (double *)malloc(sizeof(double) * (size_t)S);
        double mx = -INFINITY;
        for (int j = 0; j < S; ++j) {
            double acc = 0.0;
            for (int c = 0; c < dqk; ++c) acc += Q[(long)h * dqk + c] * cache[(long)j * dqk + c];
            s[j] = acc * scale;
            if (s[j] > mx) mx = s[j];
        }
        double l = 0.0;
        for (int j = 0; j < S; ++j) { s[j] = exp(s[j] - mx); l += s[j]; }
        for (int j = 0; j < S; ++j) s[j] /= l;
        if (P) for (int j = 0; j < S; ++j) P[(long)h * S + j] = s[j];
        for (int c = 0; c < dv; ++c) {
            double acc = 0.0;
            for (int j = 0; j < S; ++j) acc += s[j] * cache[(long)j * dqk + c];
            O[(long)h * dv + c] = acc;
        }
        free(s);
    }
}

/* ---- the decode step ---------------------------------------------------------------- */

typedef struct {
    /* dimensions */
    int d, q_lora, kv_lora, rope, nope, v, H;
    int seq_len;          /* rows attended, including the row this step writes (pos = seq_len-1) */
    int layout_dense;     /* layout of W_DQ, W_UQR, W_DKVKR, W_O (per-head weights are row-major) */
    int threads;
    double rms_eps, softmax_scale, rope_base;
    /* bf16 inputs */
    const uint16_t *h, *W_DQ, *gamma_q, *W_UQR, *W_DKVKR, *gamma_kv, *W_UK, *W_UV, *W_O; /* W_O may be NULL */
    uint16_t *kv_cache;   /* [>=seq_len][kv_lora+rope]; row seq_len-1 is written */
    /* bf16 outputs, every stage (each may be NULL) */
    uint16_t *c_q, *c_qn, *q, *q_rope, *ckr, *q_lat, *o_lat, *o, *out;
    /* fp64 extras (each may be NULL): unrounded attention output and matmul bounds */
    double *o_lat_f64, *bound_c_q, *bound_q, *bound_ckr, *bound_q_lat, *bound_o, *bound_out;
} nmo_mla_params;

static double *dalloc(size_t n) { return (double *)calloc(n ? n : 1, sizeof(double)); }
static void put_bf16(uint16_t *dst, const double *src, long n) { if (dst) for (long i = 0; i < n; ++i) dst[i] = f64_to_bf16(src[i]); }

int nmo_mla_decode_step(const nmo_mla_params *p)
{
    const int d = p->d, ql = p->q_lora, dc = p->kv_lora, dr = p->rope, dn = p->nope, dv = p->v, H = p->H;
    const int dq = dn + dr, dkv = dc + dr, S = p->seq_len, T = p->threads, L = p->layout_dense;
    const long pos = (long)S - 1;
    if (S < 1) return -1;

    /* 1. c_q = h * W_DQ  -> bf16 */
    double *c_q = dalloc(ql);
    nmo_matmul(p->h, p->W_DQ, NULL, c_q, p->bound_c_q, 1, ql, d, NMO_BF16, NMO_F64, L, T);
    nmo_quantize_bf16(c_q, ql);  put_bf16(p->c_q, c_q, ql);

    /* 2. c_qn = RMSNorm(c_q; gamma_q) -> bf16 */
    double *gq = dalloc(ql), *c_qn = dalloc(ql);
    nmo_widen(p->gamma_q, gq, ql, NMO_BF16);
    nmo_rmsnorm(c_q, gq, c_qn, ql, p->rms_eps);
    nmo_quantize_bf16(c_qn, ql);  put_bf16(p->c_qn, c_qn, ql);

    /* 3. q = c_qn * W_UQR -> bf16, per head [nope | rope] */
    double *q = dalloc((size_t)H * dq);
    {
        uint16_t *c_qn_b = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)ql);
        for (int i = 0; i < ql; ++i) c_qn_b[i] = f64_to_bf16(c_qn[i]);
        nmo_matmul(c_qn_b, p->W_UQR, NULL, q, p->bound_q, 1, H * dq, ql, NMO_BF16, NMO_F64, L, T);
        free(c_qn_b);
    }
    nmo_quantize_bf16(q, (long)H * dq);  put_bf16(p->q, q, (long)H * dq);

    /* 4. q_rope[h] = RoPE(q[h, nope:], pos) -> bf16 */
    double *q_rope = dalloc((size_t)H * dr);
    for (int h = 0; h < H; ++h) nmo_rope(q + (long)h * dq + dn, q_rope + (long)h * dr, dr, pos, p->rope_base);
    nmo_quantize_bf16(q_rope, (long)H * dr);  put_bf16(p->q_rope, q_rope, (long)H * dr);

    /* 5. ckr = h * (W_DKV | W_KR) -> bf16   (Eq. 3: one product for both projections) */
    double *ckr = dalloc(dkv);
    nmo_matmul(p->h, p->W_DKVKR, NULL, ckr, p->bound_ckr, 1, dkv, d, NMO_BF16, NMO_F64, L, T);
    nmo_quantize_bf16(ckr, dkv);  put_bf16(p->ckr, ckr, dkv);

    /* 6. cache[pos] = [ RMSNorm(ckr[:dc]; gamma_kv) -> bf16 | RoPE(ckr[dc:], pos) -> bf16 ] */
    double *gkv = dalloc(dc), *row = dalloc(dkv);
    nmo_widen(p->gamma_kv, gkv, dc, NMO_BF16);
    nmo_rmsnorm(ckr, gkv, row, dc, p->rms_eps);
    nmo_rope(ckr + dc, row + dc, dr, pos, p->rope_base);
    for (int i = 0; i < dkv; ++i) p->kv_cache[pos * dkv + i] = f64_to_bf16(row[i]);

    /* 7. q_lat[h] = q_nope[h] * W_UK[h] -> bf16   (W_UK[h]: nope x dc, row-major) */
    double *q_lat = dalloc((size_t)H * dc);
    {
        uint16_t *q_b = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)H * dq);
        for (long i = 0; i < (long)H * dq; ++i) q_b[i] = f64_to_bf16(q[i]);
        nmo_matmul_batched(q_b, p->W_UK, NULL, q_lat, p->bound_q_lat, 1, dc, dn, H,
                           (long)H * dq, dq, (long)dn * dc, (long)H * dc, dc,
                           NMO_BF16, NMO_F64, NMO_ROW_MAJOR, T);
        free(q_b);
    }
    nmo_quantize_bf16(q_lat, (long)H * dc);  put_bf16(p->q_lat, q_lat, (long)H * dc);

    /* 8-9. scores, softmax, o_lat over rows 0..S-1 (the row written in 6 included) */
    double *Q = dalloc((size_t)H * dkv), *cache = dalloc((size_t)S * dkv), *o_lat = dalloc((size_t)H * dc);
    for (int h = 0; h < H; ++h) {
        memcpy(Q + (long)h * dkv, q_lat + (long)h * dc, sizeof(double) * (size_t)dc);
        memcpy(Q + (long)h * dkv + dc, q_rope + (long)h * dr, sizeof(double) * (size_t)dr);
    }
    nmo_widen(p->kv_cache, cache, (long)S * dkv, NMO_BF16);
    nmo_mla_attention(Q, cache, o_lat, NULL, H, S, dkv, dc, p->softmax_scale, T);
    if (p->o_lat_f64) memcpy(p->o_lat_f64, o_lat, sizeof(double) * (size_t)H * dc);
    nmo_quantize_bf16(o_lat, (long)H * dc);  put_bf16(p->o_lat, o_lat, (long)H * dc);

    /* 10. o[h] = o_lat[h] * W_UV[h] -> bf16   (W_UV[h]: dc x v, row-major) */
    double *o = dalloc((size_t)H * dv);
    uint16_t *o_b = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)H * dv);
    {
        uint16_t *ol_b = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)H * dc);
        for (long i = 0; i < (long)H * dc; ++i) ol_b[i] = f64_to_bf16(o_lat[i]);
        nmo_matmul_batched(ol_b, p->W_UV, NULL, o, p->bound_o, 1, dv, dc, H,
                           (long)H * dc, dc, (long)dc * dv, (long)H * dv, dv,
                           NMO_BF16, NMO_F64, NMO_ROW_MAJOR, T);
        free(ol_b);
    }
    nmo_quantize_bf16(o, (long)H * dv);  put_bf16(p->o, o, (long)H * dv);
    for (long i = 0; i < (long)H * dv; ++i) o_b[i] = f64_to_bf16(o[i]);

    /* 11. out = flatten(o) * W_O -> bf16   (skipped when W_O is NULL) */
    if (p->W_O) {
        double *out = dalloc(d);
        nmo_matmul(o_b, p->W_O, NULL, out, p->bound_out, 1, d, H * dv, NMO_BF16, NMO_F64, L, T);
        put_bf16(p->out, out, d);
        free(out);
    }

    free(o_b); free(o); free(o_lat); free(cache); free(Q); free(q_lat); free(row); free(gkv);
    free(ckr); free(q_rope); free(q); free(c_qn); free(gq); free(c_q);
    return 0;
}

int nmo_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
