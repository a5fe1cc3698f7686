"""Pins for the CPU oracle: each test ties it to something other than itself (hand-computed
values, exact integer arithmetic, closed forms, invariants, a library routine, the restated
Algorithm 2), chosen so that a dropped term, a wrong index or a transposed operand fails one."""
import itertools
import math
import os

import numpy as np
import pytest

import nm_inputs as gen
import oracle
from oracle import BF16, COL_MAJOR, F16, F32, F64, ROW_MAJOR, alg2

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = [float(x) for x in v]
    return out


def _bits(x):
    """float array of bf16-representable values -> bf16 bit patterns (checked exact)."""
    x = np.asarray(x, dtype=np.float32)
    b = (x.view(np.uint32) >> 16).astype(np.uint16)
    assert np.all((x.view(np.uint32) & 0xFFFF) == 0), "value not representable in bf16"
    return b


# ---- P1: hand-computed case, both layouts ------------------------------------------------------

@pytest.mark.parametrize("dtype", [F32, BF16])
def test_hand_computed_case_both_layouts(dtype):
    g = _read_golden("matmul_1x3_3x2.txt")
    M, N, K = int(g["M"][0]), int(g["N"][0]), int(g["K"][0])
    conv = (lambda v: np.asarray(v, np.float32)) if dtype == F32 else _bits
    A = conv(g["A"])
    for key, layout in (("B_row_major", ROW_MAJOR), ("B_col_major", COL_MAJOR)):
        Cq, C64, bound = oracle.matmul(A, conv(g[key]), M, N, K, dtype, F32, layout)
        assert C64.ravel().tolist() == g["C"]
        assert Cq.ravel().tolist() == g["C"]
        assert bound.ravel().tolist() == g["C"]          # all terms positive: bound equals the sum


# ---- P2: brute force against exact integer arithmetic on every tiny shape --------------------------

def test_brute_force_tiny_shapes_int64():
    rng = np.random.default_rng(7)
    vals = np.array([-1, 0, 1, 2])
    for M, N, K in itertools.product(range(1, 5), repeat=3):
        Ai = rng.choice(vals, size=(M, K))
        Bi = rng.choice(vals, size=(K, N))
        Ci = np.zeros((M, N), dtype=np.int64)
        Si = np.zeros((M, N), dtype=np.int64)
        for m in range(M):
            for n in range(N):
                for k in range(K):
                    Ci[m, n] += int(Ai[m, k]) * int(Bi[k, n])
                    Si[m, n] += abs(int(Ai[m, k]) * int(Bi[k, n]))
        for layout in (ROW_MAJOR, COL_MAJOR):
            Bst = Bi if layout == ROW_MAJOR else Bi.T
            for dt, conv in ((F32, lambda v: np.ascontiguousarray(v, np.float32)),
                             (BF16, lambda v: _bits(np.ascontiguousarray(v, np.float32)))):
                Cq, C64, bound = oracle.matmul(conv(Ai), conv(Bst), M, N, K, dt, F32, layout)
                assert np.array_equal(C64, Ci.astype(np.float64)), (M, N, K, layout, dt)
                assert np.array_equal(Cq, Ci.astype(np.float32))
                assert np.array_equal(bound, Si.astype(np.float64))


# ---- P3: small integers at the real K: fp64, int64 agree exactly ---------------------------------

@pytest.mark.parametrize("layout", [ROW_MAJOR, COL_MAJOR])
def test_small_integer_exactness_full_k(layout):
    M, K, N = 3, 7168, 40
    A = gen.small_int_bf16((M, K), -8, 8, seed=11)
    B = gen.small_int_bf16((K, N), -8, 8, seed=12)
    Ai = gen.bits_to_f32(A).astype(np.int64)
    Bi = gen.bits_to_f32(B).astype(np.int64)
    Ci = Ai @ Bi                                           # exact integer product
    assert np.abs(Ci).max() < 2 ** 24
    Bst = B if layout == ROW_MAJOR else gen.to_col_major(B)
    Cq, C64, _ = oracle.matmul(A, Bst, M, N, K, BF16, F32, layout)
    assert np.array_equal(C64, Ci.astype(np.float64))
    assert np.array_equal(Cq, Ci.astype(np.float32))


# ---- P4: rounding ties of the final cast to bf16 -------------------------------------------------

def test_rounding_ties_to_even():
    with open(os.path.join(GOLDEN, "rounding_ties.txt")) as f:
        rows = [tuple(float(x) for x in l.split()) for l in f if l.strip() and not l.startswith("#")]
    for total, expect in rows:
        # a column of ones and one remainder, summing to exactly `total`
        K = 64
        A = _bits(np.ones((1, K), np.float32))
        col = np.full(K, np.sign(total) * 4.0, np.float32)
        col[0] = total - np.sign(total) * 4.0 * (K - 1)
        Cq, C64, _ = oracle.matmul(A, _bits(col.reshape(K, 1)), 1, 1, K, BF16, BF16)
        assert C64[0, 0] == total
        assert gen.bits_to_f32(Cq)[0, 0] == expect, (total, expect)
    # direct conversions, including a value that double rounding through fp32 would get wrong:
    # 1 + 2^-8 + 2^-40 lies just above the tie between 1 and 1+2^-7, so the bf16 result is 1+2^-7;
    # rounding to fp32 first gives exactly the tie, which ties-to-even would send down to 1.
    x = 1.0 + 2.0 ** -8 + 2.0 ** -40
    assert gen.bits_to_f32(oracle.f64_to_bf16(np.array([x])))[0] == np.float32(1.0 + 2.0 ** -7)
    assert gen.bits_to_f32(oracle.f64_to_bf16(np.array([1.0 + 2.0 ** -8])))[0] == np.float32(1.0)
    assert gen.bits_to_f32(oracle.f64_to_bf16(np.array([1.0 + 3 * 2.0 ** -8])))[0] == np.float32(1.0 + 2.0 ** -6)


def test_bf16_widening_is_the_upper_half_of_fp32():
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 0x7F80, size=4096, dtype=np.uint16)       # finite positive patterns
    bits[::2] |= 0x8000
    assert np.array_equal(oracle.bf16_to_f64(bits), gen.bits_to_f32(bits).astype(np.float64))
    assert np.array_equal(oracle.f64_to_bf16(oracle.bf16_to_f64(bits)), bits)  # grid points are fixed


# ---- the optional fp16 element type: binary16 widening and rounding ------------------------------

def test_fp16_widening_of_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.f16_to_f64(bits)
    want = bits.view(np.float16).astype(np.float64)                   # numpy's binary16
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))      # -0 stays -0
    # hand values: 0x3c00 = 1, 0x0001 = 2^-24 (smallest subnormal), 0x0400 = 2^-14 (smallest normal),
    # 0x7bff = 65504 (largest finite), 0xc000 = -2
    hand = {0x3C00: 1.0, 0x0001: 2.0 ** -24, 0x0400: 2.0 ** -14, 0x7BFF: 65504.0, 0xC000: -2.0, 0x3555: 0.333251953125}
    for b, v in hand.items():
        assert oracle.f16_to_f64(np.array([b], np.uint16))[0] == v
    # grid points are fixed points of the rounding
    finite = bits[~nan & ~np.isinf(want)]
    assert np.array_equal(oracle.f64_to_f16(oracle.f16_to_f64(finite)), finite)


def test_fp16_rounding_is_one_step_to_nearest_even():
    f16 = lambda x: oracle.f64_to_f16(np.array([x], np.float64))[0]
    # ties at 1: 1 + 2^-11 is halfway between 1 and 1 + 2^-10 -> even (1); 1 + 3 * 2^-11 -> 1 + 2^-9
    assert f16(1.0 + 2.0 ** -11) == 0x3C00
    assert f16(1.0 + 3 * 2.0 ** -11) == 0x3C02
    assert f16(1.0 + 2.0 ** -11 + 2.0 ** -40) == 0x3C01               # just above the tie: up (an fp32 stop would tie down)
    # overflow: 65504 is the largest finite value; 65520 is the tie to 2^16 and goes to infinity, 65519.99 does not
    assert f16(65504.0) == 0x7BFF and f16(65519.99) == 0x7BFF and f16(65520.0) == 0x7C00 and f16(-1e6) == 0xFC00
    # subnormals: quantum 2^-24; 1.5 * 2^-24 ties to even (2 * 2^-24), 0.5 * 2^-24 ties to zero, 0.51 * 2^-24 -> 2^-24
    assert f16(1.5 * 2.0 ** -24) == 0x0002 and f16(0.5 * 2.0 ** -24) == 0x0000 and f16(0.51 * 2.0 ** -24) == 0x0001
    assert f16(2.0 ** -14 - 2.0 ** -26) == 0x0400                      # rounds up into the first normal binade
    assert f16(-0.0) == 0x8000
    # against numpy's float64 -> float16 cast on random values across the range (subnormal, normal, near overflow)
    rng = np.random.default_rng(21)
    x = np.concatenate([rng.standard_normal(20000), rng.standard_normal(20000) * 1e-6, rng.standard_normal(20000) * 2e4,
                        rng.uniform(-7e-5, 7e-5, 20000)])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    assert np.array_equal(oracle.f64_to_f16(x), want)


def test_fp16_product_brute_force_and_one_rounding():
    # exact integer arithmetic on tiny shapes, fp16 storage
    rng = np.random.default_rng(8)
    to16 = lambda v: np.ascontiguousarray(v, np.float16).view(np.uint16)
    for M, N, K in itertools.product(range(1, 4), repeat=3):
        Ai = rng.integers(-3, 4, size=(M, K)); Bi = rng.integers(-3, 4, size=(K, N))
        Ci = np.zeros((M, N), dtype=np.int64)
        for m in range(M):
            for n in range(N):
                for k in range(K):
                    Ci[m, n] += int(Ai[m, k]) * int(Bi[k, n])
        for layout in (ROW_MAJOR, COL_MAJOR):
            Bst = Bi if layout == ROW_MAJOR else Bi.T
            Cq, C64, _ = oracle.matmul(to16(Ai), to16(Bst), M, N, K, F16, F16, layout)
            assert np.array_equal(C64, Ci.astype(np.float64))
            assert np.array_equal(Cq.view(np.float16).astype(np.int64), Ci)
    # a sum that is exact in fp64 and a tie in fp16: 2048 + 1 -> 2048 (even), 2048 + 3 -> 2052
    K = 4
    A = to16(np.ones((1, K)))
    for last, expect in ((1.0, 2048.0), (3.0, 2052.0)):
        col = np.array([1024.0, 512.0, 512.0, last]).reshape(K, 1)
        Cq, C64, _ = oracle.matmul(A, to16(col), 1, 1, K, F16, F16)
        assert C64[0, 0] == 2048.0 + last and float(Cq.view(np.float16)[0, 0]) == expect
    # random fp16 data against numpy in float64 (a library product), then one rounding
    A16, B16 = gen.narrow_f16(3, 300, 17, seed=77)
    Cq, C64, bound = oracle.matmul(A16, B16, 3, 17, 300, F16, F16)
    ref = A16.view(np.float16).astype(np.float64) @ B16.view(np.float16).astype(np.float64)
    assert np.allclose(C64, ref, rtol=0, atol=1e-12 * np.abs(bound).max())
    assert np.array_equal(Cq, oracle.f64_to_f16(C64))


# ---- P5: identity / one-hot -------------------------------------------------------------------

@pytest.mark.parametrize("layout", [ROW_MAJOR, COL_MAJOR])
def test_identity_and_one_hot(layout):
    M, K, N = 4, 37, 23
    A = gen.normal_bf16((M, K), 1.0, seed=21)
    B = gen.normal_bf16((K, N), 0.02, seed=22)
    st = (lambda X: X) if layout == ROW_MAJOR else gen.to_col_major
    eye = _bits(np.eye(K, dtype=np.float32))
    Cq, _, _ = oracle.matmul(A, st(eye), M, K, K, BF16, BF16, layout)
    assert np.array_equal(Cq, A)                                       # B = I  ->  C = A
    for k in (0, 5, K - 1):
        e = np.zeros((1, K), np.float32); e[0, k] = 1.0
        Cq, _, _ = oracle.matmul(_bits(e), st(B), 1, N, K, BF16, BF16, layout)
        assert np.array_equal(Cq[0], B[k])                             # A = e_k -> row k of B
    Bsel = np.zeros((K, N), np.float32)
    ks = [(3 * n + 1) % K for n in range(N)]
    for n, k in enumerate(ks):
        Bsel[k, n] = 1.0
    Cq, _, _ = oracle.matmul(A, st(_bits(Bsel)), M, N, K, BF16, BF16, layout)
    assert np.array_equal(Cq, A[:, ks])                                # column n = e_k -> A[:, k]


# ---- P5b: FRACTAL_NZ storage (the layout the paper's weight matrices have in memory) ---------------

def _fractal_nz_by_loops(B):
    """16 x 16 fractals, fractal columns one after the other (within one, the fractals from top to bottom), rows of a
    fractal one after the other - written out with loops, independently of the oracle's index formula and of
    the generator module's reshape."""
    K, N = B.shape
    out = []
    for nb in range(N // 16):
        for kb in range(K // 16):
            for kr in range(16):
                for nc in range(16):
                    out.append(B[kb * 16 + kr, nb * 16 + nc])
    return np.array(out, dtype=B.dtype)


def test_fractal_nz_storage():
    M, K, N = 3, 48, 32
    A = gen.normal_bf16((M, K), 1.0, seed=61)
    B = gen.normal_bf16((K, N), 0.02, seed=62)
    Bnz = _fractal_nz_by_loops(B)
    assert np.array_equal(Bnz, gen.to_fractal_nz(B))                   # the generator's permutation is the same storage
    # first fractal = rows 0-15 x columns 0-15 row by row; second = rows 16-31 of the SAME 16 columns
    assert np.array_equal(Bnz[:16], B[0, :16]) and np.array_equal(Bnz[16:32], B[1, :16])
    assert np.array_equal(Bnz[256:272], B[16, :16]) and np.array_equal(Bnz[3 * 256:3 * 256 + 16], B[0, 16:32])
    Cq, C64, bound = oracle.matmul(A, Bnz, M, N, K, BF16, F32, oracle.FRACTAL_NZ)
    Cq_r, C64_r, bound_r = oracle.matmul(A, B, M, N, K, BF16, F32, ROW_MAJOR)
    assert np.array_equal(C64, C64_r) and np.array_equal(bound, bound_r)   # same products in the same order
    for k in (0, 17, K - 1):                                            # A = e_k -> row k of B, exactly
        e = np.zeros((1, K), np.float32); e[0, k] = 1.0
        Cq, _, _ = oracle.matmul(_bits(e), Bnz, 1, N, K, BF16, BF16, oracle.FRACTAL_NZ)
        assert np.array_equal(Cq[0], B[k])
    ref = gen.bits_to_f32(A).astype(np.float64) @ gen.bits_to_f32(B).astype(np.float64)
    assert np.all(np.abs(C64 - ref) <= 1e-12 * bound)                   # numpy on the logical matrix


# ---- P6: closed forms ---------------------------------------------------------------------------

@pytest.mark.parametrize("layout", [ROW_MAJOR, COL_MAJOR])
def test_closed_forms(layout):
    K, N = 301, 19
    A = np.ones((1, K), np.float32)
    Bn = np.tile(np.arange(1, N + 1, dtype=np.float32), (K, 1))       # B[k,n] = n+1
    Bk = np.tile(np.arange(K, dtype=np.float32).reshape(K, 1), (1, N))  # B[k,n] = k
    st = (lambda X: X) if layout == ROW_MAJOR else (lambda X: np.ascontiguousarray(X.T))
    _, C64, _ = oracle.matmul(A, st(Bn), 1, N, K, F32, F32, layout)
    assert np.array_equal(C64[0], K * np.arange(1, N + 1, dtype=np.float64))
    _, C64, _ = oracle.matmul(A, st(Bk), 1, N, K, F32, F32, layout)
    assert np.array_equal(C64[0], np.full(N, K * (K - 1) / 2))


# ---- P7: Algorithm 2 restated: constants, coverage, agreement with the definition ----------------

def test_alg2_constants_match_hand_derivation():
    g = _read_golden("alg2_constants.txt")
    c = alg2.tiling(int(g["K"][0]), int(g["N"][0]), int(g["P"][0]))
    for k in ("kParts", "fractalNum", "S", "V", "nPartW", "groupSize"):
        assert c[k] == int(g[k][0]), k


def test_alg2_covers_every_block_once_and_equals_definition():
    K, N = 7168, 576
    c = alg2.tiling(K, N, 24)
    k_part, col_block, loaded_k_part = alg2.block_of_work_item(c)
    # every (k part, column block) pair is produced exactly once ...
    pairs = k_part * c["fractalNum"] + col_block
    assert np.array_equal(np.sort(pairs), np.arange(c["S"]))
    assert k_part.max() == c["kParts"] - 1 and col_block.max() == c["fractalNum"] - 1
    # ... by an executor that holds the token slice of that very k part
    assert np.array_equal(k_part, loaded_k_part)
    T = gen.normal_bf16((1, K), 1.0, seed=1000)
    W = gen.normal_bf16((K, N), 0.02, seed=1001)
    Cb, partials = alg2.split_k_product(T, W, K, N)
    assert partials.shape == (c["kParts"], N) and partials.dtype == np.float32
    Cq, C64, bound = oracle.matmul(T, W, 1, N, K, BF16, BF16)
    err = np.abs(gen.bits_to_f32(Cb).astype(np.float64) - C64[0])
    assert np.all(err <= 1e-5 * bound[0] + 1e-6 + oracle.ulp_bf16(C64[0]))
    # the partial sums are those of the k parts: part i against the definition on rows i*1024 ... (i+1)*1024
    Tf, Wf = gen.bits_to_f32(T).astype(np.float64).reshape(K), gen.bits_to_f32(W).astype(np.float64).reshape(K, N)
    for i in (0, 3, 6):
        want = Tf[i * 1024:(i + 1) * 1024] @ Wf[i * 1024:(i + 1) * 1024]
        assert np.allclose(partials[i], want, rtol=0, atol=1e-4)
    # small integers: every summation order is exact, so the two must agree bit for bit
    Ti = gen.small_int_bf16((1, K), -8, 8, seed=31)
    Wi = gen.small_int_bf16((K, N), -8, 8, seed=32)
    Cb, _ = alg2.split_k_product(Ti, Wi, K, N)
    Cq, _, _ = oracle.matmul(Ti, Wi, 1, N, K, BF16, BF16)
    assert np.array_equal(Cb, Cq[0])


# ---- P8: linearity and the concatenation property of the fused product ------------------------------

def test_linearity_and_concatenation():
    M, K, N1, N2 = 2, 257, 33, 9
    rng = np.random.default_rng(5)
    A1, A2 = rng.standard_normal((M, K)), rng.standard_normal((M, K))
    B1, B2 = rng.standard_normal((K, N1)), rng.standard_normal((K, N2))
    f = lambda A, B: oracle.matmul(A, B, M, B.shape[1], K, F64, F64)
    _, C1, b1 = f(A1, B1)
    _, C2, _ = f(A2, B1)
    _, C12, _ = f(2 * A1 + A2, B1)
    assert np.all(np.abs(C12 - (2 * C1 + C2)) <= 1e-12 * (1 + 3 * b1))
    # (B1 | B2): one product over the concatenation equals the two separate ones (Eq. 3)
    _, Ccat, _ = f(A1, np.concatenate([B1, B2], axis=1))
    _, C1b, _ = f(A1, B2)
    assert np.array_equal(Ccat[:, :N1], C1) and np.array_equal(Ccat[:, N1:], C1b)


# ---- P9: library cross-check ----------------------------------------------------------------------

@pytest.mark.parametrize("layout", [ROW_MAJOR, COL_MAJOR])
def test_numpy_float64_cross_check(layout):
    M, K, N = 5, 1031, 67
    A = gen.normal_bf16((M, K), 1.0, seed=41)
    B = gen.normal_bf16((K, N), 0.02, seed=42)
    ref = gen.bits_to_f32(A).astype(np.float64) @ gen.bits_to_f32(B).astype(np.float64)
    refb = np.abs(gen.bits_to_f32(A).astype(np.float64)) @ np.abs(gen.bits_to_f32(B).astype(np.float64))
    Bst = B if layout == ROW_MAJOR else gen.to_col_major(B)
    _, C64, bound = oracle.matmul(A, Bst, M, N, K, BF16, F32, layout, threads=2)
    assert np.all(np.abs(C64 - ref) <= 1e-12 * refb)
    assert np.allclose(bound, refb, rtol=1e-12)
    # sampled-column evaluation is the same function
    cols = [0, 13, N - 1]
    _, Cs, bs = oracle.matmul_columns(A, Bst, M, N, K, cols, BF16, F32, layout)
    assert np.array_equal(Cs, C64[:, cols]) and np.array_equal(bs, bound[:, cols])


def test_batched_strided_addressing():
    T, H, K, N = 3, 4, 16, 24
    q = gen.normal_bf16((T, H, K + 8), 1.0, seed=51)         # q_nope read in place from [T,H,K+8]
    W = gen.normal_bf16((H, K, N), 0.02, seed=52)
    Cq, C64, _ = oracle.matmul_batched(q, W, T, N, K, H, H * (K + 8), K + 8, K * N, H * N, N,
                                       T * H * N, BF16, BF16)
    qf, Wf = gen.bits_to_f32(q).astype(np.float64), gen.bits_to_f32(W).astype(np.float64)
    ref = np.einsum("thk,hkn->thn", qf[:, :, :K], Wf)
    assert np.allclose(C64.reshape(T, H, N), ref, rtol=0, atol=1e-12)


# ---- P10: invariants of the vector-side stages and of attention -----------------------------------

def test_rmsnorm_invariants():
    rng = np.random.default_rng(9)
    x = rng.standard_normal(512)
    y = oracle.rmsnorm(x, np.ones(512), 0.0)
    assert abs(np.sqrt(np.mean(y * y)) - 1.0) < 1e-12                   # unit RMS for gamma = 1
    assert np.allclose(oracle.rmsnorm(7.5 * x, np.ones(512), 0.0), y, atol=1e-12)  # scale invariance
    g = rng.standard_normal(512)
    assert np.allclose(oracle.rmsnorm(x, g, 0.0), y * g, atol=1e-12)
    # eps enters under the root, added to the mean square
    assert np.allclose(oracle.rmsnorm(x, np.ones(512), 0.25), x / np.sqrt(np.mean(x * x) + 0.25), atol=1e-12)


def test_rope_invariants():
    rng = np.random.default_rng(10)
    q, k = rng.standard_normal(64), rng.standard_normal(64)
    assert np.array_equal(oracle.rope(q, 0), q)                         # pos 0 is the identity
    y = oracle.rope(q, 1234)
    assert np.allclose(y[0::2] ** 2 + y[1::2] ** 2, q[0::2] ** 2 + q[1::2] ** 2, atol=1e-12)
    d1 = oracle.rope(q, 17) @ oracle.rope(k, 5)
    d2 = oracle.rope(q, 1017) @ oracle.rope(k, 1005)
    assert abs(d1 - d2) < 1e-9                                          # depends on m - n only
    # first pair turns by pos radians (frequency base^0 = 1), last pair by pos * base^(-62/64)
    e = np.zeros(64); e[0] = 1.0
    y = oracle.rope(e, 2)
    assert np.allclose(y[:2], [np.cos(2.0), np.sin(2.0)], atol=1e-15)
    e = np.zeros(64); e[62] = 1.0
    ang = 3 * 10000.0 ** (-62 / 64)
    assert np.allclose(oracle.rope(e, 3)[62:], [np.cos(ang), np.sin(ang)], atol=1e-15)


def test_attention_invariants():
    rng = np.random.default_rng(12)
    H, S, dqk, dv = 3, 11, 12, 8
    Q = rng.standard_normal((H, dqk))
    cache = rng.standard_normal((S, dqk))
    O, P = oracle.mla_attention(Q, cache, dv, 0.3, want_p=True)
    assert np.allclose(P.sum(axis=1), 1.0, atol=1e-14)                  # rows sum to one
    # against the textbook formula in numpy
    s = 0.3 * Q @ cache.T
    p = np.exp(s - s.max(axis=1, keepdims=True)); p /= p.sum(axis=1, keepdims=True)
    assert np.allclose(P, p, atol=1e-14) and np.allclose(O, p @ cache[:, :dv], atol=1e-13)
    # one row -> that row; equal rows -> that row; q = 0 -> column mean
    assert np.allclose(oracle.mla_attention(Q, cache[:1], dv, 0.3), np.tile(cache[0, :dv], (H, 1)))
    same = np.tile(cache[2], (S, 1))
    assert np.allclose(oracle.mla_attention(Q, same, dv, 0.3), np.tile(cache[2, :dv], (H, 1)), atol=1e-14)
    assert np.allclose(oracle.mla_attention(np.zeros((H, dqk)), cache, dv, 0.3),
                       np.tile(cache[:, :dv].mean(axis=0), (H, 1)), atol=1e-14)
    # P12: permuting the cache rows leaves the output unchanged
    perm = rng.permutation(S)
    assert np.allclose(oracle.mla_attention(Q, cache[perm], dv, 0.3), O, atol=1e-13)
    # shift invariance of softmax: large scores do not overflow
    assert np.all(np.isfinite(oracle.mla_attention(100 * Q, 100 * cache, dv, 1.0)))


# ---- P11: the absorbed form equals textbook MLA on a tiny instance ----------------------------------

def test_absorbed_equals_textbook_mla():
    rng = np.random.default_rng(13)
    H, S, dc, dn, dr, dv = 2, 5, 8, 4, 4, 4
    c = rng.standard_normal((S, dc))              # latent rows
    kr = rng.standard_normal((S, dr))             # shared rope keys
    q_nope = rng.standard_normal((H, dn))
    q_rope = rng.standard_normal((H, dr))
    W_UK = rng.standard_normal((H, dn, dc))       # q_lat[h] = q_nope[h] * W_UK[h]
    W_UV = rng.standard_normal((H, dc, dv))       # o[h] = o_lat[h] * W_UV[h]
    scale = 1.0 / np.sqrt(dn + dr)
    # textbook: materialise per-head keys and values
    o_ref = np.zeros((H, dv))
    for h in range(H):
        k_nope = c @ W_UK[h].T                    # k_nope[j] = W_UK[h] * c_j
        v = c @ W_UV[h]
        s = scale * (k_nope @ q_nope[h] + kr @ q_rope[h])
        p = np.exp(s - s.max()); p /= p.sum()
        o_ref[h] = p @ v
    # absorbed, through the oracle's own functions
    _, q_lat, _ = oracle.matmul_batched(q_nope, W_UK, 1, dc, dn, H, H * dn, dn, dn * dc, H * dc, dc,
                                        H * dc, F64, F64)
    Q = np.concatenate([q_lat.reshape(H, dc), q_rope], axis=1)
    cache = np.concatenate([c, kr], axis=1)
    o_lat = oracle.mla_attention(Q, cache, dc, scale)
    _, o, _ = oracle.matmul_batched(o_lat, W_UV, 1, dv, dc, H, H * dc, dc, dc * dv, H * dv, dv,
                                    H * dv, F64, F64)
    assert np.allclose(o.reshape(H, dv), o_ref, rtol=0, atol=1e-12)


# ---- the composed step: stages are wired as the definition says -----------------------------------

SMALL_DIMS = dict(d=96, q_lora=48, kv_lora=32, rope=8, nope=16, v=16, H=4)


def _dot_in_k_order(a, b):
    """sum_k a[k]*b[k] with a plain fp64 `+=` over increasing k: the same additions, in the same order, as the
    definition's loop, so the bits of the sum are fixed."""
    acc = 0.0
    for x, y in zip(a, b):
        acc += float(x) * float(y)
    return acc


def _rmsnorm_by_hand(x, gamma, eps):
    ss = 0.0
    for v in x:
        ss += float(v) * float(v)
    r = 1.0 / math.sqrt(ss / len(x) + eps)
    return np.array([float(v) * r * float(g) for v, g in zip(x, gamma)])


def _rope_by_hand(x, pos, base=10000.0):
    y = np.empty(len(x))
    for i in range(len(x) // 2):
        ang = float(pos) * base ** (-2.0 * i / len(x))
        c, s_ = math.cos(ang), math.sin(ang)
        y[2 * i] = float(x[2 * i]) * c - float(x[2 * i + 1]) * s_
        y[2 * i + 1] = float(x[2 * i]) * s_ + float(x[2 * i + 1]) * c
    return y


def test_decode_step_matches_stagewise_recomputation():
    """Every stage of the composed step recomputed by explicit loops from the previous stage's ROUNDED output and
    compared bit for bit: a stage wired to the wrong input, a transposed per-head weight, or a missing rounding
    between two stages (continuing from the unrounded sum) changes bits somewhere and fails."""
    dims, S = SMALL_DIMS, 9
    w = gen.mla_weights(dims, seed=61)
    h = gen.mla_token(dims, seed=62)
    cache = gen.mla_cache(S, dims, seed=63)
    cache0 = cache.copy()
    r = oracle.mla_decode_step(dims, w, h, cache, S)
    d, ql, dc, dr, dn, dv, H = (dims[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
    dq, dkv, pos = dn + dr, dc + dr, S - 1
    f = lambda b: gen.bits_to_f32(np.asarray(b, dtype=np.uint16)).astype(np.float64)
    rbits = oracle.f64_to_bf16
    rb = lambda x: f(rbits(np.asarray(x, dtype=np.float64)))
    hv = f(h)
    W_DQ, W_UQR, W_DKVKR = f(w["W_DQ"]).reshape(d, ql), f(w["W_UQR"]).reshape(ql, H * dq), f(w["W_DKVKR"]).reshape(d, dkv)
    W_UK, W_UV, W_O = f(w["W_UK"]).reshape(H, dn, dc), f(w["W_UV"]).reshape(H, dc, dv), f(w["W_O"]).reshape(H * dv, d)
    # 1-2: c_q, c_qn
    c_q = rb([_dot_in_k_order(hv, W_DQ[:, n]) for n in range(ql)])
    assert np.array_equal(rbits(c_q), r["c_q"])
    c_qn = rb(_rmsnorm_by_hand(c_q, f(w["gamma_q"]), 1e-6))
    assert np.array_equal(rbits(c_qn), r["c_qn"])
    # 3: q from the ROUNDED c_qn
    q = rb([_dot_in_k_order(c_qn, W_UQR[:, n]) for n in range(H * dq)]).reshape(H, dq)
    assert np.array_equal(rbits(q), r["q"])
    # 4: q_rope from the ROUNDED q
    q_rope = rb(np.stack([_rope_by_hand(q[hh, dn:], pos) for hh in range(H)]))
    assert np.array_equal(rbits(q_rope), r["q_rope"])
    # 5-6: ckr and the new cache row (from the ROUNDED ckr); rows before it untouched
    ckr = rb([_dot_in_k_order(hv, W_DKVKR[:, n]) for n in range(dkv)])
    assert np.array_equal(rbits(ckr), r["ckr"])
    assert np.array_equal(cache[:S - 1], cache0[:S - 1])
    row = np.concatenate([_rmsnorm_by_hand(ckr[:dc], f(w["gamma_kv"]), 1e-6), _rope_by_hand(ckr[dc:], pos)])
    assert np.array_equal(rbits(row), cache[S - 1])
    # 7: q_lat[h] = q_nope[h] * W_UK[h] from the ROUNDED q  (W_UK[h] is nope x kv_lora: k runs over nope)
    q_lat = rb([[_dot_in_k_order(q[hh, :dn], W_UK[hh][:, n]) for n in range(dc)] for hh in range(H)])
    assert np.array_equal(rbits(q_lat), r["q_lat"])
    # 8-9: scores over all S rows (the new one included), softmax, o_lat; from the ROUNDED q_lat and q_rope
    rows = f(cache[:S])
    scale = 1.0 / math.sqrt(dq)
    o_lat = np.empty((H, dc))
    for hh in range(H):
        qh = np.concatenate([q_lat[hh], q_rope[hh]])
        s_ = [_dot_in_k_order(qh, rows[j]) * scale for j in range(S)]
        mx = max(s_)
        e = [math.exp(v - mx) for v in s_]
        l = 0.0
        for v in e:
            l += v
        p = [v / l for v in e]
        for c in range(dc):
            o_lat[hh, c] = _dot_in_k_order(p, rows[:, c])
    assert np.allclose(r["o_lat_f64"], o_lat, rtol=0, atol=1e-15)
    assert np.array_equal(rbits(r["o_lat_f64"]), r["o_lat"])
    o_lat = f(r["o_lat"])
    # 10: o[h] = o_lat[h] * W_UV[h] from the ROUNDED o_lat
    o = rb([[_dot_in_k_order(o_lat[hh], W_UV[hh][:, n]) for n in range(dv)] for hh in range(H)])
    assert np.array_equal(rbits(o), r["o"])
    # 11: out = flatten(o) * W_O from the ROUNDED o
    out = [_dot_in_k_order(o.reshape(-1), W_O[:, n]) for n in range(d)]
    assert np.array_equal(rbits(out), r["out"])
    # the rounding points matter at this size: continuing from the unrounded sums would change bits
    q_unrounded_chain = [_dot_in_k_order(_rmsnorm_by_hand(c_q, f(w["gamma_q"]), 1e-6), W_UQR[:, n]) for n in range(H * dq)]
    assert not np.array_equal(rbits(q_unrounded_chain), np.asarray(r["q"]).reshape(-1))


NZ_DIMS = dict(d=96, q_lora=48, kv_lora=32, rope=16, nope=16, v=16, H=4)     # every dense K and N a multiple of 16


@pytest.mark.parametrize("layout", [COL_MAJOR, oracle.FRACTAL_NZ])
def test_decode_step_is_the_same_in_every_storage_of_the_dense_weights(layout):
    """`layout_dense` only changes where element (k, n) of W_DQ, W_UQR, W_DKV|W_KR and W_O is fetched from: the step on
    the permuted storage equals the step on the row-major matrices bit for bit, every stage."""
    dims, S = NZ_DIMS, 7
    w = gen.mla_weights(dims, seed=81)
    h = gen.mla_token(dims, seed=82)
    d, ql, dc, dr, dn, dv, H = (dims[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
    r0 = oracle.mla_decode_step(dims, w, h, gen.mla_cache(S, dims, seed=83), S)
    shapes = {"W_DQ": (d, ql), "W_DKVKR": (d, dc + dr), "W_UQR": (ql, H * (dn + dr)), "W_O": (H * dv, d)}
    store = gen.to_col_major if layout == COL_MAJOR else gen.to_fractal_nz
    w2 = dict(w)
    for name, shp in shapes.items():
        w2[name] = store(np.asarray(w[name]).reshape(shp))
        assert not np.array_equal(w2[name].reshape(-1), np.asarray(w[name]).reshape(-1))   # really another order
    cache = gen.mla_cache(S, dims, seed=83)
    r1 = oracle.mla_decode_step(dims, w2, h, cache, S, layout_dense=layout)
    for k in ("c_q", "c_qn", "q", "q_rope", "ckr", "q_lat", "o_lat", "o", "out"):
        assert np.array_equal(r0[k], r1[k]), k
    # and reading the permuted storage as row-major is NOT the same step (the flag is honoured)
    r2 = oracle.mla_decode_step(dims, w2, h, gen.mla_cache(S, dims, seed=83), S)
    assert not np.array_equal(r0["out"], r2["out"])


def test_decode_step_seq_len_one_attends_only_the_new_row():
    dims = SMALL_DIMS
    w = gen.mla_weights(dims, seed=71, with_wo=False)
    h = gen.mla_token(dims, seed=72)
    cache = gen.mla_cache(1, dims, seed=73)
    r = oracle.mla_decode_step(dims, w, h, cache, 1)
    f = lambda b: gen.bits_to_f32(b).astype(np.float64)
    assert np.array_equal(f(r["o_lat"]), np.tile(f(cache[0, :dims["kv_lora"]]), (dims["H"], 1)))
    assert "out" not in r
