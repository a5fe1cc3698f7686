"""Parity of the CUDA narrow matrix product with the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
from gpu_util import (NP_IN, ORACLE_IN, ORACLE_OUT, assert_matmul_close, guards_intact, out_buffer,
                      out_to_f64, to_dev)

pytestmark = pytest.mark.gpu

F32, BF16, BF16_F32OUT, F16 = 0, 1, 2, 3
ROW, COL = 0, 1


@pytest.fixture(scope="module")
def nm():
    import paper_2609_16009_b200 as nm
    ws = nm.new_workspace(64 << 20)
    nm.nm_set_workspace(ws)
    yield nm
    nm.nm_debug_set_plan(0, 0)
    nm.nm_debug_set_kernel(-1, 0)
    nm.nm_check_status()
    nm.nm_set_workspace(None)


def run_case(nm, A, B_row, M, N, K, dtype, layout, what, full_oracle=True, cols=None, twice=True):
    B = B_row if layout == ROW else gen.to_col_major(B_row)
    dA, dB = to_dev(A), to_dev(B)
    whole, dC = out_buffer(M * N, dtype)
    nm.nm_matmul(dA, dB, dC, M, N, K, dtype, layout)
    torch.cuda.synchronize()
    got = out_to_f64(dC, dtype).reshape(M, N)
    assert guards_intact(whole, M * N, dtype), f"{what}: wrote outside C"
    if twice:   # determinism: no float atomics, fixed-order reductions
        first = dC.clone()
        nm.nm_matmul(dA, dB, dC, M, N, K, dtype, layout)
        torch.cuda.synchronize()
        assert torch.equal(first, dC), f"{what}: two runs differ"
    if cols is None:
        Cq, C64, bound = oracle.matmul(A, B, M, N, K, ORACLE_IN[dtype], ORACLE_OUT[dtype], layout, threads=8)
        assert_matmul_close(got, Cq, C64, bound, dtype, what)
    else:
        Cq, C64, bound = oracle.matmul_columns(A, B, M, N, K, cols, ORACLE_IN[dtype], ORACLE_OUT[dtype], layout)
        assert_matmul_close(got[:, cols], Cq, C64, bound, dtype, what)
    return got


def make_inputs(M, K, N, dtype, seed):
    if dtype == F32:
        return gen.uniform_f32((M, K), -1, 1, seed), gen.uniform_f32((K, N), -1, 1, seed + 1)
    if dtype == F16:
        return gen.narrow_f16(M, K, N, seed)
    return gen.narrow_bf16(M, K, N, seed)


# ---- the named configurations ------------------------------------------------------------------------

def test_gemv_fp32_512(nm):
    A, B = gen.gemv_fp32(seed=0)
    run_case(nm, A, B, 1, 512, 512, F32, ROW, "fp32 GEMV 512x512")
    run_case(nm, A, B, 1, 512, 512, F32, COL, "fp32 GEMV 512x512 col-major")


@pytest.mark.parametrize("N", [1536, 576])
@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("dtype", [BF16, BF16_F32OUT])
def test_down_projection_shapes(nm, N, layout, dtype):
    A, B = gen.narrow_bf16(1, 7168, N, seed=1000 + N)
    run_case(nm, A, B, 1, N, 7168, dtype, layout, f"M=1 K=7168 N={N} layout={layout}")


@pytest.mark.parametrize("K,N", [(1536, 24576), (7168, 18432)])
@pytest.mark.parametrize("M", [1, 2, 4, 8, 16])
def test_m_sweep_full_size_sampled_columns(nm, K, N, M):
    A, B = gen.narrow_bf16(M, K, N, seed=2000 + M)
    rng = np.random.default_rng(M)
    cols = sorted(set([0, 7, 8, 255, 256, N - 1, N - 8] + rng.integers(0, N, 56).tolist()))
    run_case(nm, A, B, M, N, K, BF16, ROW, f"M={M} K={K} N={N}", cols=cols)


@pytest.mark.parametrize("M,K,N", [(1, 16384, 7168), (2, 16384, 7168), (8, 16384, 7168), (3, 7168, 1536), (16, 7168, 1536),
                                   (1, 8192, 8192), (5, 4096, 4096)])
def test_other_large_and_mid_size_shapes_sampled_columns(nm, M, K, N):
    # the output projection's shape and a few more on either side of the planner's thresholds (one CTA per SM
    # for large matrices, tensor cores from 16 MB at M >= 3, batched split-K gather)
    A, B = gen.narrow_bf16(M, K, N, seed=2100 + M + K % 97)
    rng = np.random.default_rng(M + N)
    cols = sorted(set([0, 63, 64, 127, 128, N - 1, N - 64] + rng.integers(0, N, 40).tolist()))
    run_case(nm, A, B, M, N, K, BF16, ROW, f"M={M} K={K} N={N}", cols=cols)


@pytest.mark.parametrize("M,K,N", [(3, 7168, 18432), (16, 7168, 18432), (4, 1536, 24576), (8, 7168, 1536)])
def test_column_major_on_the_tensor_cores_sampled_columns(nm, M, K, N):
    # column-major weights ([N][K]) at M >= 3 on large matrices: the swap-AB kernel with a K-major weight operand
    assert nm.nm_debug_get_plan(M, N, K, layout_B=COL)["kind"] == 4
    A, B = gen.narrow_bf16(M, K, N, seed=2300 + M)
    rng = np.random.default_rng(M + N)
    cols = sorted(set([0, 63, 64, 127, 128, N - 1, N - 64] + rng.integers(0, N, 40).tolist()))
    run_case(nm, A, B, M, N, K, BF16, COL, f"col-major M={M} K={K} N={N}", cols=cols)


@pytest.mark.parametrize("M,K,N", [(1, 64, 128), (5, 200, 136), (16, 1000, 840), (3, 4104, 72), (2, 8, 8), (7, 72, 1000)])
@pytest.mark.parametrize("dtype", [BF16, BF16_F32OUT])
def test_column_major_tensor_core_kernel_forced_on_small_and_ragged_shapes(nm, M, K, N, dtype):
    # K not a multiple of the 64-k stage, N not a multiple of the 128-column tile, several k-splits
    A, B = gen.narrow_bf16(M, K, N, seed=2400 + M + K)
    nm.nm_debug_set_kernel(4, 0)
    try:
        for nsplit in (0, 3):
            nm.nm_debug_set_plan(0, nsplit)
            run_case(nm, A, B, M, N, K, dtype, COL, f"forced col-major tensor-core kernel M={M} K={K} N={N} nsplit={nsplit}")
    finally:
        nm.nm_debug_set_kernel(-1, 0)
        nm.nm_debug_set_plan(0, 0)


@pytest.mark.parametrize("rows,K", [(576, 7168), (1536, 7168), (1000, 1001), (7, 40)])
@pytest.mark.parametrize("dtype", [F32, BF16, BF16_F32OUT])
def test_matrix_times_column_vector_by_transposition(nm, rows, K, dtype):
    """The other narrow case of the Narrow Dimension condition, N = 1: C[rows x 1] = W[rows x K] * x[K x 1].  The oracle
    computes exactly that (its M is not limited); the library is given the transposed problem C^T = x^T * W^T, in
    which the row-major W is a column-major B - no copy, no transposition pass."""
    if dtype == F32:
        W, x = gen.uniform_f32((rows, K), -1, 1, 2500 + rows), gen.uniform_f32((K, 1), -1, 1, 2501 + rows)
    else:
        x, Wt = gen.narrow_bf16(1, K, rows, seed=2500 + rows)       # x: [1][K] ~ N(0,1); Wt: [K][rows] ~ N(0, 0.02^2)
        W = np.ascontiguousarray(np.asarray(Wt).reshape(K, rows).T)
        x = np.asarray(x).reshape(K, 1)
    Cq, C64, bound = oracle.matmul(W, x, rows, 1, K, ORACLE_IN[dtype], ORACLE_OUT[dtype], ROW, threads=8)
    dW, dx = to_dev(W), to_dev(x)
    whole, dC = out_buffer(rows, dtype)
    nm.nm_matmul(dx, dW, dC, 1, rows, K, dtype, COL)             # A = x^T [1 x K], B = W read as [K x rows] column-major
    torch.cuda.synchronize()
    assert guards_intact(whole, rows, dtype)
    assert_matmul_close(out_to_f64(dC, dtype).reshape(rows, 1), Cq, C64, bound, dtype, f"column vector rows={rows} K={K}")


# ---- every M, ragged shapes, both layouts, all dtypes ------------------------------------------------------

@pytest.mark.parametrize("M", list(range(1, 17)))
@pytest.mark.parametrize("layout", [ROW, COL])
def test_every_m_vector_path(nm, M, layout):
    # several tiles in N with a ragged last tile; several k-chunks with a ragged tail
    K, N = 1000, 840
    A, B = gen.narrow_bf16(M, K, N, seed=300 + M)
    run_case(nm, A, B, M, N, K, BF16, layout, f"M={M} K={K} N={N} layout={layout}")


@pytest.mark.parametrize("dtype", [F32, BF16, BF16_F32OUT])
@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("M,K,N", [(1, 1, 1), (3, 5, 7), (2, 129, 33), (16, 77, 1), (5, 1023, 259),
                                    (1, 8, 8), (4, 4096, 8), (7, 8, 2048), (16, 2600, 72)])
def test_ragged_and_degenerate_shapes(nm, dtype, layout, M, K, N):
    A, B = make_inputs(M, K, N, dtype, seed=400 + M + K + N)
    run_case(nm, A, B, M, N, K, dtype, layout, f"dtype={dtype} layout={layout} {M}x{K}x{N}")


# ---- fp16, the optional element type (CUDA-core kernels, both layouts, 1 <= M <= 16) -----------------------

@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("M,K,N", [(1, 1, 1), (3, 5, 7), (2, 129, 33), (16, 77, 1), (5, 1023, 259), (1, 8, 8), (7, 8, 2048),
                                    (1, 1000, 840), (4, 1000, 840), (16, 1000, 840), (1, 7168, 576), (2, 7168, 1536), (16, 2600, 72)])
def test_fp16_products(nm, layout, M, K, N):
    A, B = gen.narrow_f16(M, K, N, seed=450 + M + K + N)
    run_case(nm, A, B, M, N, K, F16, layout, f"fp16 layout={layout} {M}x{K}x{N}")


@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("nsplit", [1, 3, 16])
def test_fp16_forced_splits_and_ties(nm, layout, nsplit):
    M, K, N = 3, 4096, 264
    A, B = gen.narrow_f16(M, K, N, seed=470)
    nm.nm_debug_set_plan(0, nsplit)
    try:
        run_case(nm, A, B, M, N, K, F16, layout, f"fp16 nsplit={nsplit} layout={layout}")
        # sums that are ties of the fp16 grid: 2048 + 1 -> 2048 (even), 2048 + 3 -> 2052, in every column
        to16 = lambda v: np.ascontiguousarray(v, np.float16).view(np.uint16)
        K2, N2 = 64, 16
        col = np.zeros((K2, N2)); col[0] = 1024.0; col[1] = 512.0; col[2] = 512.0; col[3, ::2] = 1.0; col[3, 1::2] = 3.0
        got = run_case(nm, to16(np.ones((1, K2))), to16(col), 1, N2, K2, F16, layout, "fp16 ties")
        assert np.array_equal(got[0, ::2], np.full(N2 // 2, 2048.0)) and np.array_equal(got[0, 1::2], np.full(N2 // 2, 2052.0))
    finally:
        nm.nm_debug_set_plan(0, 0)


@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("M,K,N,nsplit", [(1, 4096, 1024, 0), (2, 7168, 1536, 0), (5, 2048, 2304, 2), (16, 1536, 4096, 0), (9, 1000, 4104, 3),
                                           (17, 640, 512, 0), (40, 1536, 1024, 2), (64, 2048, 384, 0)])
def test_fp16_on_the_tensor_cores(nm, layout, M, K, N, nsplit):
    """fp16 operands through the swap-AB kernel (kind::f16 with both operand formats fp16): the planner's own choice from
    8 MB of weights on, forced below that; ragged k tails and column tiles; 17 to 64 rows in one pass."""
    A, B = gen.narrow_f16(M, K, N, seed=460 + M)
    nm.nm_debug_set_kernel(4, 0)
    nm.nm_debug_set_plan(0, nsplit)
    try:
        assert nm.nm_debug_get_plan(M, N, K, dtype=F16, layout_B=layout)["kind"] == 4
        run_case(nm, A, B, M, N, K, F16, layout, f"fp16 tensor cores layout={layout} {M}x{K}x{N} nsplit={nsplit}")
    finally:
        nm.nm_debug_set_kernel(-1, 0)
        nm.nm_debug_set_plan(0, 0)


def test_fp16_kernel_choice_and_refusals(nm):
    assert nm.nm_debug_get_plan(1, 18432, 7168, dtype=F16)["kind"] == 4          # 264 MB: tensor cores at every M
    assert nm.nm_debug_get_plan(16, 1536, 7168, dtype=F16)["kind"] == 4
    assert nm.nm_debug_get_plan(1, 576, 1024, dtype=F16)["kind"] == 0            # 1.2 MB: CUDA-core row kernel
    assert nm.nm_debug_get_plan(1, 576, 1024, dtype=F16, layout_B=COL)["kind"] == 1
    A, B = gen.narrow_f16(1, 64, 64, seed=480)
    C = torch.zeros(64, dtype=torch.int16, device="cuda")
    with pytest.raises(nm.NmError) as e:
        nm.nm_matmul(to_dev(A), to_dev(B), C, 1, 64, 64, F16, 2)             # FRACTAL_NZ: bf16 only
    assert e.value.status == -2
    A17, B17 = gen.narrow_f16(17, 63, 64, seed=481)                           # K = 63: no tensor map, and 17 rows need one
    with pytest.raises(nm.NmError) as e:
        nm.nm_matmul(to_dev(A17), to_dev(B17), torch.zeros(17 * 64, dtype=torch.int16, device="cuda"), 17, 64, 63, F16, ROW)
    assert e.value.status == -2
    nm.nm_check_status()


@pytest.mark.parametrize("layout", [ROW, COL])
def test_long_k_spans_several_shared_memory_chunks(nm, layout):
    M, K, N = 16, 9000, 64
    A, B = gen.narrow_bf16(M, K, N, seed=500)
    nm.nm_debug_set_plan(0, 1)           # no split: one CTA walks all of K in chunks
    try:
        run_case(nm, A, B, M, N, K, BF16, layout, f"long K layout={layout}")
    finally:
        nm.nm_debug_set_plan(0, 0)


# ---- split-K: forced plans, determinism -----------------------------------------------------------------

@pytest.mark.parametrize("layout,kernel", [(ROW, -1), (ROW, 0), (COL, -1)])
@pytest.mark.parametrize("nsplit", [1, 2, 7, 16, 64])
@pytest.mark.parametrize("tile_n", [0, 64, 128, 136, 256, 512])
def test_forced_plans_agree(nm, layout, kernel, nsplit, tile_n):
    # kernel -1: the library's choice (TMA ring for row-major bf16); 0: the plain-load kernel
    M, K, N = 3, 7168, 576
    A, B = gen.narrow_bf16(M, K, N, seed=600)
    nm.nm_debug_set_plan(tile_n, nsplit)
    nm.nm_debug_set_kernel(kernel, 0)
    try:
        run_case(nm, A, B, M, N, K, BF16, layout, f"forced tile_n={tile_n} nsplit={nsplit} layout={layout} kernel={kernel}")
    finally:
        nm.nm_debug_set_plan(0, 0)
        nm.nm_debug_set_kernel(-1, 0)


@pytest.mark.parametrize("M", list(range(1, 17)))
@pytest.mark.parametrize("tile_n", [64, 128, 256])
def test_tma_ring_every_m_and_tile(nm, M, tile_n):
    # K spans several A chunks (256 rows at M=16) and ends mid-stage; N ends mid-tile
    K, N = 1000, 840
    A, B = gen.narrow_bf16(M, K, N, seed=900 + M)
    for stages in (2, 0):
        nm.nm_debug_set_plan(tile_n, 2)
        nm.nm_debug_set_kernel(3, stages)
        try:
            assert nm.nm_debug_get_plan(M, N, K)["kind"] == 3
            run_case(nm, A, B, M, N, K, BF16, ROW, f"tma M={M} tile_n={tile_n} stages={stages}")
        finally:
            nm.nm_debug_set_plan(0, 0)
            nm.nm_debug_set_kernel(-1, 0)
    nm.nm_check_status()


@pytest.mark.parametrize("M,tile_n", [(1, 64), (1, 256), (2, 128), (4, 64), (8, 64), (16, 64), (16, 128)])
@pytest.mark.parametrize("nsplit", [2, 3, 5, 8, 9])
def test_split_k_inside_a_cluster_matches_the_workspace_path(nm, M, tile_n, nsplit):
    """Up to eight k-splits whose partial tiles fit 16 KB meet in the shared memory of a thread-block cluster; more,
    or larger ones, go through the workspace.  Same summation order either way: identical bits, and parity with
    the oracle.  K ends mid-stage and N mid-tile."""
    K, N = 2500, 840
    A, B = gen.narrow_bf16(M, K, N, seed=950 + M)
    outs = []
    for cluster in (True, False):
        nm.nm_debug_set_plan(tile_n, nsplit)
        nm.nm_debug_set_kernel(3, 0)
        nm.nm_debug_set_cluster_split(cluster)
        try:
            assert nm.nm_debug_get_plan(M, N, K)["kind"] == 3
            outs.append(run_case(nm, A, B, M, N, K, BF16, ROW, f"split-K M={M} tile_n={tile_n} nsplit={nsplit} cluster={cluster}"))
        finally:
            nm.nm_debug_set_plan(0, 0)
            nm.nm_debug_set_kernel(-1, 0)
            nm.nm_debug_set_cluster_split(True)
    assert np.array_equal(outs[0], outs[1])
    nm.nm_check_status()


@pytest.mark.parametrize("layout,dtype", [(ROW, BF16), (ROW, F32), (COL, BF16), (COL, F32)])
@pytest.mark.parametrize("M,nsplit", [(1, 2), (1, 8), (2, 5), (4, 8), (7, 3), (16, 2), (16, 4), (3, 9)])
def test_split_k_inside_a_cluster_plain_kernels(nm, layout, dtype, M, nsplit):
    """The plain row-major kernel and the column-major kernel: k-splits meeting in a cluster (up to eight, 8 KB of
    partial tiles) against the workspace path - identical bits, parity with the oracle."""
    K, N = 2056, 328
    A, B = make_inputs(M, K, N, dtype, seed=970 + M)
    outs = []
    for cluster in (True, False):
        nm.nm_debug_set_plan(0, nsplit)
        nm.nm_debug_set_kernel(0, 0)
        nm.nm_debug_set_cluster_split(cluster)
        try:
            assert nm.nm_debug_get_plan(M, N, K, 1, dtype, layout)["kind"] == (0 if layout == ROW else 1)
            outs.append(run_case(nm, A, B, M, N, K, dtype, layout, f"plain split-K M={M} nsplit={nsplit} layout={layout} cluster={cluster}"))
        finally:
            nm.nm_debug_set_plan(0, 0)
            nm.nm_debug_set_kernel(-1, 0)
            nm.nm_debug_set_cluster_split(True)
    assert np.array_equal(outs[0], outs[1])
    nm.nm_check_status()


@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("M,nsplit", [(3, 2), (4, 8), (9, 5), (16, 8), (16, 3), (5, 9)])
def test_split_k_inside_a_cluster_tensor_core_kernel(nm, layout, M, nsplit):
    """The swap-AB tensor-core kernel: up to eight k-splits (64 KB of partial tiles) meeting in a cluster against
    the workspace path - identical bits, parity with the oracle.  K ends mid-stage and N mid-tile."""
    K, N = 2600, 840
    A, B = gen.narrow_bf16(M, K, N, seed=990 + M)
    outs = []
    for cluster in (True, False):
        nm.nm_debug_set_plan(0, nsplit)
        nm.nm_debug_set_kernel(4, 0)
        nm.nm_debug_set_cluster_split(cluster)
        try:
            assert nm.nm_debug_get_plan(M, N, K, 1, BF16, layout)["kind"] == 4
            outs.append(run_case(nm, A, B, M, N, K, BF16, layout, f"tc split-K M={M} nsplit={nsplit} layout={layout} cluster={cluster}"))
        finally:
            nm.nm_debug_set_plan(0, 0)
            nm.nm_debug_set_kernel(-1, 0)
            nm.nm_debug_set_cluster_split(True)
    assert np.array_equal(outs[0], outs[1])
    nm.nm_check_status()


@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("M,K,N,nsplit", [(17, 1000, 840, 0), (24, 2600, 328, 3), (32, 512, 1536, 0), (33, 1000, 840, 2),
                                          (48, 7168, 576, 0), (64, 2600, 840, 5)])
def test_more_than_sixteen_rows_in_one_pass_on_the_tensor_cores(nm, layout, M, K, N, nsplit):
    """The paper's outlook (a remainder row beside a multiple of 16, larger tokens): up to 64 rows go through the
    swap-AB tensor-core kernel with 32 or 64 token columns, B still streamed once.  Parity with the oracle,
    both weight layouts, with and without k-splits (cluster and workspace paths)."""
    A, B = gen.narrow_bf16(M, K, N, seed=1100 + M)
    for cluster in (True, False):
        nm.nm_debug_set_plan(0, nsplit)
        nm.nm_debug_set_cluster_split(cluster)
        try:
            assert nm.nm_debug_get_plan(M, N, K, 1, BF16, layout)["kind"] == 4
            run_case(nm, A, B, M, N, K, BF16, layout, f"M={M} K={K} N={N} nsplit={nsplit} layout={layout} cluster={cluster}")
        finally:
            nm.nm_debug_set_plan(0, 0)
            nm.nm_debug_set_cluster_split(True)
    nm.nm_check_status()


def test_more_than_sixteen_rows_needs_operands_the_tensor_core_kernel_takes(nm):
    M, K, N = 20, 256, 256
    A, B = make_inputs(M, K, N, F32, seed=1200)
    dA, dB = to_dev(A), to_dev(B)
    whole, dC = out_buffer(M * N, F32)
    with pytest.raises(nm.NmError) as e:
        nm.nm_matmul(dA, dB, dC, M, N, K, F32, ROW)
    assert e.value.status == -2
    with pytest.raises(nm.NmError) as e:
        nm.nm_matmul(dA, dB, dC, 65, N, K, BF16, ROW)
    assert e.value.status == -1


NZ = 2


@pytest.mark.parametrize("M", [1, 2, 5, 16])
@pytest.mark.parametrize("K,N,tile_n,nsplit", [(7168, 576, 0, 0), (1008, 848, 64, 3), (1008, 848, 128, 2), (2048, 1280, 256, 1),
                                               (4096, 4096, 0, 0)])
def test_fractal_nz_weights_read_in_place(nm, M, K, N, tile_n, nsplit):
    """The paper's weight storage (16 x 16 fractals ordered by columns, rows inside) as a layout of B: tiled TMA copies
    present the fractals to the ring kernel, no transposition pass.  Parity with the oracle on the fractal storage."""
    A, B = gen.narrow_bf16(M, K, N, seed=1300 + M)
    Bnz = gen.to_fractal_nz(B)
    dA, dB, dBnz = to_dev(A), to_dev(B), to_dev(Bnz)
    Cq, C64, bound = oracle.matmul(A, Bnz, M, N, K, ORACLE_IN[BF16], ORACLE_OUT[BF16], oracle.FRACTAL_NZ, threads=8)
    nm.nm_debug_set_plan(tile_n, nsplit)
    nm.nm_debug_set_kernel(3, 0)
    try:
        plan_nz, plan_row = nm.nm_debug_get_plan(M, N, K, 1, BF16, NZ), nm.nm_debug_get_plan(M, N, K, 1, BF16, ROW)
        assert plan_nz["kind"] == 3
        whole, dC = out_buffer(M * N, BF16)
        nm.nm_matmul(dA, dBnz, dC, M, N, K, BF16, NZ)
        whole_r, dC_r = out_buffer(M * N, BF16)
        nm.nm_matmul(dA, dB, dC_r, M, N, K, BF16, ROW)
        torch.cuda.synchronize()
    finally:
        nm.nm_debug_set_plan(0, 0)
        nm.nm_debug_set_kernel(-1, 0)
    assert guards_intact(whole, M * N, BF16)
    assert_matmul_close(out_to_f64(dC, BF16).reshape(M, N), Cq, C64, bound, BF16, f"fractal M={M} K={K} N={N}")
    # against the row-major storage of the same matrix: the same products, summed in another order (the fractal path
    # deals the rows to the threads differently), so equal within the bound rather than bit for bit
    assert plan_nz["tile_n"] == plan_row["tile_n"]
    assert_matmul_close(out_to_f64(dC_r, BF16).reshape(M, N), Cq, C64, bound, BF16, f"row-major M={M} K={K} N={N}")
    nm.nm_check_status()


def test_fractal_nz_batched_and_refusals(nm):
    T, H, K, N = 2, 4, 256, 96
    A = gen.normal_bf16((T, H, K), 1.0, seed=1400)
    W = gen.normal_bf16((H, K, N), 0.02, seed=1401)
    Wnz = np.stack([gen.to_fractal_nz(W[h]) for h in range(H)])
    dA, dW = to_dev(A), to_dev(Wnz)
    whole, dC = out_buffer(T * H * N, BF16_F32OUT)
    nm.nm_matmul_batched(dA, dW, dC, T, N, K, H, H * K, K, K * N, H * N, N, BF16_F32OUT, NZ)
    torch.cuda.synchronize()
    Cq, C64, bound = oracle.matmul_batched(A, W, T, N, K, H, H * K, K, K * N, H * N, N, T * H * N, oracle.BF16, oracle.F32, ROW)
    assert guards_intact(whole, T * H * N, BF16_F32OUT)
    assert_matmul_close(out_to_f64(dC, BF16_F32OUT), Cq, C64, bound, BF16_F32OUT, "fractal batched")
    # partial fractals, fp32 and more than 16 rows are refused
    Cb = torch.zeros(64 * 96, dtype=torch.int16, device="cuda")
    for args in ((dA, dW, Cb, 1, 90, 256, BF16, NZ), (dA, dW, Cb, 1, 96, 250, BF16, NZ), (dA, dW, Cb, 1, 96, 256, F32, NZ),
                 (dA, dW, Cb, 17, 96, 256, BF16, NZ)):
        with pytest.raises(nm.NmError) as e:
            nm.nm_matmul(*args)
        assert e.value.status == -2
    nm.nm_check_status()


def test_paper_matmul_2_shape_takes_eight_splits_in_a_cluster(nm):
    plan = nm.nm_debug_get_plan(1, 576, 7168)
    assert plan["kind"] == 3 and plan["nsplit"] == 8


@pytest.mark.parametrize("M", [1, 2, 5, 8, 9, 13, 16])
@pytest.mark.parametrize("nsplit", [0, 1, 3])
def test_tensor_core_swap_ab_kernel(nm, M, nsplit):
    # weights as the MMA's M dimension, tokens as its N: same tolerance as the CUDA-core kernels.
    # K ends mid-stage (1000 = 15*64 + 40) and N ends mid-tile (840 = 6*128 + 72).
    K, N = 1000, 840
    A, B = gen.narrow_bf16(M, K, N, seed=1200 + M)
    nm.nm_debug_set_plan(0, nsplit)
    nm.nm_debug_set_kernel(4, 0)
    try:
        assert nm.nm_debug_get_plan(M, N, K)["kind"] == 4
        run_case(nm, A, B, M, N, K, BF16, ROW, f"tensor-core M={M} nsplit={nsplit}")
        run_case(nm, A, B, M, N, K, BF16_F32OUT, ROW, f"tensor-core fp32 out M={M} nsplit={nsplit}")
    finally:
        nm.nm_debug_set_plan(0, 0)
        nm.nm_debug_set_kernel(-1, 0)
    nm.nm_check_status()


def test_tensor_core_kernel_small_integers_bit_exact(nm):
    M, K, N = 16, 7168, 576
    A = gen.small_int_bf16((M, K), -8, 8, seed=1301)
    B = gen.small_int_bf16((K, N), -8, 8, seed=1302)
    nm.nm_debug_set_kernel(4, 0)
    try:
        got = run_case(nm, A, B, M, N, K, BF16_F32OUT, ROW, "tensor-core small ints")
    finally:
        nm.nm_debug_set_kernel(-1, 0)
    _, C64, _ = oracle.matmul(A, B, M, N, K, oracle.BF16, oracle.F32, ROW, threads=8)
    assert np.array_equal(got, C64)


def test_many_tensor_core_products_in_one_process_cycle_the_tensor_map_cache(nm):
    """The library keeps the tensor maps of recent operands (16 entries).  Forty products with distinct token and
    weight buffers make every entry be replaced several times, between the two lookups of one call as well."""
    K, N = 256, 384
    nm.nm_debug_set_kernel(4, 0)
    try:
        keep = []
        for i in range(40):
            M = 3 + i % 14
            A, B = gen.narrow_bf16(M, K, N, seed=2000 + i)
            dA, dB = to_dev(A), to_dev(B)
            whole, dC = out_buffer(M * N, BF16)
            keep.append((dA, dB, whole))                           # distinct addresses: nothing is freed in between
            assert nm.nm_debug_get_plan(M, N, K)["kind"] == 4
            nm.nm_matmul(dA, dB, dC, M, N, K, BF16, ROW)
            torch.cuda.synchronize()
            Cq, C64, bound = oracle.matmul(A, B, M, N, K, ORACLE_IN[BF16], ORACLE_OUT[BF16], ROW, threads=8)
            assert_matmul_close(out_to_f64(dC, BF16).reshape(M, N), Cq, C64, bound, BF16, f"product {i}")
    finally:
        nm.nm_debug_set_kernel(-1, 0)
    nm.nm_check_status()


def test_default_kernel_choice_by_m(nm):
    # CUDA cores (TMA ring) for one or two token rows and for small weight matrices, tensor cores from
    # three rows on for large ones; the threshold is adjustable
    assert nm.nm_debug_get_plan(2, 18432, 7168)["kind"] == 3
    assert nm.nm_debug_get_plan(3, 18432, 7168)["kind"] == 4
    assert nm.nm_debug_get_plan(16, 576, 7168)["kind"] == 3          # 8 MB in one matrix: CUDA cores at every M
    assert nm.nm_debug_get_plan(4, 1536, 7168)["kind"] == 4          # 22 MB: from M = 3 on
    assert nm.nm_debug_get_plan(4, 512, 128, H=128)["kind"] == 4     # batched per-head products, 16.8 MB in all
    assert nm.nm_debug_get_plan(2, 512, 128, H=128)["kind"] == 3
    nm.nm_set_tensor_core_min_m(17)
    try:
        assert nm.nm_debug_get_plan(16, 18432, 7168)["kind"] == 3
    finally:
        nm.nm_set_tensor_core_min_m(3)


def test_plain_row_kernel_every_m(nm):
    K, N = 1000, 840
    nm.nm_debug_set_kernel(0, 0)
    try:
        for M in range(1, 17):
            A, B = gen.narrow_bf16(M, K, N, seed=950 + M)
            assert nm.nm_debug_get_plan(M, N, K)["kind"] == 0
            run_case(nm, A, B, M, N, K, BF16, ROW, f"plain row kernel M={M}")
    finally:
        nm.nm_debug_set_kernel(-1, 0)


@pytest.mark.parametrize("layout", [ROW, COL])
def test_small_integers_bit_exact_full_k(nm, layout):
    # every product and every partial sum is an integer below 2^24: any summation order is exact,
    # so the fp32 result must match the oracle bit for bit
    M, K, N = 4, 7168, 576
    A = gen.small_int_bf16((M, K), -8, 8, seed=701)
    B = gen.small_int_bf16((K, N), -8, 8, seed=702)
    got = run_case(nm, A, B, M, N, K, BF16_F32OUT, layout, "small ints")
    _, C64, _ = oracle.matmul(A, B if layout == ROW else gen.to_col_major(B), M, N, K, oracle.BF16, oracle.F32, layout, threads=8)
    assert np.array_equal(got, C64)


def test_rounding_ties_to_even_on_device(nm):
    K = 64
    A = gen.bf16_bits(torch.ones(1, K))
    cols = []
    for total in (257.0, 259.0, 255.0, -257.0):
        col = np.full(K, np.sign(total) * 4.0, np.float32)
        col[0] = total - np.sign(total) * 4.0 * (K - 1)
        cols.append(col)
    B = gen.bf16_bits(torch.from_numpy(np.stack(cols, axis=1)))        # K x 4
    Bp = np.zeros((K, 8), np.uint16); Bp[:, :4] = B
    got = run_case(nm, A, Bp, 1, 8, K, BF16, ROW, "ties")
    assert got[0, :4].tolist() == [256.0, 260.0, 255.0, -256.0]


# ---- batched per-head products ---------------------------------------------------------------------------

@pytest.mark.parametrize("T", [1, 4, 16])
def test_per_head_absorbed_products(nm, T):
    H, nope, dc, dv, rope = 128, 128, 512, 128, 64
    d = gen.per_head(T, seed=3000 + T)
    # q_nope read in place from q[T][H][nope+rope]
    q = gen.normal_bf16((T, H, nope + rope), 1.0, seed=3100 + T)
    dq, dW = to_dev(q), to_dev(d["W_UK"])
    whole, dC = out_buffer(T * H * dc, BF16)
    nm.nm_matmul_batched(dq, dW, dC, T, dc, nope, H, H * (nope + rope), nope + rope, nope * dc, H * dc, dc, BF16, ROW)
    torch.cuda.synchronize()
    assert guards_intact(whole, T * H * dc, BF16)
    Cq, C64, bound = oracle.matmul_batched(q, d["W_UK"], T, dc, nope, H, H * (nope + rope), nope + rope,
                                           nope * dc, H * dc, dc, T * H * dc, oracle.BF16, oracle.BF16, threads=8)
    assert_matmul_close(out_to_f64(dC, BF16), Cq, C64, bound, BF16, f"W_UK T={T}")
    # o_lat [T,H,dc] * W_UV [H,dc,dv]
    dO, dW = to_dev(d["o_lat"]), to_dev(d["W_UV"])
    whole, dC = out_buffer(T * H * dv, BF16)
    nm.nm_matmul_batched(dO, dW, dC, T, dv, dc, H, H * dc, dc, dc * dv, H * dv, dv, BF16, ROW)
    torch.cuda.synchronize()
    assert guards_intact(whole, T * H * dv, BF16)
    Cq, C64, bound = oracle.matmul_batched(d["o_lat"], d["W_UV"], T, dv, dc, H, H * dc, dc, dc * dv, H * dv, dv,
                                           T * H * dv, oracle.BF16, oracle.BF16, threads=8)
    assert_matmul_close(out_to_f64(dC, BF16), Cq, C64, bound, BF16, f"W_UV T={T}")


@pytest.mark.parametrize("layout", [ROW, COL])
def test_batched_small_ragged(nm, layout):
    T, H, K, N = 3, 5, 40, 24
    A = gen.normal_bf16((T, H, K), 1.0, seed=3200)
    W = gen.normal_bf16((H, K, N), 0.02, seed=3201)
    Wst = W if layout == ROW else np.ascontiguousarray(W.transpose(0, 2, 1))
    dA, dW = to_dev(A), to_dev(Wst)
    whole, dC = out_buffer(T * H * N, BF16_F32OUT)
    nm.nm_matmul_batched(dA, dW, dC, T, N, K, H, H * K, K, K * N, H * N, N, BF16_F32OUT, layout)
    torch.cuda.synchronize()
    assert guards_intact(whole, T * H * N, BF16_F32OUT)
    Cq, C64, bound = oracle.matmul_batched(A, Wst, T, N, K, H, H * K, K, K * N, H * N, N, T * H * N,
                                           oracle.BF16, oracle.F32, layout)
    assert_matmul_close(out_to_f64(dC, BF16_F32OUT), Cq, C64, bound, BF16_F32OUT, "batched ragged")


@pytest.mark.parametrize("layout", [ROW, COL])
def test_batched_fp16(nm, layout):
    T, H, K, N = 3, 5, 136, 24
    A16, _ = gen.narrow_f16(T * H, K, 1, seed=3250)
    W16 = np.stack([gen.narrow_f16(1, K, N, seed=3251 + h)[1] for h in range(H)])
    A = A16.reshape(T, H, K)
    Wst = W16 if layout == ROW else np.ascontiguousarray(W16.transpose(0, 2, 1))
    dA, dW = to_dev(A), to_dev(Wst)
    whole, dC = out_buffer(T * H * N, F16)
    nm.nm_matmul_batched(dA, dW, dC, T, N, K, H, H * K, K, K * N, H * N, N, F16, layout)
    torch.cuda.synchronize()
    assert guards_intact(whole, T * H * N, F16)
    Cq, C64, bound = oracle.matmul_batched(A, Wst, T, N, K, H, H * K, K, K * N, H * N, N, T * H * N,
                                           oracle.F16, oracle.F16, layout)
    assert_matmul_close(out_to_f64(dC, F16), Cq, C64, bound, F16, "batched fp16")


@pytest.mark.parametrize("layout", [ROW, COL])
@pytest.mark.parametrize("T,kernel,nsplit", [(1, 3, 4), (2, 0, 3), (2, -1, 2), (5, 4, 3), (16, 4, 2), (24, -1, 0), (40, -1, 2)])
def test_batched_products_with_k_splits_in_clusters_and_with_many_rows(nm, T, kernel, nsplit, layout):
    """Per-head batches (heads = gridDim.z) through every kernel family with forced k-splits - the splits of a
    (head, tile) meet inside a cluster - and with 17 to 64 rows per head on the tensor cores."""
    H, K, N = 6, 1280, 256
    if layout == COL and kernel in (0, 3):
        kernel = -1                                               # the row-major CUDA-core kernels do not take column-major B
    A = gen.normal_bf16((T, H, K), 1.0, seed=3300 + T)
    W = gen.normal_bf16((H, K, N), 0.02, seed=3301 + T)
    Wst = W if layout == ROW else np.ascontiguousarray(W.transpose(0, 2, 1))
    dA, dW = to_dev(A), to_dev(Wst)
    Cq, C64, bound = oracle.matmul_batched(A, Wst, T, N, K, H, H * K, K, K * N, H * N, N, T * H * N,
                                           oracle.BF16, oracle.F32, layout)
    outs = []
    for cluster in (True, False):
        whole, dC = out_buffer(T * H * N, BF16_F32OUT)
        nm.nm_debug_set_plan(0, nsplit)
        nm.nm_debug_set_kernel(kernel, 0)
        nm.nm_debug_set_cluster_split(cluster)
        try:
            nm.nm_matmul_batched(dA, dW, dC, T, N, K, H, H * K, K, K * N, H * N, N, BF16_F32OUT, layout)
            torch.cuda.synchronize()
        finally:
            nm.nm_debug_set_plan(0, 0)
            nm.nm_debug_set_kernel(-1, 0)
            nm.nm_debug_set_cluster_split(True)
        assert guards_intact(whole, T * H * N, BF16_F32OUT)
        assert_matmul_close(out_to_f64(dC, BF16_F32OUT), Cq, C64, bound, BF16_F32OUT, f"batched T={T} kernel={kernel} cluster={cluster}")
        outs.append(dC.clone())
    assert torch.equal(outs[0], outs[1])
    nm.nm_check_status()


# ---- host-operand entry point ------------------------------------------------------------------------------

def test_matmul_host_operands(nm):
    M, K, N = 2, 7168, 576
    A, B = gen.narrow_bf16(M, K, N, seed=800)
    A_host = torch.from_numpy(A.view(np.int16).copy()).pin_memory()
    C_host = torch.zeros(M * N, dtype=torch.int16).pin_memory()
    dB = to_dev(B)
    dA = torch.empty(M * K, dtype=torch.int16, device="cuda")
    dC = torch.empty(M * N, dtype=torch.int16, device="cuda")
    ws = nm.new_workspace(nm.nm_matmul_workspace_bytes(M, N, K))
    nm.nm_matmul_host(A_host, dB, C_host, dA, dC, M, N, K, BF16, ROW, ws)
    torch.cuda.synchronize()
    Cq, C64, bound = oracle.matmul(A, B, M, N, K, oracle.BF16, oracle.BF16, ROW, threads=8)
    assert_matmul_close(oracle.bf16_to_f64(C_host.numpy().view(np.uint16)), Cq, C64, bound, BF16, "host operands")


# ---- error behaviour (host-side only; nothing is enqueued) --------------------------------------------------

def test_error_codes(nm):
    A = torch.zeros(16 * 64, dtype=torch.int16, device="cuda")
    B = torch.zeros(64 * 64, dtype=torch.int16, device="cuda")
    Cb = torch.zeros(16 * 64, dtype=torch.int16, device="cuda")
    def status(fn, *a):
        try:
            fn(*a)
            return 0
        except nm.NmError as e:
            return e.status
    assert status(nm.nm_matmul, A, B, Cb, 0, 64, 64, BF16, ROW) == -1
    assert status(nm.nm_matmul, A, B, Cb, 65, 64, 64, BF16, ROW) == -1
    assert status(nm.nm_matmul, A, B, Cb, 1, 0, 64, BF16, ROW) == -1
    assert status(nm.nm_matmul, None, B, Cb, 1, 64, 64, BF16, ROW) == -1
    assert status(nm.nm_matmul, A, B, Cb, 1, 64, 64, 9, ROW) == -2
    assert status(nm.nm_matmul, A, B, Cb, 1, 64, 64, BF16, 5) == -2
    assert status(nm.nm_matmul, A.data_ptr() + 1, B, Cb, 1, 64, 64, BF16, ROW) == -3
    # split-K without a workspace
    nm.nm_debug_set_plan(0, 4)
    try:
        assert status(nm.nm_matmul_ws, A, B, Cb, 1, 64, 64, BF16, ROW, None) == -4
    finally:
        nm.nm_debug_set_plan(0, 0)
    torch.cuda.synchronize()
