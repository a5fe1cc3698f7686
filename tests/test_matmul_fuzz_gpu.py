"""Randomised parity of the narrow product against the oracle: shapes, row counts, layouts, element types, forced
kernels and k-splits drawn from a seeded generator (every case is reproducible from its seed).  Sizes are small
enough for the oracle to evaluate every element; ragged K and N, unaligned strides-in-effect (odd N / K send the
call to the scalar kernel), up to 64 rows, and the three storages of B are all in the mix."""
import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
from gpu_util import guards_intact, out_buffer, out_to_f64, to_dev, assert_matmul_close

pytestmark = pytest.mark.gpu

F32, BF16, BF16_F32OUT = 0, 1, 2
ROW, COL, NZ = 0, 1, 2
ORACLE_IN = {F32: oracle.F32, BF16: oracle.BF16, BF16_F32OUT: oracle.BF16}
ORACLE_OUT = {F32: oracle.F32, BF16: oracle.BF16, BF16_F32OUT: oracle.F32}


@pytest.fixture(scope="module")
def nm():
    import paper_2609_16009_b200 as nm
    ws = nm.new_workspace(64 << 20)
    nm.nm_set_workspace(ws)
    yield nm
    nm.nm_debug_set_plan(0, 0)
    nm.nm_debug_set_kernel(-1, 0)
    nm.nm_debug_set_cluster_split(True)
    nm.nm_check_status()
    nm.nm_set_workspace(None)


def draw_case(seed):
    rng = np.random.default_rng(10_000 + seed)
    dtype = int(rng.choice([F32, BF16, BF16, BF16, BF16_F32OUT]))
    layout = int(rng.choice([ROW, ROW, COL, NZ])) if dtype != F32 else int(rng.choice([ROW, COL]))
    if layout == NZ:
        K, N = 16 * int(rng.integers(1, 80)), 16 * int(rng.integers(1, 70))
        M = int(rng.integers(1, 17))
    else:
        unit = int(rng.choice([1, 8, 8, 16, 64]))
        K, N = unit * int(rng.integers(1, 1400 // unit + 2)), unit * int(rng.integers(1, 1200 // unit + 2))
        aligned = dtype != F32 and K % 8 == 0 and N % 8 == 0
        M = int(rng.integers(1, 65)) if aligned and rng.random() < 0.3 else int(rng.integers(1, 17))
    nsplit = int(rng.choice([0, 0, 1, 2, 3, 5, 8, 9]))
    tile_n = int(rng.choice([0, 0, 64, 128, 256]))
    kernel = int(rng.choice([-1, -1, -1, 0, 3, 4])) if M <= 16 else -1
    cluster = bool(rng.random() < 0.7)
    return dtype, layout, M, K, N, nsplit, tile_n, kernel, cluster


@pytest.mark.parametrize("seed", range(400))
def test_random_case_matches_the_oracle(nm, seed):
    dtype, layout, M, K, N, nsplit, tile_n, kernel, cluster = draw_case(seed)
    if dtype == F32:
        A, B = gen.uniform_f32((M, K), -1, 1, 20_000 + seed), gen.uniform_f32((K, N), -1, 1, 30_000 + seed)
    else:
        A, B = gen.narrow_bf16(M, K, N, 20_000 + seed)
    Bst = B if layout == ROW else (gen.to_col_major(B) if layout == COL else gen.to_fractal_nz(B))
    dA, dB = to_dev(A), to_dev(Bst)
    whole, dC = out_buffer(M * N, dtype)
    what = f"seed {seed}: dtype {dtype} layout {layout} M {M} K {K} N {N} nsplit {nsplit} tile_n {tile_n} kernel {kernel} cluster {cluster}"
    nm.nm_debug_set_plan(tile_n, nsplit)
    nm.nm_debug_set_kernel(kernel, 0)
    nm.nm_debug_set_cluster_split(cluster)
    try:
        nm.nm_matmul(dA, dB, dC, M, N, K, dtype, layout)
        torch.cuda.synchronize()
    finally:
        nm.nm_debug_set_plan(0, 0)
        nm.nm_debug_set_kernel(-1, 0)
        nm.nm_debug_set_cluster_split(True)
    assert guards_intact(whole, M * N, dtype), what
    Cq, C64, bound = oracle.matmul(A, Bst, M, N, K, ORACLE_IN[dtype], ORACLE_OUT[dtype], layout, threads=8)
    assert_matmul_close(out_to_f64(dC, dtype).reshape(M, N), Cq, C64, bound, dtype, what)
    nm.nm_check_status()
