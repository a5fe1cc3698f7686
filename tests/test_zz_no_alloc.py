"""nm_matmul_static, the entry point for callers that cannot allocate device memory.

Some users of this library run where nobody can give it a workspace: their GPU memory was claimed
up front by another pool, or an allocation (which synchronises the device) is not acceptable in
their loop.  For them the split-K scratch sits in a fixed array inside the library.  This test calls
that entry point through the C ABI and checks it against nm_matmul_ws (caller-provided workspace),
twice in a row so that the second call starts from whatever the first one left in the array.

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
from gpu_util import out_to_f64, to_dev

pytestmark = pytest.mark.gpu

BF16, BF16_F32OUT, ROW, COL = 1, 2, 0, 1


def _both(nm, M, N, K, dtype, layout, seed):
    A, B = gen.narrow_bf16(M, K, N, seed)
    Bst = B if layout == ROW else gen.to_col_major(B)
    dA, dB = to_dev(A), to_dev(Bst)
    tdt = torch.int16 if dtype == BF16 else torch.float32
    c_static = torch.zeros(M * N, dtype=tdt, device="cuda")
    c_ws = torch.zeros(M * N, dtype=tdt, device="cuda")
    ws = nm.new_workspace(nm.nm_matmul_workspace_bytes(M, N, K))
    assert nm.nm_debug_get_plan(M, N, K, 1, dtype, layout)["nsplit"] > 1, "case must exercise the scratch"
    nm.nm_matmul_static(dA, dB, c_static, M, N, K, dtype, layout)
    nm.nm_matmul_ws(dA, dB, c_ws, M, N, K, dtype, layout, ws)
    torch.cuda.synchronize()
    # same tolerance as the parity tests: 1e-5 * sum|a*b| + 1e-6 (+ one bf16 ulp for bf16 outputs)
    _, C64, bound = oracle.matmul(A, Bst, M, N, K, oracle.BF16, oracle.F32, layout, threads=8)
    tol = 1e-5 * bound + 1e-6 + (oracle.ulp_bf16(C64) if dtype == BF16 else 0.0)
    got, ref = out_to_f64(c_static, dtype).reshape(M, N), out_to_f64(c_ws, dtype).reshape(M, N)
    assert np.all(np.abs(got - ref) <= tol), f"static vs workspace differ: max {np.abs(got - ref).max()}"
    assert np.all(np.abs(got - C64) <= tol + (oracle.ulp_bf16(C64) if dtype == BF16 else 0.0))


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    import paper_2609_16009_b200 as nm
    nm.nm_debug_set_plan(0, 0)
    nm.nm_debug_set_kernel(-1, 0)
    # with the k-splits gathered through the scratch array (the case this entry point exists for), then as the
    # library runs by default (up to eight splits meet inside a cluster and leave the array alone)
    for cluster in (False, True):
        nm.nm_debug_set_cluster_split(cluster)
        try:
            # first call: the paper's MatMul 2 shape; second call: another shape, layout and M, reusing the array
            _both(nm, 1, 576, 7168, BF16, ROW, seed=9100)
            _both(nm, 3, 1536, 7168, BF16_F32OUT, COL, seed=9200)
            _both(nm, 1, 576, 7168, BF16, ROW, seed=9300)
        finally:
            nm.nm_debug_set_cluster_split(True)
    nm.nm_check_status()


def test_static_scratch_refuses_problems_beyond_its_size():
    import paper_2609_16009_b200 as nm
    M, N, K = 16, 8192, 8192
    A = torch.zeros(M * K, dtype=torch.int16, device="cuda")
    B = torch.zeros(8, dtype=torch.int16, device="cuda")      # never read: the call must be refused
    C = torch.zeros(M * N, dtype=torch.int16, device="cuda")
    nm.nm_debug_set_plan(64, 64)                               # 64 k-splits: 32 MB of partial sums
    try:
        with pytest.raises(nm.NmError) as e:
            nm.nm_matmul_static(A, B, C, M, N, K, BF16, ROW)
        assert e.value.status == -7
    finally:
        nm.nm_debug_set_plan(0, 0)
    torch.cuda.synchronize()
