"""The debug build of the library (libnm_check.so, -DNM_BOUNDS_CHECK): the narrow-product kernels check every
hand-indexed global access against the extent of the operand it belongs to, report an access outside it in the device
status word and skip it.  Here: the mechanism itself (an address outside the named span but inside the caller's buffer,
so nothing can fault), and a sweep of ragged shapes, layouts, element types, forced kernels and k-splits that must come
out clean and bit-identical to the normal library - which is what shows that the kernels' index arithmetic stays inside
A, B, C and the workspace for those shapes, reads included (canaries only see writes)."""
import ctypes as C
import os

import numpy as np
import pytest
import torch

import nm_inputs as gen
from gpu_util import to_dev

pytestmark = pytest.mark.gpu

F32, BF16, BF16_F32OUT, F16 = 0, 1, 2, 3
ROW, COL = 0, 1
NM_ERR_BOUNDS, NM_ERR_UNSUPPORTED = -8, -2
_vp, _i, _sz = C.c_void_p, C.c_int, C.c_size_t


def _declare(lib):
    lib.nm_matmul_ws.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _sz, _vp]
    lib.nm_workspace_init.argtypes = [_vp, _sz, _vp]
    lib.nm_matmul_workspace_bytes.argtypes = [_i, _i, _i, _i, _i, _i]
    lib.nm_matmul_workspace_bytes.restype = _sz
    lib.nm_check_status.argtypes = [_vp]
    lib.nm_debug_bounds_selftest.argtypes = [_vp, _sz, _vp, _vp]
    lib.nm_debug_set_kernel.argtypes = [_i, _i]
    lib.nm_debug_set_plan.argtypes = [_i, _i]
    return lib


@pytest.fixture(scope="module")
def libs():
    import paper_2609_16009_b200 as nm
    from paper_2609_16009_b200 import build
    normal = _declare(C.CDLL(nm.LIB_PATH))
    check = _declare(C.CDLL(build.build(check=True)))
    assert normal.nm_debug_bounds_checked() == 0 and check.nm_debug_bounds_checked() == 1
    yield normal, check
    for lib in (normal, check):
        lib.nm_debug_set_kernel(-1, 0)
        lib.nm_debug_set_plan(0, 0)
        assert lib.nm_check_status(None) == 0


def test_an_access_outside_its_operand_is_reported_and_skipped(libs):
    normal, check = libs
    buf = torch.full((16,), 0x11111111, dtype=torch.int32, device="cuda")          # 64 bytes; the operand named is the first 32
    loaded = torch.full((2,), 0x7777, dtype=torch.int32, device="cuda")
    assert check.nm_check_status(None) == 0
    assert check.nm_debug_bounds_selftest(buf.data_ptr(), 64, loaded.data_ptr(), None) == 0
    assert check.nm_check_status(None) == NM_ERR_BOUNDS                             # reported ...
    assert check.nm_check_status(None) == 0                                         # ... once
    b = buf.cpu().numpy().view(np.uint32)
    assert b[8] == 0x11111111 and np.all(b[1:] == 0x11111111)                       # the store outside did not happen
    assert b[0] == 0x600DF00D                                                       # the one inside did
    assert loaded.cpu().numpy().view(np.uint32).tolist() == [0, 0x600DF00D]         # the load outside gave zero
    assert normal.nm_debug_bounds_selftest(buf.data_ptr(), 64, loaded.data_ptr(), None) == NM_ERR_UNSUPPORTED


CASES = [  # dtype, layout, M, K, N, forced kernel (-1 planner, 0 row, 3 TMA ring, 4 tensor cores), forced k-splits
    (F32, ROW, 1, 512, 512, -1, 0), (F32, COL, 3, 5, 7, -1, 0), (F32, ROW, 16, 77, 1, -1, 0), (F32, COL, 2, 1023, 259, -1, 3),
    (BF16, ROW, 1, 1, 1, -1, 0), (BF16, COL, 5, 1023, 259, -1, 0), (BF16, ROW, 7, 8, 2048, 0, 0), (BF16, ROW, 16, 2600, 72, 0, 5),
    (BF16, ROW, 1, 7168, 576, -1, 0), (BF16, COL, 1, 7168, 576, -1, 0), (BF16, ROW, 2, 1000, 840, 3, 3), (BF16, ROW, 9, 1000, 840, 3, 0),
    (BF16, ROW, 1, 1001, 840, -1, 0), (BF16, ROW, 4, 1536, 4104, 4, 2), (BF16, COL, 16, 2048, 1160, 4, 0), (BF16, ROW, 40, 640, 520, -1, 0),
    (BF16_F32OUT, ROW, 3, 129, 33, -1, 0), (BF16_F32OUT, COL, 6, 4096, 264, -1, 16),
    (F16, ROW, 2, 129, 33, -1, 0), (F16, COL, 4, 1000, 840, -1, 3), (F16, ROW, 16, 1536, 4104, 4, 0), (F16, ROW, 5, 777, 31, -1, 0),
]


@pytest.mark.parametrize("dtype,layout,M,K,N,kernel,nsplit", CASES)
def test_checked_build_is_clean_and_bit_identical(libs, dtype, layout, M, K, N, kernel, nsplit):
    normal, check = libs
    seed = 9000 + M + K + N
    if dtype == F32:
        A, B = gen.uniform_f32((M, K), -1, 1, seed), gen.uniform_f32((K, N), -1, 1, seed + 1)
    elif dtype == F16:
        A, B = gen.narrow_f16(M, K, N, seed)
    else:
        A, B = gen.narrow_bf16(M, K, N, seed)
    if layout == COL:
        B = gen.to_col_major(B)
    dA, dB = to_dev(A), to_dev(B)
    out_t = torch.int16 if dtype in (BF16, F16) else torch.float32
    results = []
    for lib in (normal, check):
        nbytes = lib.nm_matmul_workspace_bytes(M, N, K, 1, dtype, layout)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        assert lib.nm_workspace_init(ws.data_ptr(), nbytes, None) == 0
        Cd = torch.zeros(M * N, dtype=out_t, device="cuda")
        assert lib.nm_debug_set_kernel(kernel, 0) == 0 and lib.nm_debug_set_plan(0, nsplit) == 0
        try:
            rc = lib.nm_matmul_ws(dA.data_ptr(), dB.data_ptr(), Cd.data_ptr(), M, N, K, dtype, layout, ws.data_ptr(), nbytes, None)
        finally:
            lib.nm_debug_set_kernel(-1, 0)
            lib.nm_debug_set_plan(0, 0)
        assert rc == 0, rc
        assert lib.nm_check_status(None) == 0, "an access outside its operand (or an expired wait) was reported"
        results.append(Cd.clone())
    assert torch.equal(results[0], results[1]), "the checked build computes different bits"
