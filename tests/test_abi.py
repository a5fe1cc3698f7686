"""CPU-side checks of the C-ABI library: it loads, exports every symbol the public headers
declare, and its host-only logic (status strings, workspace sizing, tiling plans, argument
validation that needs no device) behaves.  No kernel is launched here."""
import ctypes
import glob
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_16009_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_functions():
    names = []
    for h in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = open(h).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(nm_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "nm_matmul" in names and "nm_matmul_batched" in names
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, f"declared in include/ but not exported: {missing}"


def test_the_debug_build_exports_the_same_symbols():
    """libnm_check.so (-DNM_BOUNDS_CHECK) is the same library with checked accesses: same entry points, and it says so."""
    from paper_2609_16009_b200 import build
    check = ctypes.CDLL(build.build(check=True))
    missing = [n for n in declared_functions() if not hasattr(check, n)]
    assert not missing, missing
    assert check.nm_debug_bounds_checked() == 1
    check.nm_status_string.restype = ctypes.c_char_p
    assert b"outside its operand" in check.nm_status_string(-8)


def test_status_strings_and_version(lib):
    lib.nm_status_string.restype = ctypes.c_char_p
    assert lib.nm_version() >= 100
    assert lib.nm_status_string(0) == b"ok"
    seen = {lib.nm_status_string(-i) for i in range(1, 9)}
    assert len(seen) == 8 and b"unknown status" not in seen
    assert lib.nm_debug_bounds_checked() == 0
    assert lib.nm_status_string(-99) == b"unknown status"


def test_workspace_bound_covers_every_plan(lib):
    lib.nm_matmul_workspace_bytes.restype = ctypes.c_size_t
    out = (ctypes.c_int * 6)()
    for M in (1, 3, 16):
        for (N, K, H) in ((576, 7168, 1), (1536, 7168, 1), (24576, 1536, 1), (512, 128, 128), (8, 100000, 1), (7168, 16384, 1)):
            for layout in (0, 1):
                for tile_n, nsplit in ((0, 0), (64, 64), (2048, 64), (8, 64), (136, 7)):
                    assert lib.nm_debug_set_plan(tile_n, nsplit) == 0
                    assert lib.nm_debug_get_plan(M, N, K, H, 1, layout, 1, out) == 0
                    kind, tn, ns, kr, tiles, ctas = list(out)
                    assert 1 <= ns <= 64 and kr % 8 == 0 and (ns - 1) * kr < K <= ns * kr
                    assert tiles * tn >= N > (tiles - 1) * tn
                    need = 65536 + (H * tiles * ns * M * tn * 4 if ns > 1 else 0)
                    assert need <= lib.nm_matmul_workspace_bytes(M, N, K, H, 1, layout)
    lib.nm_debug_set_plan(0, 0)


def test_heuristic_spreads_the_paper_shape_over_the_gpu(lib):
    out = (ctypes.c_int * 6)()
    lib.nm_debug_set_plan(0, 0)
    for layout in (0, 1):
        assert lib.nm_debug_get_plan(1, 576, 7168, 1, 1, layout, 1, out) == 0
        if layout == 0:
            # row-major: eight k-splits per column tile, the most that can meet inside a thread-block cluster
            # (measured 5.4 us against 7.3 us for 14 splits gathered through the workspace)
            assert out[2] == 8 and out[5] == 72
        else:
            # column-major: measured optimum on B200 is 108-144 CTAs: enough splits to use most SMs, few enough
            # that the gather of the partial sums stays short
            assert 100 <= out[5] <= 320, "MatMul 2 shape must be split over most of the 148 SMs"
    # a shape that cannot use 16-byte loads falls back to the scalar kernel, unsplit
    assert lib.nm_debug_get_plan(1, 577, 7168, 1, 1, 0, 0, out) == 0
    assert out[0] == 2 and out[2] == 1


def test_argument_validation_needs_no_device(lib):
    vp = ctypes.c_void_p
    lib.nm_matmul.argtypes = [vp, vp, vp] + [ctypes.c_int] * 5 + [vp]
    assert lib.nm_matmul(None, None, None, 1, 8, 8, 1, 0, None) == -1
    assert lib.nm_matmul(vp(256), vp(512), vp(1024), 0, 8, 8, 1, 0, None) == -1
    assert lib.nm_matmul(vp(256), vp(512), vp(1024), 65, 8, 8, 1, 0, None) == -1
    # 17 to 64 rows: only operands the tensor-core kernel takes (bf16, tensor maps available); fp32 is refused
    assert lib.nm_matmul(vp(256), vp(512), vp(1024), 17, 8, 8, 0, 0, None) == -2
    assert lib.nm_matmul(vp(256), vp(512), vp(1024), 1, 8, 8, 7, 0, None) == -2
    assert lib.nm_matmul(vp(257), vp(512), vp(1024), 1, 8, 8, 1, 0, None) == -3
    assert lib.nm_set_workspace(vp(4096), ctypes.c_size_t(16)) == -4


def test_tuning_state_is_safe_under_concurrent_host_threads(lib):
    """Two threads ask for plans while a third flips the forced plan between two settings: every answer must be one of
    the two plans in full (never the tile width of one with the split count of the other), and nothing crashes."""
    import threading
    M, N, K = 4, 4096, 8192
    out0 = (ctypes.c_int * 6)()
    settings = ((64, 4), (128, 2))
    want = set()
    for tn, ns in settings:
        assert lib.nm_debug_set_plan(tn, ns) == 0
        assert lib.nm_debug_set_kernel(3, 0) == 0
        assert lib.nm_debug_get_plan(M, N, K, 1, 1, 0, 1, out0) == 0
        want.add(tuple(out0))
    assert len(want) == 2
    stop = threading.Event()
    seen, errors = [set(), set()], []

    def flipper():
        i = 0
        while not stop.is_set():
            lib.nm_debug_set_plan(*settings[i & 1])
            i += 1

    def reader(slot):
        out = (ctypes.c_int * 6)()
        for _ in range(20000):
            if lib.nm_debug_get_plan(M, N, K, 1, 1, 0, 1, out) != 0:
                errors.append("status")
            seen[slot].add(tuple(out))

    threads = [threading.Thread(target=flipper)] + [threading.Thread(target=reader, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads[1:]:
        t.join()
    stop.set()
    threads[0].join()
    lib.nm_debug_set_plan(0, 0)
    lib.nm_debug_set_kernel(-1, 0)
    assert not errors
    for s_ in seen:
        assert s_ <= want, f"torn plan: {s_ - want}"


def test_environment_gives_the_tuning_settings_their_initial_values():
    """NM_TILE_N / NM_SPLITK / NM_FORCE_KERNEL / NM_STAGES are read when the library is loaded (a fresh process here)."""
    import subprocess
    import sys
    code = ("import ctypes, sys; lib = ctypes.CDLL(sys.argv[1]); out = (ctypes.c_int * 6)();"
            "assert lib.nm_debug_get_plan(1, 4096, 8192, 1, 1, 0, 1, out) == 0; print(list(out))")
    from paper_2609_16009_b200 import build
    path = build.build()
    env = dict(os.environ, NM_TILE_N="64", NM_SPLITK="3", NM_FORCE_KERNEL="3")
    forced = subprocess.run([sys.executable, "-c", code, path], env=env, capture_output=True, text=True, check=True).stdout
    kind, tn, ns = eval(forced)[:3]
    assert (kind, tn, ns) == (3, 64, 3), forced
    plain = subprocess.run([sys.executable, "-c", code, path], env={k: v for k, v in os.environ.items() if not k.startswith("NM_")},
                           capture_output=True, text=True, check=True).stdout
    assert eval(plain)[:3] != [3, 64, 3]
