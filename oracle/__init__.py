"""CPU oracle (test infrastructure, not product code).

Loads ``nm_oracle.c`` (plain C, fp64 accumulation, built with gcc) through ctypes and
exposes numpy-level wrappers.  Nothing here is shared with, imported by, or imports the
CUDA path.  bf16 (and fp16) tensors travel as ``numpy.uint16`` bit patterns.

Only tests, the smoke check and the bench's CPU-baseline leg may import this package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nm_oracle.c")
_LIB = os.path.join(_HERE, "libnm_oracle.so")

F32, BF16, F16, F64 = 0, 1, 2, 3
ROW_MAJOR, COL_MAJOR, FRACTAL_NZ = 0, 1, 2

_np_dtype = {F32: np.float32, BF16: np.uint16, F16: np.uint16, F64: np.float64}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.nmo_bf16_to_f64.restype = C.c_double
        _lib.nmo_bf16_to_f64.argtypes = [C.c_uint16]
        _lib.nmo_f64_to_bf16.restype = C.c_uint16
        _lib.nmo_f64_to_bf16.argtypes = [C.c_double]
        _lib.nmo_max_threads.restype = C.c_int
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def max_threads() -> int:
    return int(lib().nmo_max_threads())


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    lib().nmo_widen(_ptr(bits), _ptr(out), C.c_long(bits.size), C.c_int(BF16))
    return out


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().nmo_round(_ptr(x), _ptr(out), C.c_long(x.size), C.c_int(BF16))
    return out


def f16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    lib().nmo_widen(_ptr(bits), _ptr(out), C.c_long(bits.size), C.c_int(F16))
    return out


def f64_to_f16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().nmo_round(_ptr(x), _ptr(out), C.c_long(x.size), C.c_int(F16))
    return out


def widen(a: np.ndarray, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=_np_dtype[dtype])
    out = np.empty(a.shape, dtype=np.float64)
    lib().nmo_widen(_ptr(a), _ptr(out), C.c_long(a.size), C.c_int(dtype))
    return out


def matmul(A, B, M, N, K, in_dtype, out_dtype, layout_B=ROW_MAJOR, threads=1):
    """C = A*B by the definition.  Returns (C rounded once to out_dtype, C in fp64, bound)."""
    A = np.ascontiguousarray(A, dtype=_np_dtype[in_dtype])
    B = np.ascontiguousarray(B, dtype=_np_dtype[in_dtype])
    assert A.size == M * K and B.size == K * N
    Cq = np.empty((M, N), dtype=_np_dtype[out_dtype])
    C64 = np.empty((M, N), dtype=np.float64)
    bound = np.empty((M, N), dtype=np.float64)
    lib().nmo_matmul(_ptr(A), _ptr(B), _ptr(Cq), _ptr(C64), _ptr(bound), C.c_int(M), C.c_int(N),
                     C.c_int(K), C.c_int(in_dtype), C.c_int(out_dtype), C.c_int(layout_B),
                     C.c_int(threads))
    return Cq, C64, bound


def matmul_columns(A, B, M, N, K, cols, in_dtype, out_dtype, layout_B=ROW_MAJOR):
    """The same definition evaluated only at the output columns ``cols`` (sampled parity at
    full size).  Each sampled column is one call on a 1-column view of B."""
    A = np.ascontiguousarray(A, dtype=_np_dtype[in_dtype])
    B = np.ascontiguousarray(B, dtype=_np_dtype[in_dtype]).reshape(-1)
    esz = A.dtype.itemsize
    cols = list(cols)
    Cq = np.empty((M, len(cols)), dtype=_np_dtype[out_dtype])
    C64 = np.empty((M, len(cols)), dtype=np.float64)
    bound = np.empty((M, len(cols)), dtype=np.float64)
    cq1 = np.empty((M, 1), dtype=_np_dtype[out_dtype])
    c1 = np.empty((M, 1), dtype=np.float64)
    b1 = np.empty((M, 1), dtype=np.float64)
    for j, n in enumerate(cols):
        if layout_B == ROW_MAJOR:
            base, ldb = B.ctypes.data + n * esz, N
        else:
            base, ldb = B.ctypes.data + n * K * esz, K
        lib().nmo_matmul_strided(_ptr(A), C.c_void_p(base), _ptr(cq1), _ptr(c1), _ptr(b1),
                                 C.c_int(M), C.c_int(1), C.c_int(K), C.c_long(K), C.c_long(ldb),
                                 C.c_long(1), C.c_int(in_dtype), C.c_int(out_dtype),
                                 C.c_int(layout_B), C.c_int(1))
        Cq[:, j], C64[:, j], bound[:, j] = cq1[:, 0], c1[:, 0], b1[:, 0]
    return Cq, C64, bound


def matmul_batched(A, B, M, N, K, H, lda, strideA, strideB, ldc, strideC, c_elems,
                   in_dtype, out_dtype, layout_B=ROW_MAJOR, threads=1):
    """H independent products with the strided addressing of the per-head call.
    ``c_elems`` is the number of elements of the C buffer.  Returns (C, C64, bound), flat."""
    A = np.ascontiguousarray(A, dtype=_np_dtype[in_dtype])
    B = np.ascontiguousarray(B, dtype=_np_dtype[in_dtype])
    Cq = np.zeros(c_elems, dtype=_np_dtype[out_dtype])
    C64 = np.zeros(c_elems, dtype=np.float64)
    bound = np.zeros(c_elems, dtype=np.float64)
    lib().nmo_matmul_batched(_ptr(A), _ptr(B), _ptr(Cq), _ptr(C64), _ptr(bound), C.c_int(M),
                             C.c_int(N), C.c_int(K), C.c_int(H), C.c_long(lda), C.c_long(strideA),
                             C.c_long(strideB), C.c_long(ldc), C.c_long(strideC),
                             C.c_int(in_dtype), C.c_int(out_dtype), C.c_int(layout_B),
                             C.c_int(threads))
    return Cq, C64, bound


def rmsnorm(x, gamma, eps):
    x = np.ascontiguousarray(x, dtype=np.float64)
    gamma = np.ascontiguousarray(gamma, dtype=np.float64)
    y = np.empty_like(x)
    lib().nmo_rmsnorm(_ptr(x), _ptr(gamma), _ptr(y), C.c_int(x.size), C.c_double(eps))
    return y


def rope(x, pos, base=10000.0):
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    lib().nmo_rope(_ptr(x), _ptr(y), C.c_int(x.size), C.c_long(pos), C.c_double(base))
    return y


def mla_attention(Q, cache, dv, scale, threads=1, want_p=False):
    """Q [H, dqk], cache [S, dqk] in fp64.  Returns o [H, dv] (and p [H, S])."""
    Q = np.ascontiguousarray(Q, dtype=np.float64)
    cache = np.ascontiguousarray(cache, dtype=np.float64)
    H, dqk = Q.shape
    S = cache.shape[0]
    assert cache.shape[1] == dqk
    O = np.empty((H, dv), dtype=np.float64)
    P = np.empty((H, S), dtype=np.float64) if want_p else None
    lib().nmo_mla_attention(_ptr(Q), _ptr(cache), _ptr(O), _ptr(P), C.c_int(H), C.c_int(S),
                            C.c_int(dqk), C.c_int(dv), C.c_double(scale), C.c_int(threads))
    return (O, P) if want_p else O


class _MlaParams(C.Structure):
    _fields_ = ([(n, C.c_int) for n in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H",
                                        "seq_len", "layout_dense", "threads")]
                + [(n, C.c_double) for n in ("rms_eps", "softmax_scale", "rope_base")]
                + [(n, C.c_void_p) for n in ("h", "W_DQ", "gamma_q", "W_UQR", "W_DKVKR", "gamma_kv",
                                             "W_UK", "W_UV", "W_O", "kv_cache",
                                             "c_q", "c_qn", "q", "q_rope", "ckr", "q_lat", "o_lat",
                                             "o", "out",
                                             "o_lat_f64", "bound_c_q", "bound_q", "bound_ckr",
                                             "bound_q_lat", "bound_o", "bound_out")])


def mla_decode_step(dims: dict, w: dict, h, kv_cache, seq_len, rms_eps=1e-6, softmax_scale=None,
                    rope_base=10000.0, layout_dense=ROW_MAJOR, threads=1):
    """Naive eleven-stage decode step.  ``dims`` has d, q_lora, kv_lora, rope, nope, v, H;
    ``w`` has the bf16 (uint16) weights W_DQ, gamma_q, W_UQR, W_DKVKR, gamma_kv, W_UK, W_UV and
    optionally W_O.  ``kv_cache`` ([>=seq_len, kv_lora+rope] uint16) gets row seq_len-1 written in
    place.  Returns a dict with every stage output (uint16), the unrounded ``o_lat_f64`` and the
    per-element matmul bounds."""
    d, ql, dc, dr, dn, dv, H = (dims[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
    if softmax_scale is None:
        softmax_scale = 1.0 / np.sqrt(dn + dr)
    p = _MlaParams()
    for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"):
        setattr(p, k, int(dims[k]))
    p.seq_len, p.layout_dense, p.threads = int(seq_len), int(layout_dense), int(threads)
    p.rms_eps, p.softmax_scale, p.rope_base = float(rms_eps), float(softmax_scale), float(rope_base)
    keep = []

    def inp(name, arr):
        a = np.ascontiguousarray(arr, dtype=np.uint16)
        keep.append(a)
        setattr(p, name, a.ctypes.data)

    inp("h", h)
    for k in ("W_DQ", "gamma_q", "W_UQR", "W_DKVKR", "gamma_kv", "W_UK", "W_UV"):
        inp(k, w[k])
    if w.get("W_O") is not None:
        inp("W_O", w["W_O"])
    assert kv_cache.dtype == np.uint16 and kv_cache.flags.c_contiguous
    assert kv_cache.shape[0] >= seq_len and kv_cache.shape[1] == dc + dr
    p.kv_cache = kv_cache.ctypes.data
    out = {}
    shapes = {"c_q": (ql,), "c_qn": (ql,), "q": (H, dn + dr), "q_rope": (H, dr), "ckr": (dc + dr,),
              "q_lat": (H, dc), "o_lat": (H, dc), "o": (H, dv), "out": (d,)}
    for k, shp in shapes.items():
        out[k] = np.zeros(shp, dtype=np.uint16)
        setattr(p, k, out[k].ctypes.data)
    f64s = {"o_lat_f64": (H, dc), "bound_c_q": (ql,), "bound_q": (H, dn + dr), "bound_ckr": (dc + dr,),
            "bound_q_lat": (H, dc), "bound_o": (H, dv), "bound_out": (d,)}
    for k, shp in f64s.items():
        out[k] = np.zeros(shp, dtype=np.float64)
        setattr(p, k, out[k].ctypes.data)
    rc = lib().nmo_mla_decode_step(C.byref(p))
    if rc != 0:
        raise RuntimeError(f"nmo_mla_decode_step failed: {rc}")
    if w.get("W_O") is None:
        out.pop("out"), out.pop("bound_out")
    return out


def ulp_f16(x: np.ndarray) -> np.ndarray:
    """Spacing of the fp16 grid at |x| (2^(floor(log2|x|) - 10); 2^-24 throughout the subnormal range)."""
    ax = np.abs(np.asarray(x, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(ax, 2.0 ** -14)))
    return np.exp2(e - 10)


def ulp_bf16(x: np.ndarray) -> np.ndarray:
    """Spacing of the bf16 grid at |x| (2^(floor(log2|x|) - 7); smallest normal binade below that)."""
    ax = np.abs(np.asarray(x, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(ax, 2.0 ** -126)))
    return np.exp2(e - 7)
