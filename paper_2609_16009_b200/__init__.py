"""Thin Python binding over the C-ABI library ``libnm.so`` (argument marshalling only).

Every function has the name of the C entry point it calls.  Tensors are ``torch`` CUDA tensors
used purely as device memory: bf16 data may be passed as ``torch.bfloat16`` or as its raw
``int16``/``uint16`` bits.  There is no CPU path: importing this package without the built
library raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libnm.so")

F32, BF16, BF16_F32OUT, F16 = 0, 1, 2, 3
ROW_MAJOR, COL_MAJOR, FRACTAL_NZ = 0, 1, 2
MAX_M = 16
WS_COUNTER_BYTES = 65536

if not os.path.exists(LIB_PATH):
    # No CPU fallback exists: either the library gets built here (nvcc present) or the import fails.
    try:
        import importlib.util as _ilu
        _spec = _ilu.spec_from_file_location("_nm_build", os.path.join(_PKG, "build.py"))
        _build = _ilu.module_from_spec(_spec)
        _spec.loader.exec_module(_build)
        _build.build()
    except Exception as exc:  # noqa: BLE001
        raise ImportError(f"{LIB_PATH} is missing and could not be built with nvcc ({exc}); "
                          "there is no CPU fallback") from exc
_lib = C.CDLL(LIB_PATH)


class NmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.nm_status_string(status).decode()
        cuda = _lib.nm_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})" + (f" [{cuda}]" if status == -5 and cuda else ""))


_vp, _i, _l, _sz = C.c_void_p, C.c_int, C.c_long, C.c_size_t
_lib.nm_version.restype = _i
_lib.nm_status_string.restype = C.c_char_p
_lib.nm_status_string.argtypes = [_i]
_lib.nm_last_cuda_error.restype = C.c_char_p
_lib.nm_matmul_workspace_bytes.restype = _sz
_lib.nm_matmul_workspace_bytes.argtypes = [_i, _i, _i, _i, _i, _i]
_lib.nm_workspace_init.argtypes = [_vp, _sz, _vp]
_lib.nm_set_workspace.argtypes = [_vp, _sz]
_lib.nm_matmul.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]
_lib.nm_matmul_ws.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _sz, _vp]
_lib.nm_matmul_batched.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _l, _l, _l, _l, _l, _i, _i, _vp]
_lib.nm_matmul_batched_ws.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _l, _l, _l, _l, _l, _i, _i, _vp, _sz, _vp]
_lib.nm_matmul_host.argtypes = [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _sz, _vp]
_lib.nm_matmul_static.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp]
_lib.nm_debug_set_plan.argtypes = [_i, _i]
_lib.nm_debug_set_kernel.argtypes = [_i, _i]
_lib.nm_set_tensor_core_min_m.argtypes = [_i]
_lib.nm_set_programmatic_launch.argtypes = [_i]
_lib.nm_check_status.argtypes = [_vp]
_lib.nm_debug_get_plan.argtypes = [_i, _i, _i, _i, _i, _i, _i, C.POINTER(_i)]


class MlaParams(C.Structure):
    """Mirror of nm_mla_params (include/nm.h)."""
    _fields_ = ([(n, _i) for n in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H", "seq_len", "layout_dense")]
                + [("rms_eps", C.c_float), ("softmax_scale", C.c_float)]
                + [(n, _vp) for n in ("h", "W_DQ", "gamma_q", "W_UQR", "W_DKVKR", "gamma_kv", "W_UK", "W_UV", "W_O",
                                      "rope_cos_sin", "kv_cache", "out", "workspace")]
                + [("workspace_bytes", _sz)]
                + [(n, _vp) for n in ("c_q", "c_qn", "q", "q_full", "ckr", "o_lat", "o", "o_lat_f32",
                                      "event_before_wo", "event_after_wo")]
                + [("programmatic_entry", _i), ("W_DQKV", _vp)])


class MlaBatch(C.Structure):
    """Mirror of nm_mla_batch (include/nm.h)."""
    _fields_ = [("T", _i), ("seq_lens", C.POINTER(_i)), ("h", _vp), ("rope_cos_sin", _vp), ("kv_cache", _vp),
                ("cache_stride", C.c_long), ("out", _vp), ("q_full", _vp), ("o_lat", _vp), ("o", _vp),
                ("c_q", _vp), ("c_qn", _vp), ("q", _vp), ("ckr", _vp)]


_lib.nm_mla_batch_workspace_bytes.restype = _sz
_lib.nm_mla_batch_workspace_bytes.argtypes = [C.POINTER(MlaParams), _i]
_lib.nm_mla_decode_batch.argtypes = [C.POINTER(MlaParams), C.POINTER(MlaBatch), _vp]
_lib.nm_rmsnorm.argtypes = [_vp, _vp, _vp, _i, C.c_float, _vp]
_lib.nm_rope.argtypes = [_vp, _vp, _i, _i, _l, _l, _vp, _vp]
_lib.nm_rope_table.argtypes = [_vp, _l, _i, _i, C.c_double, _vp]
_lib.nm_mla_attention_workspace_bytes.restype = _sz
_lib.nm_mla_attention_workspace_bytes.argtypes = [_i, _i, _i]
_lib.nm_mla_attention.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _l, _i, _i, C.c_float, _vp, _sz, _vp]
_lib.nm_mla_attention_partial.argtypes = [_vp, _vp, _i, _i, _i, _i, C.c_float, _vp, _sz, _vp]
_lib.nm_mla_attention_combine.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _l, _i, _i, C.c_float, _vp, _sz, _vp]
_lib.nm_mla_workspace_bytes.restype = _sz
_lib.nm_mla_workspace_bytes.argtypes = [C.POINTER(MlaParams)]
_lib.nm_mla_decode_step.argtypes = [C.POINTER(MlaParams), _vp, _vp]
_lib.nm_mla_decode_step_host.argtypes = [C.POINTER(MlaParams), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.nm_debug_set_attention.argtypes = [_i]
_lib.nm_debug_set_attention_wide.argtypes = [_i, _i, _i]
_lib.nm_debug_set_step_kv_beside_attention.argtypes = [_i]
_lib.nm_debug_bounds_selftest.argtypes = [_vp, _sz, _vp, _vp]
_lib.nm_debug_set_step_pdl.argtypes = [_i]
_lib.nm_debug_stream_read.argtypes = [_vp, _sz, _vp, _i, _vp]
_lib.nm_debug_set_step_knobs.argtypes = [_i, _i]
_lib.nm_debug_set_step_tails.argtypes = [_i]
_lib.nm_debug_set_cluster_split.argtypes = [_i]
_lib.nm_debug_set_batch_per_head_min_tokens.argtypes = [_i]
_lib.nm_debug_set_step_plan.argtypes = [_i, _i, _i, _i]
_lib.nm_debug_set_step_prefetch.argtypes = [_i]
_lib.nm_debug_set_step_fusion.argtypes = [_i]
_lib.nm_debug_set_attention_trace.argtypes = [_vp]
_lib.nm_debug_wait_probe.argtypes = [C.c_ulonglong, _vp, _vp]
_lib.nm_debug_mma_probe.argtypes = [_i] * 8 + [_vp, _vp]


def _check(status: int, where: str) -> None:
    if status != 0:
        raise NmError(status, where)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def nm_version() -> int:
    return _lib.nm_version()


def nm_status_string(status: int) -> str:
    return _lib.nm_status_string(status).decode()


def nm_matmul_workspace_bytes(M, N, K, H=1, dtype=BF16, layout_B=ROW_MAJOR) -> int:
    return int(_lib.nm_matmul_workspace_bytes(M, N, K, H, dtype, layout_B))


def nm_workspace_init(workspace, stream=None) -> None:
    _check(_lib.nm_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _stream(stream)), "nm_workspace_init")


def nm_set_workspace(workspace) -> None:
    if workspace is None:
        _check(_lib.nm_set_workspace(None, 0), "nm_set_workspace")
    else:
        _check(_lib.nm_set_workspace(_ptr(workspace), workspace.numel() * workspace.element_size()),
               "nm_set_workspace")


def nm_matmul(A, B, C_out, M, N, K, dtype, layout_B, stream=None) -> None:
    _check(_lib.nm_matmul(_ptr(A), _ptr(B), _ptr(C_out), M, N, K, dtype, layout_B, _stream(stream)),
           "nm_matmul")


def nm_matmul_ws(A, B, C_out, M, N, K, dtype, layout_B, workspace, stream=None) -> None:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.nm_matmul_ws(_ptr(A), _ptr(B), _ptr(C_out), M, N, K, dtype, layout_B,
                             _ptr(workspace), nbytes, _stream(stream)), "nm_matmul_ws")


def nm_matmul_batched(A, B, C_out, M, N, K, H, lda, strideA, strideB, ldc, strideC, dtype, layout_B,
                      stream=None) -> None:
    _check(_lib.nm_matmul_batched(_ptr(A), _ptr(B), _ptr(C_out), M, N, K, H, lda, strideA, strideB,
                                  ldc, strideC, dtype, layout_B, _stream(stream)), "nm_matmul_batched")


def nm_matmul_batched_ws(A, B, C_out, M, N, K, H, lda, strideA, strideB, ldc, strideC, dtype, layout_B,
                         workspace, stream=None) -> None:
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.nm_matmul_batched_ws(_ptr(A), _ptr(B), _ptr(C_out), M, N, K, H, lda, strideA, strideB,
                                     ldc, strideC, dtype, layout_B, _ptr(workspace), nbytes,
                                     _stream(stream)), "nm_matmul_batched_ws")


def nm_matmul_host(A_host, B, C_host, A_staging, C_staging, M, N, K, dtype, layout_B, workspace,
                   stream=None) -> None:
    """A_host / C_host are pinned CPU tensors; the rest are CUDA tensors."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.nm_matmul_host(_ptr(A_host), _ptr(B), _ptr(C_host), _ptr(A_staging), _ptr(C_staging),
                               M, N, K, dtype, layout_B, _ptr(workspace), nbytes, _stream(stream)),
           "nm_matmul_host")


STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


def nm_matmul_static(A, B, C_out, M, N, K, dtype, layout_B, stream=None) -> None:
    """nm_matmul without any workspace: the scratch is a fixed array inside the library, for
    callers that cannot allocate.  Calls on one GPU must not overlap; the first call on a device
    should come before any stream capture."""
    _check(_lib.nm_matmul_static(_ptr(A), _ptr(B), _ptr(C_out), M, N, K, dtype, layout_B, _stream(stream)),
           "nm_matmul_static")


def nm_debug_set_plan(tile_n: int = 0, nsplit: int = 0) -> None:
    _check(_lib.nm_debug_set_plan(tile_n, nsplit), "nm_debug_set_plan")


def nm_set_tensor_core_min_m(m: int) -> None:
    _check(_lib.nm_set_tensor_core_min_m(int(m)), "nm_set_tensor_core_min_m")


def nm_debug_set_kernel(kind: int = -1, stages: int = 0) -> None:
    _check(_lib.nm_debug_set_kernel(kind, stages), "nm_debug_set_kernel")


def nm_set_programmatic_launch(enable: bool) -> None:
    _check(_lib.nm_set_programmatic_launch(int(enable)), "nm_set_programmatic_launch")


def nm_check_status(stream=None) -> None:
    """Synchronise the stream and raise if a kernel gave up on a bounded wait."""
    _check(_lib.nm_check_status(_stream(stream)), "nm_check_status")


def nm_debug_get_plan(M, N, K, H=1, dtype=BF16, layout_B=ROW_MAJOR, vec_ok=True) -> dict:
    out = (_i * 6)()
    _check(_lib.nm_debug_get_plan(M, N, K, H, dtype, layout_B, int(vec_ok), out), "nm_debug_get_plan")
    return dict(kind=out[0], tile_n=out[1], nsplit=out[2], k_rows=out[3], tiles=out[4], ctas=out[5])


def new_workspace(nbytes: int, device="cuda", stream=None) -> torch.Tensor:
    """Allocate (with torch) and initialise a workspace of at least ``nbytes`` bytes."""
    ws = torch.empty(max(int(nbytes), WS_COUNTER_BYTES), dtype=torch.uint8, device=device)
    nm_workspace_init(ws, stream)
    return ws


# ---- MLA decode step -----------------------------------------------------------------------------------

def nm_rmsnorm(x, gamma, y, n, eps, stream=None) -> None:
    _check(_lib.nm_rmsnorm(_ptr(x), _ptr(gamma), _ptr(y), n, eps, _stream(stream)), "nm_rmsnorm")


def nm_rope(x, y, n_vec, dim, x_stride, y_stride, cos_sin, stream=None) -> None:
    _check(_lib.nm_rope(_ptr(x), _ptr(y), n_vec, dim, x_stride, y_stride, _ptr(cos_sin), _stream(stream)), "nm_rope")


def nm_rope_table(table, pos_begin, n_pos, dim, base=10000.0, stream=None) -> None:
    _check(_lib.nm_rope_table(_ptr(table), pos_begin, n_pos, dim, base, _stream(stream)), "nm_rope_table")


def nm_mla_attention_workspace_bytes(H, n_rows, kv_lora) -> int:
    return int(_lib.nm_mla_attention_workspace_bytes(H, n_rows, kv_lora))


def nm_mla_attention(Q, kv_cache, o_bf16, o_f32, H, n_rows, extra_row, kv_lora, rope, scale, workspace, stream=None) -> None:
    _check(_lib.nm_mla_attention(_ptr(Q), _ptr(kv_cache), _ptr(o_bf16), _ptr(o_f32), H, n_rows, extra_row, kv_lora, rope,
                                 scale, _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "nm_mla_attention")


def nm_mla_attention_partial(Q, kv_cache, H, n_rows, kv_lora, rope, scale, workspace, stream=None) -> None:
    _check(_lib.nm_mla_attention_partial(_ptr(Q), _ptr(kv_cache), H, n_rows, kv_lora, rope, scale, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)),
           "nm_mla_attention_partial")


def nm_mla_attention_combine(Q, kv_cache, o_bf16, o_f32, H, n_rows, extra_row, kv_lora, rope, scale, workspace,
                             stream=None) -> None:
    _check(_lib.nm_mla_attention_combine(_ptr(Q), _ptr(kv_cache), _ptr(o_bf16), _ptr(o_f32), H, n_rows, extra_row, kv_lora,
                                         rope, scale, _ptr(workspace), workspace.numel() * workspace.element_size(),
                                         _stream(stream)), "nm_mla_attention_combine")


def mla_params(dims: dict, seq_len: int, tensors: dict, rms_eps=1e-6, softmax_scale=None, layout_dense=ROW_MAJOR,
               workspace=None) -> MlaParams:
    """Fill an nm_mla_params from a dict of device tensors (keys as the struct's pointer fields;
    missing optional ones stay NULL)."""
    p = MlaParams()
    for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"):
        setattr(p, k, int(dims[k]))
    p.seq_len, p.layout_dense = int(seq_len), int(layout_dense)
    p.rms_eps = float(rms_eps)
    p.softmax_scale = float(softmax_scale if softmax_scale is not None else (dims["nope"] + dims["rope"]) ** -0.5)
    for name, _t in MlaParams._fields_:
        if _t is _vp and name in tensors and tensors[name] is not None:
            setattr(p, name, _ptr(tensors[name]))
    if workspace is not None:
        p.workspace = _ptr(workspace)
        p.workspace_bytes = workspace.numel() * workspace.element_size()
    return p


def nm_mla_workspace_bytes(p: MlaParams) -> int:
    return int(_lib.nm_mla_workspace_bytes(C.byref(p)))


def nm_mla_decode_step(p: MlaParams, main_stream=None, side_stream=None) -> None:
    ms = _stream(main_stream)
    ss = ms if side_stream is None else _stream(side_stream)
    _check(_lib.nm_mla_decode_step(C.byref(p), ms, ss), "nm_mla_decode_step")


def nm_mla_batch_workspace_bytes(p: MlaParams, T: int) -> int:
    return int(_lib.nm_mla_batch_workspace_bytes(C.byref(p), int(T)))


def mla_batch(seq_lens, h, rope_cos_sin, kv_cache, cache_stride, out=None, q_full=None, o_lat=None, o=None,
              c_q=None, c_qn=None, q=None, ckr=None) -> MlaBatch:
    """Fill an nm_mla_batch; seq_lens is a host sequence of ints (kept alive by the returned object)."""
    b = MlaBatch()
    b.T = len(seq_lens)
    b._seq_lens = (_i * b.T)(*[int(x) for x in seq_lens])
    b.seq_lens = C.cast(b._seq_lens, C.POINTER(_i))
    b.h, b.rope_cos_sin, b.kv_cache = _ptr(h), _ptr(rope_cos_sin), _ptr(kv_cache)
    b.cache_stride = int(cache_stride)
    b.out, b.q_full, b.o_lat, b.o = _ptr(out), _ptr(q_full), _ptr(o_lat), _ptr(o)
    b.c_q, b.c_qn, b.q, b.ckr = _ptr(c_q), _ptr(c_qn), _ptr(q), _ptr(ckr)
    return b


def nm_mla_decode_batch(p: MlaParams, b: MlaBatch, main_stream=None) -> None:
    _check(_lib.nm_mla_decode_batch(C.byref(p), C.byref(b), _stream(main_stream)), "nm_mla_decode_batch")


def nm_mla_decode_step_host(p: MlaParams, h_host, out_host, h_staging, out_staging, main_stream=None,
                            side_stream=None) -> None:
    ms = _stream(main_stream)
    ss = ms if side_stream is None else _stream(side_stream)
    _check(_lib.nm_mla_decode_step_host(C.byref(p), _ptr(h_host), _ptr(out_host), _ptr(h_staging), _ptr(out_staging),
                                        ms, ss), "nm_mla_decode_step_host")


def nm_debug_set_attention_trace(buf) -> None:
    _check(_lib.nm_debug_set_attention_trace(_ptr(buf)), "nm_debug_set_attention_trace")


def nm_debug_set_step_fusion(enable: bool) -> None:
    _check(_lib.nm_debug_set_step_fusion(int(enable)), "nm_debug_set_step_fusion")


def nm_debug_set_step_prefetch(megabytes: int) -> None:
    _check(_lib.nm_debug_set_step_prefetch(int(megabytes)), "nm_debug_set_step_prefetch")


def nm_debug_set_step_knobs(uv_programmatic: int = 1, prefetch_w_uv: int = 1) -> None:
    _check(_lib.nm_debug_set_step_knobs(int(uv_programmatic), int(prefetch_w_uv)), "nm_debug_set_step_knobs")


def nm_debug_set_batch_per_head_min_tokens(tokens: int) -> None:
    _check(_lib.nm_debug_set_batch_per_head_min_tokens(int(tokens)), "nm_debug_set_batch_per_head_min_tokens")


def nm_debug_set_cluster_split(enable: bool) -> None:
    _check(_lib.nm_debug_set_cluster_split(int(enable)), "nm_debug_set_cluster_split")


def nm_debug_set_step_tails(enable: int) -> None:
    _check(_lib.nm_debug_set_step_tails(int(enable)), "nm_debug_set_step_tails")


def nm_debug_set_step_plan(which: int, tile_n: int = 0, nsplit: int = 0, stages: int = 0) -> None:
    _check(_lib.nm_debug_set_step_plan(which, tile_n, nsplit, stages), "nm_debug_set_step_plan")


def nm_debug_stream_read(src, nbytes: int, sink, ctas_per_sm: int = 4, stream=None) -> None:
    _check(_lib.nm_debug_stream_read(_ptr(src), int(nbytes), _ptr(sink), int(ctas_per_sm), _stream(stream)), "nm_debug_stream_read")


def nm_debug_set_step_pdl(enable: bool) -> None:
    _check(_lib.nm_debug_set_step_pdl(int(enable)), "nm_debug_set_step_pdl")


def nm_debug_wait_probe(limit_ns: int, elapsed_ns=None, stream=None) -> None:
    """One CTA waits on an mbarrier nobody arrives at, with the wait limit set to limit_ns for that launch; the
    wait runs out, the kernel returns by itself and nm_check_status reports the timeout once."""
    _check(_lib.nm_debug_wait_probe(int(limit_ns), _ptr(elapsed_ns), _stream(stream)), "nm_debug_wait_probe")


def nm_debug_mma_probe(m, n, a_from_tmem, b_mn_major, reps, n_acc, a_step_bytes, b_step_bytes, out_clocks, stream=None) -> None:
    _check(_lib.nm_debug_mma_probe(int(m), int(n), int(a_from_tmem), int(b_mn_major), int(reps), int(n_acc), int(a_step_bytes),
                                   int(b_step_bytes), _ptr(out_clocks), _stream(stream)), "nm_debug_mma_probe")


def nm_debug_set_attention_wide(tile_rows: int = 0, max_runs: int = 0, cluster: int = 0) -> None:
    _check(_lib.nm_debug_set_attention_wide(int(tile_rows), int(max_runs), int(cluster)), "nm_debug_set_attention_wide")


def nm_debug_set_step_kv_beside_attention(enable: bool = True) -> None:
    _check(_lib.nm_debug_set_step_kv_beside_attention(1 if enable else 0), "nm_debug_set_step_kv_beside_attention")


def nm_debug_set_attention(impl: int) -> None:
    _check(_lib.nm_debug_set_attention(impl), "nm_debug_set_attention")
