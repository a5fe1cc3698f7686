"""Helpers for the GPU parity tests: move bit patterns to the device, call the C-ABI binding,
compare element by element with the oracle under the stated tolerance."""
from __future__ import annotations

import numpy as np
import torch

import oracle

NP_IN = {0: np.float32, 1: np.uint16, 2: np.uint16}
ORACLE_IN = {0: oracle.F32, 1: oracle.BF16, 2: oracle.BF16}
ORACLE_OUT = {0: oracle.F32, 1: oracle.BF16, 2: oracle.F32}


def to_dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16).copy()).cuda()
    return torch.from_numpy(a.copy()).cuda()


def out_buffer(numel: int, dtype: int, guard: int = 64):
    """Output buffer with canary guard bands on both sides.  Returns (whole, view of the middle)."""
    tdt = torch.int16 if dtype == 1 else torch.float32
    whole = torch.empty(numel + 2 * guard, dtype=tdt, device="cuda")
    if dtype == 1:
        whole.fill_(0x7A7A)
    else:
        whole.fill_(-12345.5)
    return whole, whole[guard:guard + numel]


def guards_intact(whole: torch.Tensor, numel: int, dtype: int, guard: int = 64) -> bool:
    w = whole.cpu()
    canary = 0x7A7A if dtype == 1 else -12345.5
    return bool((w[:guard] == canary).all() and (w[guard + numel:] == canary).all())


def out_to_f64(t: torch.Tensor, dtype: int) -> np.ndarray:
    a = t.cpu().numpy()
    if dtype == 1:
        return oracle.bf16_to_f64(a.view(np.uint16))
    return a.astype(np.float64)


def assert_matmul_close(got: np.ndarray, Cq: np.ndarray, C64: np.ndarray, bound: np.ndarray, dtype: int, what=""):
    """|gpu - oracle| <= 1e-5 * sum_k|a*b| + 1e-6, plus one output ulp for bf16 outputs."""
    ref = oracle.bf16_to_f64(Cq) if dtype == 1 else Cq.astype(np.float64)
    tol = 1e-5 * bound + 1e-6
    if dtype == 1:
        tol = tol + oracle.ulp_bf16(C64)
    err = np.abs(got.reshape(ref.shape) - ref)
    bad = err > tol
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} elements outside tolerance; "
                           f"worst err {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}, "
                           f"tol there {tol.reshape(err.shape)[np.unravel_index(err.argmax(), err.shape)]:.3e}")


def assert_output_side_stage_by_stage(dims, w, q_full, cache_rows, o_lat, o, out, what=""):
    """The output side of the decode step checked stage by stage on the values the GPU itself produced (uint16 bit
    patterns): the oracle recomputes each stage from the GPU's inputs to that stage, so a rounding of an earlier
    stage that fell the other way than the oracle's (both are valid: fp32 and fp64 sums differ in the last bits)
    does not enter.  Attention: the softmax criterion (2e-3 of the largest output, plus one bf16 ulp);
    the per-head W_UV product and W_O: the matmul criterion (1e-5 * sum|a b| + 1e-6, plus one ulp).
    cache_rows: [S][kv_lora + rope], the new row included.  out (and W_O) may be None."""
    H, dc, dr, dn, dv, d = (dims[k] for k in ("H", "kv_lora", "rope", "nope", "v", "d"))
    f64 = lambda bits: oracle.bf16_to_f64(np.asarray(bits, dtype=np.uint16))
    q_full, o_lat, o = (np.asarray(x, dtype=np.uint16) for x in (q_full, o_lat, o))
    ref = oracle.mla_attention(f64(q_full).reshape(H, dc + dr), f64(cache_rows), dc, (dn + dr) ** -0.5, threads=8)
    got = f64(o_lat).reshape(H, dc)
    assert np.all(np.abs(got - ref) <= 2e-3 * np.abs(ref).max() + oracle.ulp_bf16(ref)), f"{what}: attention stage"
    Cq, C64, bound = oracle.matmul_batched(o_lat.reshape(-1), np.asarray(w["W_UV"]).reshape(-1), 1, dv, dc, H, H * dc, dc, dc * dv,
                                           H * dv, dv, H * dv, oracle.BF16, oracle.BF16, threads=8)
    assert_matmul_close(f64(o).reshape(-1), Cq, C64, bound, 1, f"{what}: W_UV stage")
    if out is not None:
        Cq, C64, bound = oracle.matmul(o.reshape(1, -1), np.asarray(w["W_O"]), 1, d, H * dv, oracle.BF16, oracle.BF16, threads=8)
        assert_matmul_close(f64(out).reshape(1, -1), Cq, C64, bound, 1, f"{what}: W_O stage")
