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
