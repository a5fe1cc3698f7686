"""Seeded synthetic inputs shared by the tests, the smoke check and the bench.

This module holds none of the method's arithmetic: it only draws random numbers with torch's CPU
generator, scales them, and casts them to the storage type.  bf16 tensors are returned as
``numpy.uint16`` bit patterns so that the CPU oracle and the GPU library receive identical bits.

Recipe (shapes and distributions of the paper's workload, the DeepSeek-V3 MLA operator on one
token; trained weights are replaced by seeded random tensors):
  * fp32 GEMV: A 1x512, B 512x512, uniform[-1, 1], seed 0;
  * bf16 products (and the optional fp16 ones): A ~ N(0,1), B ~ N(0, 0.02^2);
  * MLA step: weights ~ N(0, 0.02^2), gamma ~ 1 + N(0, 0.02^2), h ~ N(0,1), cache rows ~ N(0,1).
Seeds: ``1000 * config_index + tensor_index`` unless given.
"""
from __future__ import annotations

import numpy as np
import torch

DSV3_DIMS = dict(d=7168, q_lora=1536, kv_lora=512, rope=64, nope=128, v=128, H=128)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """fp32 tensor -> bf16 storage (round-to-nearest-even cast) -> uint16 bit patterns."""
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> the fp32 values they denote (exact)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def normal_bf16(shape, std: float, seed: int, mean: float = 0.0) -> np.ndarray:
    t = torch.randn(shape, generator=_gen(seed), dtype=torch.float32) * std + mean
    return bf16_bits(t)


def uniform_f32(shape, lo: float, hi: float, seed: int) -> np.ndarray:
    t = torch.rand(shape, generator=_gen(seed), dtype=torch.float32) * (hi - lo) + lo
    return t.numpy().copy()


def small_int_bf16(shape, lo: int, hi: int, seed: int) -> np.ndarray:
    """Integers in [lo, hi] stored as bf16 (exactly representable for |x| <= 256)."""
    t = torch.randint(lo, hi + 1, shape, generator=_gen(seed)).to(torch.float32)
    return bf16_bits(t)


def small_int_f32(shape, lo: int, hi: int, seed: int) -> np.ndarray:
    return torch.randint(lo, hi + 1, shape, generator=_gen(seed)).to(torch.float32).numpy().copy()


def to_col_major(B_rowmajor: np.ndarray) -> np.ndarray:
    """Storage of the same K x N matrix with element (k, n) at n*K + k."""
    return np.ascontiguousarray(B_rowmajor.T)


def to_fractal_nz(B_rowmajor: np.ndarray) -> np.ndarray:
    """Storage of the same K x N matrix in 16 x 16 fractals, fractals ordered by columns, elements inside a fractal by
    rows (K and N multiples of 16).  A pure permutation: [K/16, 16, N/16, 16] -> [N/16, K/16, 16, 16], flattened."""
    K, N = B_rowmajor.shape
    assert K % 16 == 0 and N % 16 == 0
    return np.ascontiguousarray(B_rowmajor.reshape(K // 16, 16, N // 16, 16).transpose(2, 0, 1, 3)).reshape(-1)


def gemv_fp32(seed: int = 0, K: int = 512, N: int = 512, M: int = 1):
    """fp32 GEMV case: both operands uniform[-1, 1] from one generator stream (A first)."""
    g = _gen(seed)
    A = (torch.rand((M, K), generator=g, dtype=torch.float32) * 2 - 1).numpy().copy()
    B = (torch.rand((K, N), generator=g, dtype=torch.float32) * 2 - 1).numpy().copy()
    return A, B


def narrow_bf16(M: int, K: int, N: int, seed: int):
    """A [M,K] ~ N(0,1), B [K,N] ~ N(0, 0.02^2) row-major, as bf16 bits."""
    A = normal_bf16((M, K), 1.0, seed)
    B = normal_bf16((K, N), 0.02, seed + 1)
    return A, B


def narrow_f16(M: int, K: int, N: int, seed: int):
    """The same recipe stored as fp16 (IEEE binary16) bit patterns: the optional element type of the product."""
    g = _gen(seed)
    A = torch.randn((M, K), generator=g, dtype=torch.float32)
    B = torch.randn((K, N), generator=g, dtype=torch.float32) * 0.02
    to_bits = lambda t: t.to(torch.float16).contiguous().view(torch.int16).numpy().view(np.uint16).copy()
    return to_bits(A), to_bits(B)


def per_head(T: int, seed: int, H: int = 128, nope: int = 128, kv_lora: int = 512, v: int = 128):
    """Per-head absorbed-MLA products: q_nope [T,H,nope], W_UK [H,nope,kv_lora],
    o_lat [T,H,kv_lora], W_UV [H,kv_lora,v]."""
    return dict(q_nope=normal_bf16((T, H, nope), 1.0, seed),
                W_UK=normal_bf16((H, nope, kv_lora), 0.02, seed + 1),
                o_lat=normal_bf16((T, H, kv_lora), 1.0, seed + 2),
                W_UV=normal_bf16((H, kv_lora, v), 0.02, seed + 3))


def mla_weights(dims: dict = DSV3_DIMS, seed: int = 4000, with_wo: bool = True) -> dict:
    d, ql, dc, dr, dn, dv, H = (dims[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
    w = dict(W_DQ=normal_bf16((d, ql), 0.02, seed + 0),
             gamma_q=normal_bf16((ql,), 0.02, seed + 1, mean=1.0),
             W_UQR=normal_bf16((ql, H * (dn + dr)), 0.02, seed + 2),
             W_DKVKR=normal_bf16((d, dc + dr), 0.02, seed + 3),
             gamma_kv=normal_bf16((dc,), 0.02, seed + 4, mean=1.0),
             W_UK=normal_bf16((H, dn, dc), 0.02, seed + 5),
             W_UV=normal_bf16((H, dc, dv), 0.02, seed + 6))
    if with_wo:
        w["W_O"] = normal_bf16((H * dv, d), 0.02, seed + 7)
    return w


def mla_token(dims: dict = DSV3_DIMS, seed: int = 4100) -> np.ndarray:
    return normal_bf16((dims["d"],), 1.0, seed)


def mla_cache(seq_len: int, dims: dict = DSV3_DIMS, seed: int = 4200, rows: int | None = None) -> np.ndarray:
    """Latent cache [rows, kv_lora+rope]: rows 0..seq_len-2 ~ N(0,1); the rest zero (row
    seq_len-1 is written by the step)."""
    rows = rows or seq_len
    cache = np.zeros((rows, dims["kv_lora"] + dims["rope"]), dtype=np.uint16)
    if seq_len > 1:
        cache[:seq_len - 1] = normal_bf16((seq_len - 1, dims["kv_lora"] + dims["rope"]), 1.0, seed)
    return cache
