"""Algorithm 2 ("Specialized MatMul 2 on AIV") restated on the CPU (test infrastructure).

The steps are taken in the algorithm's order and notation: constants, executor pool size V,
per-executor token slice, the compute loop over nPartW weight blocks with fp32 dot products
stored to ``tmpBuf``, then the gather over kParts partial sums and one final cast to bf16.
The fractal transpose and the strided cast exist only to undo the FRACTAL_NZ storage of the
weights; here W is a plain row-major K x N array, so a block is read column by column directly.

Readings taken where the algorithm is ambiguous:
  * the column block of ``W[off_T, fracId]`` is ``fracId mod fractalNum`` and its k-part is
    ``fracId DIV fractalNum`` (equal to ``v DIV groupSize``, which is how off_T is defined);
  * ``tmpBuf`` is indexed in elements: block ``fracId`` starts at element ``fracId*fractalSize``,
    which equals ``kpart*N + fcol*fractalSize`` and so matches the gather's ``off_C + i*N``;
  * ``groupSize = V DIV kParts`` needs kParts | V, true for the paper's case only.
"""
from __future__ import annotations

import numpy as np

from . import bf16_to_f64, f64_to_bf16


def executor_pool(K: int, N: int, P: int, fractalSize: int = 16, kSplitSize: int = 1024):
    """Init stage: the tiling constants and the pool size V = max divisor of S not above 2P."""
    kParts = K // kSplitSize
    fractalNum = N // fractalSize
    S = fractalNum * kParts
    V = max(dv for dv in range(1, S + 1) if S % dv == 0 and dv <= 2 * P)
    nPartW = S // V
    groupSize = V // kParts
    return dict(kParts=kParts, fractalNum=fractalNum, S=S, V=V, nPartW=nPartW, groupSize=groupSize,
                fractalSize=fractalSize, kSplitSize=kSplitSize)


def matmul2(T_bits: np.ndarray, W_bits: np.ndarray, K: int, N: int, P: int = 24,
            fractalSize: int = 16, kSplitSize: int = 1024):
    """C[1xN] = T[1xK] * W[KxN], bf16 in/out, fp32 partial sums, following Algorithm 2.

    Returns (C bits uint16 [N], tmpBuf fp32 [kParts*N], list of every fracId produced)."""
    c = executor_pool(K, N, P, fractalSize, kSplitSize)
    kParts, fractalNum, V, nPartW, groupSize = (c[k] for k in ("kParts", "fractalNum", "V", "nPartW", "groupSize"))
    T = bf16_to_f64(T_bits.reshape(K)).astype(np.float32)          # widening is exact
    W = bf16_to_f64(W_bits.reshape(K, N)).astype(np.float32)
    tmpBuf = np.full(kParts * N, np.nan, dtype=np.float32)
    produced = []
    # compute stage, one executor v at a time
    for v in range(V):
        off_T = (v // groupSize) * kSplitSize
        T_v = T[off_T:off_T + kSplitSize]                           # loaded once per executor
        for w in range(nPartW):
            fracId = v * nPartW + w
            fcol = fracId % fractalNum
            W_vw = W[off_T:off_T + kSplitSize, fcol * fractalSize:(fcol + 1) * fractalSize]
            partSum = np.empty(fractalSize, dtype=np.float32)
            for j in range(fractalSize):
                partSum[j] = np.sum(T_v * W_vw[:, j], dtype=np.float32)   # fp32 Mul + ReduceSum
            tmpBuf[fracId * fractalSize:(fracId + 1) * fractalSize] = partSum
            produced.append(fracId)
    # gather stage (after the barrier): executors v < fractalNum
    Cout = np.zeros(N, dtype=np.uint16)
    for v in range(fractalNum):
        off_C = v * fractalSize
        Acc = np.zeros(fractalSize, dtype=np.float32)
        for i in range(kParts):
            Acc = (Acc + tmpBuf[off_C + i * N: off_C + i * N + fractalSize]).astype(np.float32)
        Cout[off_C:off_C + fractalSize] = f64_to_bf16(Acc.astype(np.float64))
    return Cout, tmpBuf, produced
