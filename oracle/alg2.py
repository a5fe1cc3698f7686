"""Split-K tiling of the paper's MatMul 2 (Algorithm 2), as a CPU check (test infrastructure).

Algorithm 2 cuts the K x N weight matrix into blocks of ``k_split`` rows by ``col_block`` columns, deals
the blocks out to a pool of executors, lets each block produce an fp32 partial sum per column, and
then adds the partial sums of a column block in k order and rounds once to bf16.  What the tests need
from it is stated here in three independent pieces, none of which walks the executors one by one:

  * ``tiling(K, N, cores)``       - the closed-form constants of the Init stage;
  * ``block_of_work_item(...)``   - which (k part, column block) the i-th item of the flattened
                                    executor x slot grid stands for, vectorised over all items;
  * ``split_k_product(...)``      - the arithmetic: per-part fp32 column sums, parts added in order,
                                    one rounding.

Readings taken where the algorithm is ambiguous (valid for the paper's constants, which the tests pin):
the flattened item index counts column blocks fastest and k parts slowest; the scratch buffer is indexed
in elements, so the partial sums of k part i for column block c start at ``i*N + c*col_block``; the pool
size must be a multiple of the number of k parts.
"""
from __future__ import annotations

import numpy as np

from . import bf16_to_f64, f64_to_bf16


def tiling(K: int, N: int, cores: int, col_block: int = 16, k_split: int = 1024) -> dict:
    """Constants of Algorithm 2's Init stage.  ``pool`` is the largest divisor of the block count that
    does not exceed two executors per core."""
    k_parts = K // k_split
    col_blocks = N // col_block
    blocks = k_parts * col_blocks
    divisors = np.arange(1, blocks + 1)
    divisors = divisors[(blocks % divisors == 0) & (divisors <= 2 * cores)]
    pool = int(divisors.max())
    return dict(kParts=k_parts, fractalNum=col_blocks, S=blocks, V=pool, nPartW=blocks // pool,
                groupSize=pool // k_parts)


def block_of_work_item(c: dict):
    """For every item of the executor x slot grid (executor-major), the k part and the column block it
    computes, and the k part its executor's token slice was loaded for.  Returns three int arrays of
    length ``pool * slots``; the tests require (k part, column block) to hit every block exactly once and
    the two k parts to agree."""
    item = np.arange(c["V"] * c["nPartW"])
    executor = item // c["nPartW"]
    return item // c["fractalNum"], item % c["fractalNum"], executor // c["groupSize"]


def split_k_product(T_bits: np.ndarray, W_bits: np.ndarray, K: int, N: int, k_split: int = 1024):
    """C[1xN] = T[1xK] * W[KxN] with bf16 operands, fp32 partial sums per k part, the parts added in
    increasing k order in fp32, and one final rounding to bf16.  Returns (C bits [N], partials fp32
    [k_parts, N])."""
    T = bf16_to_f64(T_bits.reshape(K)).astype(np.float32)           # bf16 -> fp32 widening is exact
    W = bf16_to_f64(W_bits.reshape(K, N)).astype(np.float32)
    k_parts = K // k_split
    products = T.reshape(k_parts, k_split, 1) * W.reshape(k_parts, k_split, N)      # exact in fp32
    partials = products.sum(axis=1, dtype=np.float32)
    total = np.zeros(N, dtype=np.float32)
    for part in partials:                                            # fixed order, fp32 adds
        total = (total + part).astype(np.float32)
    return f64_to_bf16(total.astype(np.float64)), partials
