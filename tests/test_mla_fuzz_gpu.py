"""Randomised parity of the single-token decode step against the oracle: sequence length, weight storage, schedule,
where the vector stages run, fused or separate per-head stages, attention kernel and programmatic launch are drawn
from a seeded generator; every case is checked stage by stage like the fixed cases of test_mla_gpu.py."""
import os

import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
import test_mla_gpu as base
from gpu_util import to_dev

pytestmark = pytest.mark.gpu

DIMS = gen.DSV3_DIMS
ROW, COL, NZ = 0, 1, 2


@pytest.fixture(scope="module")
def nm():
    import paper_2609_16009_b200 as nm
    yield nm
    nm.nm_debug_set_attention(0)
    nm.nm_debug_set_step_tails(1)
    nm.nm_debug_set_step_fusion(True)
    nm.nm_debug_set_step_pdl(True)
    nm.nm_debug_set_step_kv_beside_attention(False)
    nm.nm_check_status()


@pytest.fixture(scope="module")
def weights():
    w = gen.mla_weights(DIMS, seed=4000, with_wo=True)
    return w


def stored(w, layout, concat):
    """Device copies of the weights with the dense ones in the given storage (per-head weights stay row-major)."""
    d, ql, dkv = DIMS["d"], DIMS["q_lora"], DIMS["kv_lora"] + DIMS["rope"]
    H, dq, dv = DIMS["H"], DIMS["nope"] + DIMS["rope"], DIMS["v"]
    shapes = {"W_DQ": (d, ql), "W_DKVKR": (d, dkv), "W_UQR": (ql, H * dq), "W_O": (H * dv, d)}
    conv = {ROW: lambda X: X, COL: gen.to_col_major, NZ: gen.to_fractal_nz}[layout]
    out = {}
    for k, v in w.items():
        out[k] = to_dev(conv(np.asarray(v).reshape(shapes[k])) if k in shapes else v)
    if concat:
        cat = np.concatenate([np.asarray(w["W_DQ"]).reshape(d, ql), np.asarray(w["W_DKVKR"]).reshape(d, dkv)], axis=1)
        out["W_DQKV"] = to_dev(conv(cat))
        out.pop("W_DQ"); out.pop("W_DKVKR")
    return out


# NM_FUZZ_SEEDS=<n> widens the draw for a soak run; the default keeps the suite short
@pytest.mark.parametrize("seed", range(int(os.environ.get("NM_FUZZ_SEEDS", "24"))))
def test_random_step_matches_the_oracle(nm, weights, seed):
    rng = np.random.default_rng(50_000 + seed)
    S = int(rng.choice([1, 2, 3, 31, 64, 65, 127, 128, 129, int(rng.integers(130, 3000)), int(rng.integers(130, 3000))]))
    layout = int(rng.choice([ROW, ROW, COL, NZ]))
    concat = bool(rng.random() < 0.5) and layout != COL            # the concatenated down-projection is row-major or fractal
    overlap = bool(rng.random() < 0.5)
    tails, fusion, pdl = int(rng.integers(0, 3)), bool(rng.random() < 0.8), bool(rng.random() < 0.8)
    attn = int(rng.choice([0, 0, 1, 2, 3, 4]))
    kv_late = bool(np.random.default_rng(70_000 + seed).random() < 0.5)       # own generator: the other draws keep their values
    what = (f"seed {seed}: S {S} layout {layout} concat {concat} overlap {overlap} tails {tails} fusion {fusion} pdl {pdl} attention {attn} "
            f"kv beside attention {kv_late}")
    h, cache_ref, r = base.oracle_step(weights, S, seed=60_000 + seed)
    cache_in = gen.mla_cache(S, DIMS, seed=60_000 + seed)
    dw = stored(weights, layout, concat)
    nm.nm_debug_set_step_tails(tails); nm.nm_debug_set_step_fusion(fusion); nm.nm_debug_set_step_pdl(pdl); nm.nm_debug_set_attention(attn)
    nm.nm_debug_set_step_kv_beside_attention(kv_late)             # acts on the two-stream schedule only
    try:
        t = base.run_step(nm, dw, h, cache_in, S, overlap=overlap, layout_dense=layout)
    finally:
        nm.nm_debug_set_step_tails(1); nm.nm_debug_set_step_fusion(True); nm.nm_debug_set_step_pdl(True); nm.nm_debug_set_attention(0)
        nm.nm_debug_set_step_kv_beside_attention(False)
    try:
        base.check_step(t, r, cache_ref, S, weights, h, what=what)
    except AssertionError as e:
        raise AssertionError(f"{what}: {e}") from e


@pytest.mark.parametrize("seed", range(16))
def test_random_tokens_match_the_oracle(nm, weights, seed):
    """A different token per case (the cases above share one token and vary everything else).  The bf16 rounding after
    every stage makes the chain sensitive to the last bits of a sum: where the GPU's fp32 sum and the oracle's fp64 sum
    round one element of the query latent to different neighbours (both valid; about one token in ten), 1-2 % of q
    and up to a quarter of q_lat follow.  The check is therefore stage by stage on the GPU's own stage inputs, at the
    stated criteria; the end-to-end distance is printed and held to one fixed bound."""
    rng = np.random.default_rng(51_000 + seed)
    S = int(rng.choice([1, 2, 64, 65, 129, int(rng.integers(130, 3000)), int(rng.integers(130, 3000))]))
    concat = bool(rng.random() < 0.7)
    attn = int(rng.choice([0, 0, 1, 2, 3, 4]))
    h, cache_ref, r = base.oracle_step(weights, S, seed=62_000 + seed, token_seed=63_000 + seed)
    cache_in = gen.mla_cache(S, DIMS, seed=62_000 + seed)
    dw = stored(weights, ROW, concat)
    nm.nm_debug_set_attention(attn)
    try:
        t = base.run_step(nm, dw, h, cache_in, S)
    finally:
        nm.nm_debug_set_attention(0)
    try:
        base.check_step(t, r, cache_ref, S, weights, h)
    except AssertionError as e:
        raise AssertionError(f"seed {seed}: S {S} concat {concat} attention {attn}: {e}") from e


@pytest.mark.parametrize("seed", range(16))
def test_random_attention_stage_matches_the_oracle(nm, seed):
    """The attention pass alone on its own random operands (not the output of earlier GPU stages): every kernel,
    lengths from one row to a few thousand, the new row through the merge or through the pass."""
    rng = np.random.default_rng(90_000 + seed)
    S = int(rng.choice([1, 2, 33, 64, 65, 128, 129, int(rng.integers(130, 6000)), int(rng.integers(130, 6000))]))
    impl = int(rng.choice([0, 1, 2, 3, 4]))
    extra = bool(rng.random() < 0.5) or S == 1
    err = base.attention_case(nm, S, impl, extra, seed=91_000 + 10 * seed)
    assert err <= 2e-3, f"seed {seed}: S {S} impl {impl} extra {extra}: {err:.2e}"
