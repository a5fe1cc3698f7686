"""Parity of the MLA decode step with the CPU oracle: every stage in isolation (fed the oracle's
bf16 stage inputs) and the whole step end to end."""
import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
from gpu_util import END_TO_END_BOUND, assert_matmul_close, assert_step_stage_by_stage, end_to_end_distance, out_to_f64, to_dev

pytestmark = pytest.mark.gpu

DIMS = gen.DSV3_DIMS
BF16, ROW = 1, 0


def f64(bits):
    return oracle.bf16_to_f64(np.asarray(bits, dtype=np.uint16))


def dev_bits_to_f64(t):
    return oracle.bf16_to_f64(t.cpu().numpy().view(np.uint16))


def rel_max(got, ref):
    return float(np.abs(got - ref).max() / np.abs(ref).max())


@pytest.fixture(scope="module")
def nm():
    import paper_2609_16009_b200 as nm
    yield nm
    nm.nm_debug_set_attention(0)
    nm.nm_check_status()


@pytest.fixture(scope="module")
def weights():
    w = gen.mla_weights(DIMS, seed=4000, with_wo=True)
    dw = {k: to_dev(v) for k, v in w.items()}
    return w, dw


def oracle_step(w, S, seed=4200, with_wo=True, token_seed=4100):
    h = gen.mla_token(DIMS, seed=token_seed)
    cache = gen.mla_cache(S, DIMS, seed=seed)
    ww = dict(w)
    if not with_wo:
        ww.pop("W_O", None)
    r = oracle.mla_decode_step(DIMS, ww, h, cache, S, threads=8)
    return h, cache, r


@pytest.fixture(scope="module")
def ref1024(weights):
    w, _ = weights
    return oracle_step(w, 1024)


def rope_row(nm, pos):
    table = torch.empty(DIMS["rope"], dtype=torch.float32, device="cuda")
    nm.nm_rope_table(table, pos, 1, DIMS["rope"])
    return table


# ---- vector-side stages ---------------------------------------------------------------------------------

@pytest.mark.parametrize("pos", [0, 1, 1023, 16383, 1000003])
def test_rope_table_matches_oracle_angles(nm, pos):
    dim = DIMS["rope"]
    table = rope_row(nm, pos).cpu().numpy().astype(np.float64)
    # the oracle's rotation of unit vectors (1,0) gives (cos, sin) of every pair
    e = np.zeros(dim); e[0::2] = 1.0
    cs = oracle.rope(e, pos)
    assert np.abs(table - cs).max() <= 2.0 ** -23         # fp32 rounding of values in [-1, 1]


def test_rmsnorm_stage(nm, ref1024, weights):
    w, dw = weights
    _, _, r = ref1024
    y = torch.zeros(DIMS["q_lora"], dtype=torch.int16, device="cuda")
    nm.nm_rmsnorm(to_dev(r["c_q"]), dw["gamma_q"], y, DIMS["q_lora"], 1e-6)
    torch.cuda.synchronize()
    got, ref = dev_bits_to_f64(y), f64(r["c_qn"])
    assert np.all(np.abs(got - ref) <= 1e-5 * np.abs(ref) + oracle.ulp_bf16(ref))
    assert np.mean(got == ref) > 0.99                      # a rounding flip is rare


@pytest.mark.parametrize("n", [1, 7, 512, 1536, 16384])
def test_rmsnorm_sizes(nm, n):
    x = gen.normal_bf16((n,), 3.0, seed=50 + n)
    g = gen.normal_bf16((n,), 0.02, seed=51 + n, mean=1.0)
    y = torch.zeros(n, dtype=torch.int16, device="cuda")
    nm.nm_rmsnorm(to_dev(x), to_dev(g), y, n, 1e-6)
    torch.cuda.synchronize()
    ref = f64(oracle.f64_to_bf16(oracle.rmsnorm(f64(x), f64(g), 1e-6)))
    assert np.all(np.abs(dev_bits_to_f64(y) - ref) <= 1e-5 * np.abs(ref) + oracle.ulp_bf16(ref))


def test_rope_stage(nm, ref1024):
    _, _, r = ref1024
    H, dn, dr = DIMS["H"], DIMS["nope"], DIMS["rope"]
    pos = 1023
    q = to_dev(r["q"])                                      # [H][nope+rope]
    y = torch.zeros(H * dr, dtype=torch.int16, device="cuda")
    nm.nm_rope(q.view(-1)[dn:], y, H, dr, dn + dr, dr, rope_row(nm, pos))
    torch.cuda.synchronize()
    got, ref = dev_bits_to_f64(y).reshape(H, dr), f64(r["q_rope"])
    qf = f64(r["q"])[:, dn:]
    mag = np.abs(qf[:, 0::2]) + np.abs(qf[:, 1::2])         # size of the terms of each output
    mag = np.repeat(mag, 2, axis=1)
    assert np.all(np.abs(got - ref) <= 1e-5 * mag + oracle.ulp_bf16(ref))


# ---- narrow products of the step, each fed the oracle's inputs ---------------------------------------------

def test_matmul_stages_of_the_step(nm, ref1024, weights):
    w, dw = weights
    h, cache, r = ref1024
    d, ql, dc, dr, dn, dv, H = (DIMS[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
    dq, dkv = dn + dr, dc + dr
    ws = nm.new_workspace(max(nm.nm_matmul_workspace_bytes(1, H * dq, ql), nm.nm_matmul_workspace_bytes(1, dc, dn, H)))

    def run(A, Wd, W_bits, M, N, K, ref_bits, what):
        C = torch.zeros(M * N, dtype=torch.int16, device="cuda")
        nm.nm_matmul_ws(to_dev(A), Wd, C, M, N, K, BF16, ROW, ws)
        torch.cuda.synchronize()
        Cq, C64, bound = oracle.matmul(np.asarray(A).reshape(M, K), W_bits, M, N, K, oracle.BF16, oracle.BF16, threads=8)
        assert np.array_equal(Cq.reshape(-1), np.asarray(ref_bits).reshape(-1)), what      # the step's stage IS this product
        assert_matmul_close(dev_bits_to_f64(C).reshape(M, N), Cq, C64, bound, 1, what)

    run(h, dw["W_DQ"], w["W_DQ"], 1, ql, d, r["c_q"], "c_q = h*W_DQ")
    run(r["c_qn"], dw["W_UQR"], w["W_UQR"], 1, H * dq, ql, r["q"], "q = c_qn*W_UQR")
    run(h, dw["W_DKVKR"], w["W_DKVKR"], 1, dkv, d, r["ckr"], "ckr = h*(W_DKV|W_KR)")
    run(r["o"].reshape(-1), dw["W_O"], w["W_O"], 1, d, H * dv, r["out"], "out = o*W_O")
    # per-head: q_lat written with the attention operand's stride, o from o_lat
    qfull = torch.zeros(H * dkv, dtype=torch.int16, device="cuda")
    nm.nm_matmul_batched_ws(to_dev(r["q"]), dw["W_UK"], qfull, 1, dc, dn, H, H * dq, dq, dn * dc, H * dkv, dkv, BF16, ROW, ws)
    o = torch.zeros(H * dv, dtype=torch.int16, device="cuda")
    nm.nm_matmul_batched_ws(to_dev(r["o_lat"]), dw["W_UV"], o, 1, dv, dc, H, H * dc, dc, dc * dv, H * dv, dv, BF16, ROW, ws)
    torch.cuda.synchronize()
    Cq, C64, bound = oracle.matmul_batched(np.asarray(r["q"]).reshape(-1), np.asarray(w["W_UK"]).reshape(-1), 1, dc, dn, H, H * dq, dq,
                                           dn * dc, H * dc, dc, H * dc, oracle.BF16, oracle.BF16, threads=8)
    assert np.array_equal(Cq.reshape(H, dc), np.asarray(r["q_lat"]))
    assert_matmul_close(dev_bits_to_f64(qfull).reshape(H, dkv)[:, :dc].reshape(-1), Cq, C64, bound, 1, "q_lat = q_nope*W_UK")
    Cq, C64, bound = oracle.matmul_batched(np.asarray(r["o_lat"]).reshape(-1), np.asarray(w["W_UV"]).reshape(-1), 1, dv, dc, H, H * dc, dc,
                                           dc * dv, H * dv, dv, H * dv, oracle.BF16, oracle.BF16, threads=8)
    assert np.array_equal(Cq.reshape(H, dv), np.asarray(r["o"]))
    assert_matmul_close(dev_bits_to_f64(o).reshape(-1), Cq, C64, bound, 1, "o = o_lat*W_UV")


# ---- attention stage -----------------------------------------------------------------------------------

def attention_case(nm, S, impl, extra, seed=7000):
    """Q ~ what the step produces in scale; cache rows ~ N(0,1).  extra: attend the last row through
    the merge (as the step does) or through the row pass."""
    H, dc, dr = DIMS["H"], DIMS["kv_lora"], DIMS["rope"]
    dkv = dc + dr
    Q = np.concatenate([gen.normal_bf16((H, dc), 0.18, seed), gen.normal_bf16((H, dr), 0.78, seed + 1)], axis=1)
    cache = gen.normal_bf16((S, dkv), 1.0, seed + 2)
    scale = (DIMS["nope"] + dr) ** -0.5
    ref = oracle.mla_attention(f64(Q), f64(cache), dc, scale, threads=8)
    ws = torch.empty(nm.nm_mla_attention_workspace_bytes(H, S, dc), dtype=torch.uint8, device="cuda")
    o16 = torch.zeros(H * dc, dtype=torch.int16, device="cuda")
    o32 = torch.zeros(H * dc, dtype=torch.float32, device="cuda")
    nm.nm_debug_set_attention(impl)
    try:
        n_rows, extra_row = (S - 1, S - 1) if extra else (S, -1)
        nm.nm_mla_attention(to_dev(Q), to_dev(cache), o16, o32, H, n_rows, extra_row, dc, dr, scale, ws)
        torch.cuda.synchronize()
    finally:
        nm.nm_debug_set_attention(0)
    got32 = o32.cpu().numpy().astype(np.float64).reshape(H, dc)
    assert rel_max(got32, ref) <= 2e-3, f"S={S} impl={impl}: unrounded output off by {rel_max(got32, ref):.2e}"
    got16 = dev_bits_to_f64(o16).reshape(H, dc)
    assert np.all(np.abs(got16 - ref) <= 2e-3 * np.abs(ref).max() + oracle.ulp_bf16(ref))
    return rel_max(got32, ref)


@pytest.mark.parametrize("S", [1, 2, 63, 64, 65, 200, 1000, 1024, 4096])
@pytest.mark.parametrize("extra", [True, False])
def test_attention_stage_cuda_cores(nm, S, extra):
    if S == 1 and not extra:
        attention_case(nm, S, 1, False)
        return
    err = attention_case(nm, S, 1, extra)
    assert err <= 1e-5                                       # fp32 throughout: far inside the bound


@pytest.mark.parametrize("S", [1, 2, 63, 64, 65, 129, 200, 1000, 1024, 4096, 16384])
@pytest.mark.parametrize("extra", [True, False])
def test_attention_stage_default_path(nm, S, extra):
    attention_case(nm, S, 0, extra)


@pytest.mark.parametrize("S", [1, 2, 33, 64, 65, 129, 1000, 4096, 16384])
@pytest.mark.parametrize("extra", [True, False])
def test_attention_stage_128_heads_per_cta(nm, S, extra):
    """The tensor-core kernel that keeps all 128 heads in one CTA (32-row cache stages) stays selectable."""
    attention_case(nm, S, 2, extra)


@pytest.mark.parametrize("tile,runs,cluster", [(64, 0, 1), (64, 0, 2), (64, 0, 4), (128, 0, 1), (128, 0, 4), (256, 0, 1), (256, 0, 2), (256, 0, 4),
                                               (64, 3, 1), (128, 5, 2), (256, 5, 4)])
def test_attention_stage_wide_tiles(nm, tile, runs, cluster):
    """The wide-tile tensor-core kernel (the default from 6144 cache rows on) forced at every length, with every tile
    width, on-chip merges of 1, 2 and 4 row runs, one tile per CTA and several (few runs over many rows)."""
    nm.nm_debug_set_attention_wide(tile, runs, cluster)
    try:
        for S in (1, 2, 63, 64, 65, 129, 257, 1000, 1024, 4096, 5000, 16384, 20000):
            for extra in (True, False):
                if S == 1 and not extra:
                    continue
                attention_case(nm, S, 4, extra)
                nm.nm_check_status()
    finally:
        nm.nm_debug_set_attention_wide(0, 0, 0)


@pytest.mark.parametrize("impl", [0, 3, 2])
def test_attention_stage_long_sequence(nm, impl):
    """A long sequence: the default (the wide-tile kernel, several 256-row tiles per CTA) and the two older kernels."""
    attention_case(nm, 66001, impl, True)


def test_attention_kernels_agree_on_heavy_tailed_scores(nm):
    """Scores whose maximum grows along the sequence by more than the lazy-rescale threshold force the rescale of
    the running output in both tensor-core kernels; all three implementations must agree with the oracle."""
    H, dc, dr = DIMS["H"], DIMS["kv_lora"], DIMS["rope"]
    dkv, S = dc + dr, 700
    Q = np.concatenate([gen.normal_bf16((H, dc), 0.18, 7100), gen.normal_bf16((H, dr), 0.78, 7101)], axis=1)
    c64 = f64(gen.normal_bf16((S, dkv), 1.0, 7102)) * np.linspace(0.05, 6.0, S)[:, None]     # norms grow with the row
    cache = oracle.f64_to_bf16(c64)
    scale = (DIMS["nope"] + dr) ** -0.5
    ref = oracle.mla_attention(f64(Q), f64(cache), dc, scale, threads=8)
    ws = torch.empty(nm.nm_mla_attention_workspace_bytes(H, S, dc), dtype=torch.uint8, device="cuda")
    for impl in (0, 1, 2, 3, 4):
        o16 = torch.zeros(H * dc, dtype=torch.int16, device="cuda")
        o32 = torch.zeros(H * dc, dtype=torch.float32, device="cuda")
        nm.nm_debug_set_attention(impl)
        try:
            nm.nm_mla_attention(to_dev(Q), to_dev(cache), o16, o32, H, S, -1, dc, dr, scale, ws)
            torch.cuda.synchronize()
        finally:
            nm.nm_debug_set_attention(0)
        nm.nm_check_status()
        got = o32.cpu().numpy().astype(np.float64).reshape(H, dc)
        assert rel_max(got, ref) <= 2e-3, f"impl {impl}: {rel_max(got, ref):.2e}"


# ---- the whole step ---------------------------------------------------------------------------------------

def run_step(nm, dw, h, cache_in, S, with_wo=True, overlap=True, rows=None, concat_down=False, layout_dense=0):
    H, dc, dr, dn, dv, d, ql = (DIMS[k] for k in ("H", "kv_lora", "rope", "nope", "v", "d", "q_lora"))
    dkv, dq = dc + dr, dn + dr
    t = dict(dw)
    if not with_wo:
        t.pop("W_O")
    if concat_down:      # (W_DQ | W_DKV | W_KR) stored as one matrix; the separate ones are not passed
        t["W_DQKV"] = torch.cat([t.pop("W_DQ").view(d, ql), t.pop("W_DKVKR").view(d, dkv)], dim=1).contiguous().view(-1)
    t["h"] = to_dev(h)
    t["kv_cache"] = to_dev(cache_in)
    t["rope_cos_sin"] = rope_row(nm, S - 1)
    outs = {"c_q": ql, "c_qn": ql, "q": H * dq, "q_full": H * dkv, "ckr": dkv, "o_lat": H * dc, "o": H * dv, "out": d}
    for k, n in outs.items():
        t[k] = torch.zeros(n, dtype=torch.int16, device="cuda")
    t["o_lat_f32"] = torch.zeros(H * dc, dtype=torch.float32, device="cuda")
    p = nm.mla_params(DIMS, S, t, layout_dense=layout_dense)
    ws = nm.new_workspace(nm.nm_mla_workspace_bytes(p))
    p = nm.mla_params(DIMS, S, t, workspace=ws, layout_dense=layout_dense)
    main = torch.cuda.Stream()
    side = torch.cuda.Stream() if overlap else None
    torch.cuda.synchronize()
    nm.nm_mla_decode_step(p, main, side)
    torch.cuda.synchronize()
    nm.nm_check_status()
    return t


def check_step(t, r, cache_ref, S, w, h, with_wo=True, what="step"):
    """The parity check of a whole step.
    (a) Stage by stage, every stage, at the stated criteria: the oracle recomputes each stage from the GPU's own input
        to that stage (gpu_util.assert_step_stage_by_stage).  This is what the parity claim rests on.
    (b) The cache rows before the new one are untouched, bit for bit.
    (c) End to end against the oracle's own chain from h: the first-stage products (whose inputs ARE the oracle's) at
        the matmul criterion; for everything downstream the distance max|g - o| / max|o| is printed and held to one
        fixed bound (gpu_util.END_TO_END_BOUND) that does not depend on the data: two valid chains of eleven bf16
        roundings may part by a rounding flip early on, so the stated criteria are applied per stage in (a), not here."""
    H, dc, dr, dn = DIMS["H"], DIMS["kv_lora"], DIMS["rope"], DIMS["nope"]
    dkv = dc + dr
    cache = t["kv_cache"].cpu().numpy().view(np.uint16).reshape(-1, dkv)
    g = {k: t[k] for k in ("c_q", "c_qn", "q", "q_full", "ckr", "o_lat", "o", "o_lat_f32")}
    g["cache"] = cache[:S]
    g["out"] = t["out"] if with_wo else None
    ww = dict(w)
    if not with_wo:
        ww.pop("W_O", None)
    assert_step_stage_by_stage(DIMS, ww, h, S - 1, g, what)
    assert np.array_equal(cache[:S - 1], cache_ref[:S - 1]), f"{what}: old cache rows changed"
    for name, bound in (("c_q", "bound_c_q"), ("ckr", "bound_ckr")):
        got, ref = dev_bits_to_f64(t[name]), f64(r[name])
        assert np.all(np.abs(got - ref) <= 1e-5 * r[bound] + 1e-6 + oracle.ulp_bf16(ref)), f"{what}: {name} end to end"
    refs = {"c_qn": r["c_qn"], "q": r["q"], "q_full": np.concatenate([np.asarray(r["q_lat"]), np.asarray(r["q_rope"])], axis=1),
            "kv_cache row": cache_ref[S - 1], "o_lat": r["o_lat"], "o": r["o"]}
    if with_wo:
        refs["out"] = r["out"]
    dist = {k: end_to_end_distance(cache[S - 1] if k == "kv_cache row" else t[k], v) for k, v in refs.items()}
    dist["o_lat_f32"] = rel_max(t["o_lat_f32"].cpu().numpy().astype(np.float64).reshape(H, dc), r["o_lat_f64"])
    print(f"{what}: S {S}: end-to-end distance to the oracle's chain: " + ", ".join(f"{k} {v:.1e}" for k, v in dist.items()))
    worst = max(dist, key=dist.get)
    assert dist[worst] <= END_TO_END_BOUND, f"{what}: {worst} is {dist[worst]:.2e} from the oracle's chain"


@pytest.mark.parametrize("overlap", [True, False])
def test_decode_step_s1024(nm, weights, ref1024, overlap):
    w, dw = weights
    h, cache_ref, r = ref1024
    cache_in = gen.mla_cache(1024, DIMS, seed=4200)
    t = run_step(nm, dw, h, cache_in, 1024, overlap=overlap)
    check_step(t, r, cache_ref, 1024, w, h)


@pytest.mark.parametrize("S", [1, 300, 1024, 7000])
def test_decode_step_with_the_kv_chain_beside_the_attention_pass(nm, weights, S):
    """Two-stream schedule, KV chain forked when the attention operand is ready: the narrow product h * (W_DKV | W_KR) with its
    RMSNorm / RoPE / cache-row write runs on the side stream while the tensor-core pass attends the old rows; the merge
    waits for it.  Same stages, same criteria; and the bits of the ordinary two-stream schedule."""
    w, dw = weights
    h, cache_ref, r = oracle_step(w, S, seed=4550 + S)
    cache_in = gen.mla_cache(S, DIMS, seed=4550 + S)
    early = run_step(nm, dw, h, cache_in, S, overlap=True)
    nm.nm_debug_set_step_kv_beside_attention(True)
    try:
        late = run_step(nm, dw, h, cache_in, S, overlap=True)
    finally:
        nm.nm_debug_set_step_kv_beside_attention(False)
    check_step(late, r, cache_ref, S, w, h, what=f"KV chain beside attention, S={S}")
    for k in ("out", "o", "o_lat", "q_full", "kv_cache"):
        assert torch.equal(early[k], late[k]), k


@pytest.mark.parametrize("S", [1, 70, 1024])
def test_decode_step_with_concatenated_down_projections(nm, weights, S):
    # h * (W_DQ | W_DKV | W_KR) as one product on one stream (Eq. 3's concatenation extended by W_DQ)
    w, dw = weights
    h, cache_ref, r = oracle_step(w, S, seed=4500 + S)
    cache_in = gen.mla_cache(S, DIMS, seed=4500 + S)
    t = run_step(nm, dw, h, cache_in, S, concat_down=True)
    check_step(t, r, cache_ref, S, w, h)


@pytest.mark.parametrize("concat_down", [True, False])
def test_decode_step_with_the_dense_weights_in_fractal_storage(nm, weights, concat_down):
    """The storage of the paper's test case: W_DQ, W_DKV|W_KR (or the three as one matrix), W_UQR and W_O in 16 x 16
    fractals ordered by columns.  Same logical matrices as the row-major fixture, so the same oracle reference."""
    w, dw = weights
    S = 700
    h, cache_ref, r = oracle_step(w, S, seed=4600)
    cache_in = gen.mla_cache(S, DIMS, seed=4600)
    d, ql, dkv = DIMS["d"], DIMS["q_lora"], DIMS["kv_lora"] + DIMS["rope"]
    H, dq, dv = DIMS["H"], DIMS["nope"] + DIMS["rope"], DIMS["v"]
    nz = dict(dw)
    shapes = {"W_DQ": (d, ql), "W_DKVKR": (d, dkv), "W_UQR": (ql, H * dq), "W_O": (H * dv, d)}
    for name, (K, N) in shapes.items():
        nz[name] = to_dev(gen.to_fractal_nz(np.asarray(w[name]).reshape(K, N)))
    if concat_down:      # run_step concatenates the (row-major) fixtures; store that concatenation in fractals instead
        cat = np.concatenate([np.asarray(w["W_DQ"]).reshape(d, ql), np.asarray(w["W_DKVKR"]).reshape(d, dkv)], axis=1)
        nz["W_DQKV"] = to_dev(gen.to_fractal_nz(cat))
        nz.pop("W_DQ"); nz.pop("W_DKVKR")
    t = run_step(nm, nz, h, cache_in, S, layout_dense=2)
    check_step(t, r, cache_ref, S, w, h)
    # the oracle on the fractal storage itself gives the same reference (its index formula, pinned on its own)
    wnz = dict(w)
    for name, (K, N) in shapes.items():
        wnz[name] = gen.to_fractal_nz(np.asarray(w[name]).reshape(K, N))
    r2 = oracle.mla_decode_step(DIMS, wnz, h, gen.mla_cache(S, DIMS, seed=4600), S, layout_dense=2, threads=8)
    assert np.array_equal(np.asarray(r2["out"]), np.asarray(r["out"]))


@pytest.mark.parametrize("S", [1, 2, 65, 4096])
def test_decode_step_other_lengths(nm, weights, S):
    w, dw = weights
    h, cache_ref, r = oracle_step(w, S, seed=4300 + S)
    cache_in = gen.mla_cache(S, DIMS, seed=4300 + S)
    t = run_step(nm, dw, h, cache_in, S)
    check_step(t, r, cache_ref, S, w, h)


def test_decode_step_fused_and_unfused_per_head_stages_agree(nm, weights, ref1024):
    w, dw = weights
    h, cache_ref, r = ref1024
    cache_in = gen.mla_cache(1024, DIMS, seed=4200)
    t1 = run_step(nm, dw, h, cache_in, 1024)
    nm.nm_debug_set_step_fusion(False)
    try:
        t2 = run_step(nm, dw, h, cache_in, 1024)
        check_step(t2, r, cache_ref, 1024, w, h)
    finally:
        nm.nm_debug_set_step_fusion(True)
    # the two routes sum in different orders: q_full is the same bf16 value up to a rounding flip on a few
    # elements; what follows the softmax inherits those flips and is compared on the scale of the tensor
    a, b = dev_bits_to_f64(t1["q_full"]), dev_bits_to_f64(t2["q_full"])
    assert np.all(np.abs(a - b) <= 2 * oracle.ulp_bf16(b) + 1e-6)
    assert np.mean(a == b) > 0.97
    for k in ("o_lat", "o", "out"):
        a, b = dev_bits_to_f64(t1[k]), dev_bits_to_f64(t2[k])
        assert np.all(np.abs(a - b) <= 2e-3 * np.abs(b).max() + oracle.ulp_bf16(b)), k      # rounded outputs: one ulp on top


@pytest.mark.parametrize("concat_down", [False, True])
def test_decode_step_vector_stages_inside_and_outside_the_products_agree(nm, weights, ref1024, concat_down):
    # RMSNorm / RoPE / cache-row write in the completion of the down-projection products (default) against the
    # same stages as kernels of their own: both routes against the oracle, and against each other
    w, dw = weights
    h, cache_ref, r = ref1024
    cache_in = gen.mla_cache(1024, DIMS, seed=4200)
    # three forms: 1 (default) - with the down-projections stored as one matrix: k-splits meeting in clusters, RMSNorm of
    # the query latent applied by W_UQR while loading its row, KV consumers in an extra CTA of the per-head query
    # kernel; 2 - the CTA completing the product's last tile runs the stages; 0 - kernels of their own
    t1 = run_step(nm, dw, h, cache_in, 1024, concat_down=concat_down)
    check_step(t1, r, cache_ref, 1024, w, h)
    for mode in (2, 0):
        nm.nm_debug_set_step_tails(mode)
        try:
            t2 = run_step(nm, dw, h, cache_in, 1024, concat_down=concat_down)
            check_step(t2, r, cache_ref, 1024, w, h)
        finally:
            nm.nm_debug_set_step_tails(1)
        # the products are bit-identical (same summation order); the norms sum their squares in a
        # different order, so c_qn and the cache row may differ by a rounding flip
        for k in ("c_q", "ckr"):
            assert torch.equal(t1[k], t2[k]), (mode, k)
        for k in ("c_qn", "kv_cache"):
            a, b = dev_bits_to_f64(t1[k]), dev_bits_to_f64(t2[k])
            assert np.all(np.abs(a - b) <= oracle.ulp_bf16(b) + 1e-6), (mode, k)
            assert np.mean(a == b) > 0.99, (mode, k)


def test_decode_step_forced_product_plans_inside_the_step(nm, weights, ref1024):
    # the step's products under other tilings / k-splits / ring depths than the planner's: same result within
    # the bound (parity against the oracle), the plan goes back to the planner afterwards
    w, dw = weights
    h, cache_ref, r = ref1024
    cache_in = gen.mla_cache(1024, DIMS, seed=4200)
    try:
        for which, plan in ((0, (64, 7, 3)), (1, (256, 2, 4)), (2, (128, 3, 5)), (2, (64, 2, 5))):
            nm.nm_debug_set_step_plan(which, *plan)
            t = run_step(nm, dw, h, cache_in, 1024, concat_down=True)
            check_step(t, r, cache_ref, 1024, w, h)
            nm.nm_debug_set_step_plan(which, 0, 0, 0)
    finally:
        for which in range(3):
            nm.nm_debug_set_step_plan(which, 0, 0, 0)


def test_decode_step_without_wo_and_repeatable(nm, weights):
    w, dw = weights
    S = 300
    h, cache_ref, r = oracle_step(w, S, seed=4400, with_wo=False)
    cache_in = gen.mla_cache(S, DIMS, seed=4400)
    t1 = run_step(nm, dw, h, cache_in, S, with_wo=False)
    check_step(t1, r, cache_ref, S, w, h, with_wo=False)
    t2 = run_step(nm, dw, h, cache_in, S, with_wo=False)
    for k in ("c_q", "q_full", "o_lat", "o"):
        assert torch.equal(t1[k], t2[k]), f"{k}: two runs differ"


def test_decode_step_same_bits_with_and_without_programmatic_launch(nm, weights, ref1024):
    w, dw = weights
    h, cache_ref, r = ref1024
    cache_in = gen.mla_cache(1024, DIMS, seed=4200)
    t1 = run_step(nm, dw, h, cache_in, 1024)
    nm.nm_debug_set_step_pdl(False)
    try:
        t2 = run_step(nm, dw, h, cache_in, 1024)
    finally:
        nm.nm_debug_set_step_pdl(True)
    for k in ("c_q", "c_qn", "q", "q_full", "ckr", "o_lat", "o", "out", "kv_cache"):
        assert torch.equal(t1[k], t2[k]), k
    check_step(t2, r, cache_ref, 1024, w, h)


def test_decode_step_back_to_back_steps_do_not_interfere(nm, weights, ref1024):
    # several steps enqueued without host synchronisation in between: programmatic launch lets a
    # step's first kernels overlap the previous step's tail; results must not change
    w, dw = weights
    h, cache_ref, r = ref1024
    H, dc, dr, dn, dv, d, ql = (DIMS[k] for k in ("H", "kv_lora", "rope", "nope", "v", "d", "q_lora"))
    t = dict(dw)
    t["h"] = to_dev(h)
    t["kv_cache"] = to_dev(gen.mla_cache(1024, DIMS, seed=4200))
    t["rope_cos_sin"] = rope_row(nm, 1023)
    t["out"] = torch.zeros(d, dtype=torch.int16, device="cuda")
    p = nm.mla_params(DIMS, 1024, t)
    ws = nm.new_workspace(nm.nm_mla_workspace_bytes(p))
    p = nm.mla_params(DIMS, 1024, t, workspace=ws)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    with torch.cuda.stream(main):
        for _ in range(6):
            nm.nm_mla_decode_step(p, main, side)
            outs.append(t["out"].clone())
    torch.cuda.synchronize()
    nm.nm_check_status()
    for o in outs[1:]:
        assert torch.equal(o, outs[0])
    ref = f64(r["out"])
    assert np.all(np.abs(dev_bits_to_f64(outs[0]) - ref) <= 2e-3 * np.abs(ref).max() + oracle.ulp_bf16(ref))


@pytest.mark.parametrize("S", [4096, 16384])
def test_decode_step_in_the_configuration_the_bench_times(nm, weights, S):
    # the bench's launch configuration at its full sizes: the three down-projections stored as one matrix (one
    # stream, six kernels), the step's first product allowed to start under the previous step's tail, steps
    # enqueued back to back without a host synchronisation; every output element against the oracle
    w, dw = weights
    h, cache_ref, r = oracle_step(w, S, seed=4600 + S)
    H, dc, dr, dn, dv, d, ql = (DIMS[k] for k in ("H", "kv_lora", "rope", "nope", "v", "d", "q_lora"))
    dkv = dc + dr
    t = dict(dw)
    t["W_DQKV"] = torch.cat([t.pop("W_DQ").view(d, ql), t.pop("W_DKVKR").view(d, dkv)], dim=1).contiguous().view(-1)
    t["h"] = to_dev(h)
    t["kv_cache"] = to_dev(gen.mla_cache(S, DIMS, seed=4600 + S))
    t["rope_cos_sin"] = rope_row(nm, S - 1)
    t["out"] = torch.zeros(d, dtype=torch.int16, device="cuda")
    t["o_lat_f32"] = torch.zeros(H * dc, dtype=torch.float32, device="cuda")
    p = nm.mla_params(DIMS, S, t)
    ws = nm.new_workspace(nm.nm_mla_workspace_bytes(p))
    p = nm.mla_params(DIMS, S, t, workspace=ws)
    p.programmatic_entry = 1
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    with torch.cuda.stream(main):
        for _ in range(4):
            nm.nm_mla_decode_step(p, main, side)
            outs.append(t["out"].clone())
    torch.cuda.synchronize()
    nm.nm_check_status()
    for o in outs[1:]:
        assert torch.equal(o, outs[0])
    # on these fixed inputs the two chains agree closely enough that the stated criteria also hold end to end
    o32 = t["o_lat_f32"].cpu().numpy().astype(np.float64).reshape(H, dc)
    assert rel_max(o32, r["o_lat_f64"]) <= 2e-3
    ref = f64(r["out"]).reshape(-1)
    assert np.all(np.abs(dev_bits_to_f64(outs[0]) - ref) <= 2e-3 * np.abs(ref).max() + oracle.ulp_bf16(ref))
    # once more with every stage output requested (the copies that deliver them sit between the kernels, so this is
    # not the timed configuration any more): same result bit for bit, and every stage at its criterion
    dq = dn + dr
    for k, n in {"c_q": ql, "c_qn": ql, "q": H * dq, "q_full": H * dkv, "ckr": dkv, "o_lat": H * dc, "o": H * dv}.items():
        t[k] = torch.zeros(n, dtype=torch.int16, device="cuda")
    p2 = nm.mla_params(DIMS, S, t, workspace=ws)
    p2.programmatic_entry = 1
    with torch.cuda.stream(main):
        nm.nm_mla_decode_step(p2, main, side)
    torch.cuda.synchronize()
    nm.nm_check_status()
    assert torch.equal(t["out"], outs[0])
    check_step(t, r, cache_ref, S, w, h, what="bench configuration")


def test_decode_step_replayed_from_a_cuda_graph(nm, weights, ref1024):
    # both streams, the events between them and the programmatic launches are captured once; replays must
    # reproduce the directly launched result bit for bit
    w, dw = weights
    h, cache_ref, r = ref1024
    d = DIMS["d"]
    t = dict(dw)
    t["h"] = to_dev(h)
    t["kv_cache"] = to_dev(gen.mla_cache(1024, DIMS, seed=4200))
    t["rope_cos_sin"] = rope_row(nm, 1023)
    t["out"] = torch.zeros(d, dtype=torch.int16, device="cuda")
    p = nm.mla_params(DIMS, 1024, t)
    ws = nm.new_workspace(nm.nm_mla_workspace_bytes(p))
    p = nm.mla_params(DIMS, 1024, t, workspace=ws)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(main):
        nm.nm_mla_decode_step(p, main, side)          # direct launch (also does every one-time set-up)
        torch.cuda.synchronize()
        direct = t["out"].clone()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=main):
            nm.nm_mla_decode_step(p, main, side)
        for _ in range(3):
            t["out"].zero_()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(t["out"], direct)
    nm.nm_check_status()
    ref = f64(r["out"])
    assert np.all(np.abs(dev_bits_to_f64(direct) - ref) <= 2e-3 * np.abs(ref).max() + oracle.ulp_bf16(ref))


def test_decode_step_host_operands(nm, weights, ref1024):
    w, dw = weights
    h, cache_ref, r = ref1024
    d = DIMS["d"]
    t = dict(dw)
    t["kv_cache"] = to_dev(gen.mla_cache(1024, DIMS, seed=4200))
    t["rope_cos_sin"] = rope_row(nm, 1023)
    t["h"] = torch.zeros(d, dtype=torch.int16, device="cuda")
    t["out"] = torch.zeros(d, dtype=torch.int16, device="cuda")
    p = nm.mla_params(DIMS, 1024, t)
    ws = nm.new_workspace(nm.nm_mla_workspace_bytes(p))
    p = nm.mla_params(DIMS, 1024, t, workspace=ws)
    h_host = torch.from_numpy(h.view(np.int16).copy()).pin_memory()
    out_host = torch.zeros(d, dtype=torch.int16).pin_memory()
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    nm.nm_mla_decode_step_host(p, h_host, out_host, t["h"], t["out"], main, side)
    torch.cuda.synchronize()
    ref = f64(r["out"])
    got = oracle.bf16_to_f64(out_host.numpy().view(np.uint16))
    assert np.all(np.abs(got - ref) <= 2e-3 * np.abs(ref).max() + oracle.ulp_bf16(ref))
    # the same call again and again with another token written into the SAME pinned buffer in between (the token is fetched
    # from host memory by a kernel: it must see the new bytes every time), also replayed from a CUDA graph; each result
    # equals the device-operand step on that token, bit for bit
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=main):
        nm.nm_mla_decode_step_host(p, h_host, out_host, t["h"], t["out"], main, side)
    for k in range(4):
        tok = gen.mla_token(DIMS, seed=4700 + k)
        h_host.copy_(torch.from_numpy(tok.view(np.int16).copy()))
        out_host.zero_()
        if k % 2 == 0:
            nm.nm_mla_decode_step_host(p, h_host, out_host, t["h"], t["out"], main, side)
        else:
            g.replay()
        torch.cuda.synchronize()
        t2 = dict(t)
        t2["h"] = to_dev(tok)
        t2["out"] = torch.zeros(d, dtype=torch.int16, device="cuda")
        p2 = nm.mla_params(DIMS, 1024, t2, workspace=ws)
        nm.nm_mla_decode_step(p2, main, side)
        torch.cuda.synchronize()
        assert torch.equal(out_host, t2["out"].cpu()), f"token {k}"
    nm.nm_check_status()


def test_step_error_codes(nm, weights):
    _, dw = weights
    t = dict(dw)
    p = nm.mla_params(DIMS, 16, t)                          # h, cache, table, workspace missing
    with pytest.raises(nm.NmError) as e:
        nm.nm_mla_decode_step(p)
    assert e.value.status == -1
