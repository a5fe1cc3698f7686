"""Small-batch decode (nm_mla_decode_batch): T independent sequences, one new token each, against T runs of
the oracle's single-token step, and against the library's own single-token step."""
import numpy as np
import pytest
import torch

import nm_inputs as gen
import oracle
from gpu_util import END_TO_END_BOUND, assert_step_stage_by_stage, end_to_end_distance, to_dev

pytestmark = pytest.mark.gpu
DIMS = gen.DSV3_DIMS


def f64(bits):
    return oracle.bf16_to_f64(np.asarray(bits, dtype=np.uint16))


def dev_bits_to_f64(t):
    return oracle.bf16_to_f64(t.contiguous().cpu().numpy().view(np.uint16))


@pytest.fixture(scope="module")
def nm():
    import paper_2609_16009_b200 as nm
    yield nm
    nm.nm_check_status()


@pytest.fixture(scope="module")
def weights():
    w = gen.mla_weights(DIMS, seed=4000, with_wo=True)
    return w, {k: to_dev(v) for k, v in w.items()}


def run_batch(nm, dw, tokens, caches, seq_lens, concat_down, with_wo=True, graph=False, back_to_back=0):
    H, dc, dr, dn, dv, d, ql = (DIMS[k] for k in ("H", "kv_lora", "rope", "nope", "v", "d", "q_lora"))
    dkv = dc + dr
    T = len(seq_lens)
    t = dict(dw)
    if not with_wo:
        t.pop("W_O")
    if concat_down:
        t["W_DQKV"] = torch.cat([t.pop("W_DQ").view(d, ql), t.pop("W_DKVKR").view(d, dkv)], dim=1).contiguous().view(-1)
    stride = (max(seq_lens) + 3) * dkv                      # a few spare rows between the sequences' caches
    stride += (-stride) % 8
    cache = torch.zeros(T * stride, dtype=torch.int16, device="cuda")
    for i, c in enumerate(caches):
        cache[i * stride:i * stride + c.size] = to_dev(c).view(-1)
    h = to_dev(np.stack(tokens))
    cs = torch.empty(T, dr, dtype=torch.float32, device="cuda")
    for i, S in enumerate(seq_lens):
        nm.nm_rope_table(cs[i], S - 1, 1, dr)
    out = torch.zeros(T * d, dtype=torch.int16, device="cuda")
    q_full = torch.zeros(T * H * dkv, dtype=torch.int16, device="cuda")
    o_lat = torch.zeros(T * H * dc, dtype=torch.int16, device="cuda")
    o = torch.zeros(T * H * dv, dtype=torch.int16, device="cuda")
    dq = dn + dr
    c_q, c_qn = (torch.zeros(T * ql, dtype=torch.int16, device="cuda") for _ in range(2))
    q = torch.zeros(T * H * dq, dtype=torch.int16, device="cuda")
    ckr = torch.zeros(T * dkv, dtype=torch.int16, device="cuda")
    p = nm.mla_params(DIMS, 1, t)
    ws = nm.new_workspace(nm.nm_mla_batch_workspace_bytes(p, T))
    p = nm.mla_params(DIMS, 1, t, workspace=ws)
    b = nm.mla_batch(seq_lens, h, cs, cache, stride, out=out, q_full=q_full, o_lat=o_lat, o=o, c_q=c_q, c_qn=c_qn, q=q, ckr=ckr)
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    if back_to_back:                                         # the same step several times in a row, each allowed to start under its predecessor
        p.programmatic_entry = 1
        for _ in range(back_to_back):
            nm.nm_mla_decode_batch(p, b, st)
    elif graph:                                                # captured once, replayed: the call allocates and synchronises nothing
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            nm.nm_mla_decode_batch(p, b, st)
        g.replay()
    else:
        nm.nm_mla_decode_batch(p, b, st)
    torch.cuda.synchronize()
    nm.nm_check_status()
    return {"out": out.view(T, d), "q_full": q_full.view(T, H, dkv), "o_lat": o_lat.view(T, H, dc), "o": o.view(T, H * dv),
            "c_q": c_q.view(T, ql), "c_qn": c_qn.view(T, ql), "q": q.view(T, H * dq), "ckr": ckr.view(T, dkv),
            "cache": cache.view(T, stride), "stride": stride}


def rel_max(got, ref):
    return np.abs(got - ref).max() / np.abs(ref).max()


def check_against_oracle(w, res, tokens, caches, seq_lens, with_wo=True):
    """Each sequence of the batch as a single-token step: every stage against the oracle on the GPU's own input to that
    stage at the stated criteria (gpu_util.assert_step_stage_by_stage) - this covers the batch-only kernels of the query
    side (RMSNorm and the cache-row write after the down-projections, RoPE, the per-head products in both forms) as well as
    the attention pass and the output side; old cache rows bit for bit; and the end-to-end distance to the oracle's own
    chain, printed and held to one fixed bound."""
    H, dc, dr = DIMS["H"], DIMS["kv_lora"], DIMS["rope"]
    dkv = dc + dr
    ww = dict(w)
    if not with_wo:
        ww.pop("W_O", None)
    worst = {}
    for i, S in enumerate(seq_lens):
        r = oracle.mla_decode_step(DIMS, ww, tokens[i], caches[i], S, threads=8)
        cache_ref = caches[i]                                # the oracle wrote row S-1 in place
        got = res["cache"][i].cpu().numpy().view(np.uint16)[:S * dkv].reshape(S, dkv)
        assert np.array_equal(got[:S - 1], cache_ref[:S - 1]), f"sequence {i}: old rows changed"
        g = {k: res[k][i] for k in ("c_q", "c_qn", "q", "q_full", "ckr", "o_lat", "o")}
        g["cache"] = got
        g["out"] = res["out"][i] if with_wo else None
        assert_step_stage_by_stage(DIMS, ww, tokens[i], S - 1, g, f"sequence {i} (S {S})")
        refs = {"q_full": np.concatenate([np.asarray(r["q_lat"]), np.asarray(r["q_rope"])], axis=1), "o_lat": r["o_lat"], "o": r["o"]}
        if with_wo:
            refs["out"] = r["out"]
        for k, v in refs.items():
            worst[k] = max(worst.get(k, 0.0), end_to_end_distance(res[k][i], v))
        worst["cache row"] = max(worst.get("cache row", 0.0), end_to_end_distance(got[S - 1], cache_ref[S - 1]))
    print(f"batch of {len(seq_lens)}: end-to-end distance to the oracle's chain: " + ", ".join(f"{k} {v:.1e}" for k, v in worst.items()))
    k = max(worst, key=worst.get)
    assert worst[k] <= END_TO_END_BOUND, f"{k} is {worst[k]:.2e} from the oracle's chain"


def make_inputs(seq_lens, seed):
    tokens = [gen.mla_token(DIMS, seed=seed + 10 * i) for i in range(len(seq_lens))]
    caches = [gen.mla_cache(S, DIMS, seed=seed + 10 * i + 1) for i, S in enumerate(seq_lens)]
    return tokens, caches


@pytest.mark.parametrize("seq_lens,concat", [([300], True), ([1, 70], True), ([1024, 65, 2, 500], True), ([129, 64, 1000], False),
                                             ([200, 1, 333, 64, 65, 1500, 2, 700], True)])
def test_batch_matches_oracle(nm, weights, seq_lens, concat):
    w, dw = weights
    tokens, caches = make_inputs(seq_lens, seed=8000 + len(seq_lens))
    res = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, concat)
    check_against_oracle(w, res, tokens, caches, seq_lens)


@pytest.mark.parametrize("seq_lens,with_wo", [([300], True), ([90, 1, 257], True), ([1024, 65, 2, 500, 130], True),
                                              ([64 + 31 * i for i in range(12)], False),
                                              # split plans of the attention pass with clusters of 1, 2 and 4 merged on chip
                                              ([650 + 17 * i for i in range(7)], False), ([900 - 13 * i for i in range(6)], False),
                                              ([300 + 41 * i for i in range(10)], False), ([1100, 900, 1000], False)])
def test_batch_with_the_per_head_products_as_batched_products(nm, weights, seq_lens, with_wo):
    """From three sequences on the per-head products run as batched products (tensor cores from M = 3) with RoPE and
    the merge as kernels of their own; below, fused per-head kernels do them.  Here the first form at every batch
    size (the switch that turns the fused per-head kernels off), against the oracle."""
    w, dw = weights
    tokens, caches = make_inputs(seq_lens, seed=8300 + len(seq_lens))
    nm.nm_debug_set_step_fusion(False)
    try:
        res = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True, with_wo=with_wo)
    finally:
        nm.nm_debug_set_step_fusion(True)
    check_against_oracle(w, res, tokens, caches, seq_lens, with_wo=with_wo)


@pytest.mark.parametrize("seq_lens,with_wo", [([513, 64, 2], True), ([300, 1, 70, 1024, 65], True), ([40 + 53 * i for i in range(16)], False)])
def test_batch_with_the_fused_per_head_kernels_at_every_size(nm, weights, seq_lens, with_wo):
    """The fused per-head kernels (one CTA per head walking every token) stay selectable beyond the two sequences they
    serve by default."""
    w, dw = weights
    tokens, caches = make_inputs(seq_lens, seed=8400 + len(seq_lens))
    nm.nm_debug_set_batch_per_head_min_tokens(17)
    try:
        res = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True, with_wo=with_wo)
    finally:
        nm.nm_debug_set_batch_per_head_min_tokens(3)
    check_against_oracle(w, res, tokens, caches, seq_lens, with_wo=with_wo)


@pytest.mark.parametrize("seq_lens", [[700, 650, 600, 90, 333, 1000], [257, 64]])
def test_batch_replayed_from_a_cuda_graph(nm, weights, seq_lens):
    w, dw = weights
    tokens, caches = make_inputs(seq_lens, seed=8500 + len(seq_lens))
    direct = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True)
    replayed = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True, graph=True)
    for k in ("out", "q_full", "o_lat", "o", "cache"):
        assert torch.equal(direct[k], replayed[k]), k
    check_against_oracle(w, replayed, tokens, caches, seq_lens)


@pytest.mark.parametrize("seq_lens", [[700, 650, 90, 333], [64] * 16])
def test_batch_steps_back_to_back_with_programmatic_entry(nm, weights, seq_lens):
    """programmatic_entry: the first product of a step may start (weights only) while the previous step's W_O product is
    still running.  Three steps in a row on the same buffers give the bits of one step on its own."""
    w, dw = weights
    tokens, caches = make_inputs(seq_lens, seed=8600 + len(seq_lens))
    alone = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True)
    chained = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True, back_to_back=3)
    for k in ("out", "q_full", "o_lat", "o", "cache", "c_q", "q"):
        assert torch.equal(alone[k], chained[k]), k
    check_against_oracle(w, chained, tokens, caches, seq_lens)


def test_batch_of_sixteen_without_wo(nm, weights):
    w, dw = weights
    seq_lens = [40 + 37 * i for i in range(16)]
    tokens, caches = make_inputs(seq_lens, seed=8100)
    res = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True, with_wo=False)
    check_against_oracle(w, res, tokens, caches, seq_lens, with_wo=False)


def test_batch_is_repeatable_and_rejects_bad_arguments(nm, weights):
    w, dw = weights
    seq_lens = [100, 257]
    tokens, caches = make_inputs(seq_lens, seed=8200)
    a = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True)
    b = run_batch(nm, dw, tokens, [c.copy() for c in caches], seq_lens, True)
    for k in ("out", "o", "o_lat", "q_full"):
        assert torch.equal(a[k], b[k]), k
    t = dict(dw)
    p = nm.mla_params(DIMS, 1, t)
    ws = nm.new_workspace(nm.nm_mla_batch_workspace_bytes(p, 2))
    p = nm.mla_params(DIMS, 1, t, workspace=ws)
    dkv = DIMS["kv_lora"] + DIMS["rope"]
    cache = torch.zeros(2 * 300 * dkv, dtype=torch.int16, device="cuda")
    h = torch.zeros(2 * DIMS["d"], dtype=torch.int16, device="cuda")
    cs = torch.zeros(2 * DIMS["rope"], dtype=torch.float32, device="cuda")
    out = torch.zeros(2 * DIMS["d"], dtype=torch.int16, device="cuda")
    with pytest.raises(nm.NmError):                          # cache stride smaller than a sequence
        nm.nm_mla_decode_batch(p, nm.mla_batch([100, 257], h, cs, cache, 200 * dkv, out=out))
    with pytest.raises(nm.NmError):                          # empty sequence
        nm.nm_mla_decode_batch(p, nm.mla_batch([100, 0], h, cs, cache, 300 * dkv, out=out))
    with pytest.raises(nm.NmError):                          # more sequences than the library takes
        nm.nm_mla_decode_batch(p, nm.mla_batch([5] * 17, h, cs, cache, 8 * dkv, out=out))
    small = nm.new_workspace(1 << 20)
    p2 = nm.mla_params(DIMS, 1, t, workspace=small)
    with pytest.raises(nm.NmError):                          # workspace too small
        nm.nm_mla_decode_batch(p2, nm.mla_batch([100, 257], h, cs, cache, 300 * dkv, out=out))
