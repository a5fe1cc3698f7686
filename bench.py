#!/usr/bin/env python
"""Benchmark of the narrow-MatMul / MLA-decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mla|projections] [--seq-len S]
    python bench.py --impl reference ...        # the CPU oracle on the host cores (reported baseline)

One step is one pass of the whole hot path over one token.  Prints ONE JSON line (rank 0).
`value` is the algorithmic HBM traffic of a step (weights + activations + KV rows, each once)
divided by the device time of the step, summed over ranks: GB/s.  `ms_per_step` is the decode
latency.  Every rank runs an independent replica (the path has no exchange step): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import nm_inputs as gen  # noqa: E402

DIMS = gen.DSV3_DIMS
L2_BYTES = 126 * 1024 * 1024


# --------------------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------------------
def projection_specs(dims=DIMS):
    """The narrow products of one decode step at M = 1: (name, K, N, heads)."""
    d, ql, dc, dr, dn, dv, H = (dims[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
    return [("W_DQ", d, ql, 1), ("W_DKVKR", d, dc + dr, 1), ("W_UQR", ql, H * (dn + dr), 1),
            ("W_UK", dn, dc, H), ("W_UV", dc, dv, H), ("W_O", H * dv, d, 1)]


def algorithmic_bytes(specs, M=1):
    return sum((K * N + M * K + M * N) * 2 * H for _, K, N, H in specs)


class ProjectionChain:
    """All narrow products of the decode step, M = 1, each fed a resident activation vector."""

    name = "projections"

    def __init__(self, nm, device, seed=4000):
        self.nm = nm
        self.specs = projection_specs()
        w = gen.mla_weights(DIMS, seed=seed, with_wo=True)
        self.W = {k: torch.from_numpy(w[k].view(np.int16)).to(device) for k in ("W_DQ", "W_DKVKR", "W_UQR", "W_UK", "W_UV", "W_O")}
        self.h_host = torch.from_numpy(gen.mla_token(DIMS, seed=seed + 100).view(np.int16).copy()).pin_memory()
        self.x = {}
        self.y = {}
        for name, K, N, H in self.specs:
            self.x[name] = torch.from_numpy(gen.normal_bf16((H * K,), 1.0, seed + 200 + len(self.x)).view(np.int16)).to(device)
            self.y[name] = torch.empty(H * N, dtype=torch.int16, device=device)
        self.out_host = torch.empty(DIMS["d"], dtype=torch.int16).pin_memory()
        need = max(nm.nm_matmul_workspace_bytes(1, N, K, H) for _, K, N, H in self.specs)
        self.ws = nm.new_workspace(need, device=device)
        self.bytes_per_step = algorithmic_bytes(self.specs)
        self.dominant = "W_O"
        self.dominant_bytes = algorithmic_bytes([s for s in self.specs if s[0] == "W_O"])
        self.launches_per_step = len(self.specs)
        self.h2d = self.h_host.numel() * 2
        self.d2h = self.out_host.numel() * 2

    def describe(self):
        return {"workload": "narrow products of one DeepSeek-V3 MLA decode step, M=1 (W_DQ 7168x1536, W_DKV|KR 7168x576, "
                            "W_UQR 1536x24576, W_UK/W_UV per head x128, W_O 16384x7168), bf16 row-major",
                "l2": "weights 374 MB per step > 126 MB L2, so every step streams from HBM; no flush"}

    def launch(self, name, stream):
        nm = self.nm
        _, K, N, H = next(s for s in self.specs if s[0] == name)
        if H == 1:
            nm.nm_matmul_ws(self.x[name], self.W[name], self.y[name], 1, N, K, nm.BF16, nm.ROW_MAJOR, self.ws, stream)
        else:
            nm.nm_matmul_batched_ws(self.x[name], self.W[name], self.y[name], 1, N, K, H, H * K, K, K * N, H * N, N,
                                    nm.BF16, nm.ROW_MAJOR, self.ws, stream)

    def step(self, stream, dom_events=None):
        for name, _, _, _ in self.specs:
            if dom_events is not None and name == self.dominant:
                dom_events[0].record(stream)
                self.launch(name, stream)
                dom_events[1].record(stream)
            else:
                self.launch(name, stream)

    def step_e2e(self, stream):
        # token in from pinned host memory, result out to pinned host memory, inside the timed region
        self.x["W_DQ"].copy_(self.h_host, non_blocking=True)
        self.step(stream)
        self.out_host.copy_(self.y["W_O"], non_blocking=True)


def ncu_dram_bytes(path):
    """dram__bytes_read.sum + dram__bytes_write.sum (bytes) from a text summary of an ncu capture, or None."""
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    total, seen = 0.0, 0
    try:
        for line in open(path):
            f = line.split()
            if len(f) >= 3 and f[0] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and f[2] in scale:
                total += float(f[1].replace(",", "")) * scale[f[2]]
                seen += 1
    except OSError:
        return None
    return int(round(total)) if seen == 2 else None


class MlaStep:
    """The whole single-token decode step (nm_mla_decode_step): Q chain, KV chain on a side stream,
    tensor-core latent attention over the cache, output side including W_O."""

    name = "mla"

    def __init__(self, nm, device, seq_len, seed=4000, schedule="fused", weights="row", share=None):
        self.nm = nm
        self.S = seq_len
        self.schedule = schedule
        self.weights = weights
        d, ql, dc, dr, dn, dv, H = (DIMS[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
        if share is not None:
            # the same resident weights (and token) at another sequence length: own cache, table, output and workspace
            self._finish(nm, device, seq_len, seed, dict(share.t), share.layout_dense, share.h_host)
            return
        w = gen.mla_weights(DIMS, seed=seed, with_wo=True)
        t = {k: torch.from_numpy(v.view(np.int16)).to(device) for k, v in w.items()}
        if schedule == "fused":
            # the three down-projections stored as one matrix (W_DQ | W_DKV | W_KR): a storage choice made
            # when the weights are loaded, like the paper's concatenation of W_DKV and W_KR
            t["W_DQKV"] = torch.from_numpy(np.concatenate([w["W_DQ"], w["W_DKVKR"]], axis=1).view(np.int16)).to(device)
            del t["W_DQ"], t["W_DKVKR"]
        layout_dense = nm.ROW_MAJOR
        if weights == "fractal":
            # the storage of the paper's test case: the dense weights in 16 x 16 fractals (a permutation of the same values)
            layout_dense = nm.FRACTAL_NZ
            shapes = {"W_DQKV": (d, ql + dc + dr), "W_DQ": (d, ql), "W_DKVKR": (d, dc + dr), "W_UQR": (ql, H * (dn + dr)), "W_O": (H * dv, d)}
            for name, (K_, N_) in shapes.items():
                if name in t:
                    t[name] = torch.from_numpy(gen.to_fractal_nz(t[name].cpu().numpy().reshape(K_, N_))).to(device)
        h_host = torch.from_numpy(gen.mla_token(DIMS, seed=seed + 100).view(np.int16).copy()).pin_memory()
        t["h"] = h_host.to(device)
        self._finish(nm, device, seq_len, seed, t, layout_dense, h_host)

    def _finish(self, nm, device, seq_len, seed, t, layout_dense, h_host):
        d, ql, dc, dr, dn, dv, H = (DIMS[k] for k in ("d", "q_lora", "kv_lora", "rope", "nope", "v", "H"))
        schedule = self.schedule
        self.layout_dense = layout_dense
        self.h_host = h_host
        self.out_host = torch.empty(d, dtype=torch.int16).pin_memory()
        t["out"] = torch.zeros(d, dtype=torch.int16, device=device)
        t["kv_cache"] = torch.from_numpy(gen.mla_cache(seq_len, DIMS, seed=seed + 200).view(np.int16)).to(device)
        t["rope_cos_sin"] = torch.empty(dr, dtype=torch.float32, device=device)
        nm.nm_rope_table(t["rope_cos_sin"], seq_len - 1, 1, dr)
        self.t = t
        p = nm.mla_params(DIMS, seq_len, t, layout_dense=layout_dense)
        self.ws = nm.new_workspace(nm.nm_mla_workspace_bytes(p), device=device)
        self.p = nm.mla_params(DIMS, seq_len, t, workspace=self.ws, layout_dense=layout_dense)
        self.p.programmatic_entry = 1        # steps follow each other like the layers of a model: weights are static
        self.side = torch.cuda.Stream(device)
        self.graph = None
        self.graph_error = None
        self.specs = projection_specs()
        self.kv_bytes = seq_len * (dc + dr) * 2 + (dc + dr) * 2        # rows read once + the row written
        self.bytes_per_step = algorithmic_bytes(self.specs) + self.kv_bytes
        self.dominant = "W_O product (nm_row_tma_kernel, K=16384, N=7168, M=1)"
        self.dominant_bytes = algorithmic_bytes([s for s in self.specs if s[0] == "W_O"])
        # dram__bytes_read.sum + dram__bytes_write.sum of one launch of this kernel on this shape, read from the
        # committed summary of its ncu capture (None if the file is not there)
        self.dominant_traffic_source = "profiles/ncu_nm_row_tma_WO_M1_K16384_N7168.txt"
        self.dominant_traffic = ncu_dram_bytes(os.path.join(ROOT, self.dominant_traffic_source))
        self.launches_per_step = 6 if schedule == "fused" else 7
        # two-stream schedules: the KV chain beside the first Q-chain product, or beside the attention pass
        nm.nm_debug_set_step_kv_beside_attention(schedule == "kv-beside-attention")
        self.h2d = d * 2
        self.d2h = d * 2

    def describe(self):
        return {"workload": f"full single-token MLA decode step, DeepSeek-V3 dims (hidden 7168, q_lora 1536, kv_lora 512, rope 64, "
                            f"nope 128, v 128, 128 heads), seq_len {self.S}, bf16 weights "
                            + ("row-major" if self.weights == "row" else "in FRACTAL_NZ storage") + ", W_O included",
                "seq_len": self.S,
                "l2": "weights 374 MB per step > 126 MB L2, so every step streams from HBM; no flush",
                "schedule": self.schedule,
                "overlap": ("one stream: h*(W_DQ|W_DKV|W_KR) as one product; " if self.schedule == "fused" else
                            ("two streams: KV chain (W_DKV|KR product, RMSNorm, RoPE, cache write) beside the W_DQ product; "
                             if self.schedule == "two-stream" else
                             "two streams: KV chain (W_DKV|KR product on CUDA cores, RMSNorm, RoPE, cache write) beside the tcgen05 attention pass; "))
                           + "RMSNorm / RoPE / cache write inside the completion of the products that feed them; L2 prefetch of "
                             "W_UV and 40 MB of W_O while the tcgen05 attention kernel runs; programmatic dependent launch along "
                             "the chain, also across steps"}

    def step(self, stream, dom_events=None):
        if dom_events is not None:
            self.p.event_before_wo, self.p.event_after_wo = dom_events[0].cuda_event, dom_events[1].cuda_event
        else:
            self.p.event_before_wo, self.p.event_after_wo = None, None
        self.nm.nm_mla_decode_step(self.p, stream, self.side)

    def batch_step(self, T, stream):
        """The small-batch step (nm_mla_decode_batch) on T sequences of this length, one new token each: returns the
        call and the buffers it uses (to be kept alive by the caller)."""
        dkv = DIMS["kv_lora"] + DIMS["rope"]
        stride = (self.S + 8) * dkv
        cache = self.t["kv_cache"].view(-1)[:self.S * dkv].repeat(T, 1)
        cache = torch.nn.functional.pad(cache, (0, stride - self.S * dkv)).contiguous().view(-1)
        h = self.t["h"].repeat(T)
        cs = self.t["rope_cos_sin"].repeat(T)
        res = torch.zeros(T * DIMS["d"], dtype=torch.int16, device=cache.device)
        ws = self.nm.new_workspace(self.nm.nm_mla_batch_workspace_bytes(self.p, T), device=cache.device)
        pb = self.nm.mla_params(DIMS, 1, self.t, workspace=ws)
        pb.programmatic_entry = 1            # steps follow each other; the weights are static
        b = self.nm.mla_batch([self.S] * T, h, cs, cache, stride, out=res)
        return (lambda: self.nm.nm_mla_decode_batch(pb, b, stream)), (cache, h, cs, res, ws, pb, b)

    def extra_measurements(self, stream):
        """Outside the timed region, reported beside it: the same step replayed from a CUDA graph of ten steps
        (device time without per-launch work of the host-side queue), and the step without its last product
        (W_O = NULL; it is 63 % of the step's bytes)."""
        out = {}
        def timed(fn, n):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(n):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b)
        self.p.event_before_wo, self.p.event_after_wo = None, None
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(10):
                    self.nm.nm_mla_decode_step(self.p, stream, self.side)
            g.replay(); torch.cuda.synchronize()
            out["graph_replay"] = {"decode_us": min(timed(g.replay, 20) for _ in range(3)) / 200 * 1e3, "steps_per_graph": 10}
            del g
        except Exception as exc:          # capture is an extra; the main number does not depend on it
            out["graph_replay"] = {"error": repr(exc)}
        # the small-batch step (nm_mla_decode_batch): T sequences of this length, one new token each
        out["small_batch"] = []
        for T in ((4, 8, 12, 16) if self.weights == "row" else ()):       # the batch entry point takes row- / column-major weights
            fn, keep = self.batch_step(T, stream)
            timed(fn, 20)
            us = min(timed(fn, 100) for _ in range(3)) / 100 * 1e3
            nb = self.bytes_per_step - self.kv_bytes + T * self.kv_bytes       # weights once, every sequence's cache rows
            out["small_batch"].append({"T": T, "step_us": us, "us_per_token": us / T, "tokens_per_s": T / us * 1e6,
                                       "GBps": nb / us / 1e3})
            del fn, keep
        wo = self.p.W_O
        self.p.W_O = None
        try:
            fn = lambda: self.nm.nm_mla_decode_step(self.p, stream, self.side)
            timed(fn, 50)
            us = min(timed(fn, 200) for _ in range(3)) / 200 * 1e3
            nb = self.bytes_per_step - self.dominant_bytes
            out["without_W_O"] = {"decode_us": us, "GBps": nb / us / 1e3, "algorithmic_bytes": nb}
        finally:
            self.p.W_O = wo
        return out

    def step_e2e(self, stream):
        """Token in from pinned host memory, step, result out to pinned host memory.  The whole
        sequence (two copies, the kernels of both streams) is captured once into a CUDA graph and
        replayed, so that a step costs one launch on the host."""
        if self.graph is None:
            self.p.event_before_wo, self.p.event_after_wo = None, None
            g = torch.cuda.CUDAGraph()
            try:
                with torch.cuda.graph(g, stream=stream):
                    self.nm.nm_mla_decode_step_host(self.p, self.h_host, self.out_host, self.t["h"], self.t["out"], stream, self.side)
                self.graph = g
            except Exception as exc:                      # capture refused: fall back to direct launches
                self.graph = False
                self.graph_error = str(exc)[:200]
        if self.graph:
            self.graph.replay()
        else:
            self.p.event_before_wo, self.p.event_after_wo = None, None
            self.nm.nm_mla_decode_step_host(self.p, self.h_host, self.out_host, self.t["h"], self.t["out"], stream, self.side)


class SingleProduct:
    """One narrow product C[MxN] = A[MxK] * B[KxN] (bf16, or fp32 in and out), B rotated through copies that
    together exceed 512 MB (256 copies at most: 256 MB for the 1 MiB fp32 case, still above the L2) so that every
    launch streams from HBM.  For kernel-level captures."""

    name = "matmul"

    def __init__(self, nm, device, M, K, N, layout, dtype="bf16"):
        self.nm, self.M, self.K, self.N, self.layout = nm, M, K, N, layout
        self.dtype_name = dtype
        self.dtype = nm.F32 if dtype == "f32" else nm.BF16
        tdt, es = (torch.float32, 4) if dtype == "f32" else (torch.bfloat16, 2)
        nbytes = K * N * es
        self.R = max(2, min(256, (1 << 29) // nbytes + 1))
        if dtype == "f32":                                   # the fp32 GEMV case: values uniform in [-1, 1]
            self.B = torch.rand(self.R, K * N, device=device) * 2 - 1
            self.A = torch.rand(M * K, device=device) * 2 - 1
        else:
            self.B = (torch.randn(self.R, K * N, device=device) * 0.02).to(tdt)
            self.A = torch.randn(M * K, device=device).to(tdt)
        self.C = torch.empty(M * N, device=device, dtype=tdt)
        self.A_host = self.A.cpu().pin_memory()
        self.C_host = torch.empty(M * N, dtype=tdt).pin_memory()
        self.ws = nm.new_workspace(nm.nm_matmul_workspace_bytes(M, N, K, 1, self.dtype, layout), device=device)
        self.i = 0
        self.bytes_per_step = (K * N + M * K + M * N) * es
        self.dominant = f"narrow product M={M} K={K} N={N}"
        self.dominant_bytes = self.bytes_per_step
        self.launches_per_step = 1
        self.h2d, self.d2h = M * K * es, M * N * es

    def describe(self):
        return {"workload": f"single narrow product M={self.M} K={self.K} N={self.N} {self.dtype_name}, B {'column' if self.layout else 'row'}-major",
                "l2": f"B rotates through {self.R} copies (> 512 MB in total): every launch reads HBM"}

    def step(self, stream, dom_events=None):
        self.i = (self.i + 1) % self.R
        if dom_events is not None:
            dom_events[0].record(stream)
        self.nm.nm_matmul_ws(self.A, self.B[self.i], self.C, self.M, self.N, self.K, self.dtype, self.layout, self.ws, stream)
        if dom_events is not None:
            dom_events[1].record(stream)

    def step_e2e(self, stream):
        self.i = (self.i + 1) % self.R
        self.nm.nm_matmul_host(self.A_host, self.B[self.i], self.C_host, self.A, self.C, self.M, self.N, self.K, self.dtype,
                               self.layout, self.ws, stream)


class AttentionOnly:
    """The latent-attention pass alone (tcgen05 kernel + merge) over seq_len cache rows."""

    name = "attention"

    def __init__(self, nm, device, seq_len):
        self.nm, self.S = nm, seq_len
        H, dc, dr = DIMS["H"], DIMS["kv_lora"], DIMS["rope"]
        self.Q = (torch.randn(H, dc + dr, device=device) * 0.3).to(torch.bfloat16)
        self.cache = torch.randn(seq_len, dc + dr, device=device).to(torch.bfloat16)
        self.o = torch.empty(H * dc, dtype=torch.bfloat16, device=device)
        self.ws = torch.empty(nm.nm_mla_attention_workspace_bytes(H, seq_len, dc), dtype=torch.uint8, device=device)
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        self.bytes_per_step = (seq_len + H) * (dc + dr) * 2 + H * dc * 2
        self.flops_per_step = 2 * H * seq_len * (dc + dr + dc)
        self.dominant = "attn_tc_kernel"
        self.dominant_bytes = self.bytes_per_step
        self.launches_per_step = 2
        self.h2d = self.d2h = 0

    def describe(self):
        return {"workload": f"latent attention pass alone, 128 heads, seq_len {self.S}", "l2": "256 MB written between launches"}

    def step(self, stream, dom_events=None):
        H, dc, dr = DIMS["H"], DIMS["kv_lora"], DIMS["rope"]
        self.flush.fill_(1)
        if dom_events is not None:
            dom_events[0].record(stream)
        self.nm.nm_mla_attention(self.Q, self.cache, self.o, None, H, self.S, -1, dc, dr, (DIMS["nope"] + dr) ** -0.5, self.ws, stream)
        if dom_events is not None:
            dom_events[1].record(stream)

    step_e2e = step


def make_workload(args, nm, device):
    if args.workload == "projections":
        return ProjectionChain(nm, device)
    if args.workload == "mla":
        return MlaStep(nm, device, args.seq_len, schedule=args.schedule, weights=args.weights)
    if args.workload == "matmul":
        M, K, N = (int(x) for x in args.mkn.split(","))
        return SingleProduct(nm, device, M, K, N, 1 if args.layout == "col" else 0, args.dtype)
    if args.workload == "attention":
        return AttentionOnly(nm, device, args.seq_len)
    raise SystemExit(f"unknown workload {args.workload}")


def print_timeline(wl, stream, steps=6):
    """Kernel timeline of one step (start offset, duration, name) from CUPTI through torch.profiler:
    shows which kernels overlap (side-stream work beside the main stream, programmatic launches)."""
    from torch.profiler import ProfilerActivity, profile
    with profile(activities=[ProfilerActivity.CUDA]) as prof:
        for _ in range(steps):
            wl.step(stream)
        torch.cuda.synchronize()
    evs = sorted((e for e in prof.events() if e.device_type == torch.autograd.DeviceType.CUDA), key=lambda e: e.time_range.start)
    per = len(evs) // steps
    k0 = (steps - 2) * per
    t0 = evs[k0].time_range.start
    print(f"# kernel timeline of one step ({per} kernels), microseconds from the step's first kernel")
    for e in evs[k0:k0 + per]:
        print(f"{e.time_range.start - t0:9.1f}  +{e.time_range.end - e.time_range.start:7.1f}  {e.name[:90]}")
    print(f"# next step starts at {evs[k0 + per].time_range.start - t0:.1f}")


def batched_case(nm, device, T, K, N, H):
    """One batched per-head product (bf16, row-major weights [H][K][N], activations [T][H][K]) timed like the
    other sweep cases: CUDA-graph replay over rotating copies of the weights, serial and programmatic."""
    nbytes = H * K * N * 2
    R = max(2, min(64, (1 << 29) // nbytes + 1))
    Bs = (torch.randn(R, H * K * N, device=device) * 0.02).to(torch.bfloat16)
    A = torch.randn(T * H * K, device=device).to(torch.bfloat16)
    C = torch.empty(R, T * H * N, device=device, dtype=torch.bfloat16)
    ws = nm.new_workspace(nm.nm_matmul_workspace_bytes(T, N, K, H), device=device)
    s = torch.cuda.Stream(device)
    row = {"M": T, "K": K, "N": N, "H": H, "dtype": "bf16", "layout_B": "row", "batched": True}
    algo = (H * K * N + T * H * K + T * H * N) * 2
    def launch(i):
        nm.nm_matmul_batched_ws(A, Bs[i], C[i], T, N, K, H, H * K, K, K * N, H * N, N, nm.BF16, nm.ROW_MAJOR, ws, s)
    for mode in ("serial", "programmatic"):
        nm.nm_set_programmatic_launch(mode == "programmatic")
        with torch.cuda.stream(s):
            for i in range(R):
                launch(i)
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for i in range(R):
                    launch(i)
            g.replay(); s.synchronize()
            ts = []
            for _ in range(21):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s); g.replay(); b.record(s); s.synchronize()
                ts.append(a.elapsed_time(b) * 1e3 / R)
        ts.sort()
        us = statistics.median(ts)
        key = "" if mode == "serial" else "_programmatic"
        row["us" + key] = round(us, 2)
        row["us_mean_p5_p95" + key] = [round(statistics.mean(ts), 2), round(ts[1], 2), round(ts[-2], 2)]
        row["GBps" + key] = round(algo / us / 1e3, 1)
        del g
    nm.nm_set_programmatic_launch(False)
    row["pct_of_8TBs"] = round(max(row["GBps"], row["GBps_programmatic"]) / 80.0, 1)
    return row


def read_only_stream(nm, device):
    """GB/s of a kernel that only reads 1 GiB once (nm_debug_stream_read: the products' own streaming load, nothing
    else), best of the CTA counts tried: what a read-only stream reaches on this GPU, beside the copy bandwidth
    that the roofline uses as its peak."""
    n = 1 << 30
    buf = torch.empty(n, dtype=torch.uint8, device=device)
    buf.random_(0, 255)
    sink = torch.zeros(1, dtype=torch.int32, device=device)
    s = torch.cuda.Stream(device)
    best = {}
    with torch.cuda.stream(s):
        for ctas in (2, 4, 8):
            for _ in range(3):
                nm.nm_debug_stream_read(buf, n, sink, ctas, s)
            ts = []
            for _ in range(9):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s); nm.nm_debug_stream_read(buf, n, sink, ctas, s); b.record(s); s.synchronize()
                ts.append(a.elapsed_time(b))
            gbs = n / (statistics.median(ts) * 1e-3) / 1e9
            if not best or gbs > best["GBps"]:
                best = {"GBps": round(gbs, 1), "ctas_per_sm": ctas, "bytes": n}
    return best


def matmul_sweep(nm, device, args_no_cpu=False, compact=False, peak=None):
    """GB/s of single narrow products (cold L2: the launches of a CUDA graph rotate through copies of
    B that together exceed 512 MB).  Two figures per case: launches in plain stream order (each kernel
    starts when the one before has finished: latency of an isolated call plus the launch gap), and
    launched programmatically (a kernel may fetch its weights while its predecessor drains, as inside
    the decode step).  Reported beside the step; not part of the timed region.
    compact: the configurations the metric names and the GPU legs only (the default line); otherwise also the
    fractal storage, 17 and 64 rows, the paper's 100 x 100 schedule, warm-L2 figures and the oracle's times."""
    out = []
    cases = [(1, 512, 512, 0, "f32"), (1, 7168, 1536, 0, "bf16"), (1, 7168, 576, 0, "bf16"), (1, 7168, 1536, 1, "bf16"),
             (1, 7168, 576, 1, "bf16")]
    if not compact:
        # the storage the paper's test case has in memory (16 x 16 fractals): layout code 2
        cases += [(1, 7168, 1536, 2, "bf16"), (1, 7168, 576, 2, "bf16"), (1, 7168, 18432, 2, "bf16")]
    for M in (1, 2, 4, 8, 16):
        cases += [(M, 1536, 24576, 0, "bf16"), (M, 7168, 18432, 0, "bf16")]
    if not compact:
        # beyond the narrow range: a remainder row on top of 16, and 64 rows, still one pass over B (tensor cores)
        cases += [(17, 7168, 18432, 0, "bf16"), (64, 7168, 18432, 0, "bf16")]
    # the per-head products of the absorbed MLA form, T tokens at once: q_nope * W_UK (128 -> 512) and
    # o_lat * W_UV (512 -> 128), 128 heads, activations laid out [T][128][K]
    for T in (1, 4, 16):
        cases += [(T, 128, 512, 0, "bf16", 128), (T, 512, 128, 0, "bf16", 128)]
    for case in cases:
        M, K, N, layout, dt = case[:5]
        H = case[5] if len(case) > 5 else 1
        if H > 1:
            out.append(batched_case(nm, device, M, K, N, H))
            if peak:
                out[-1]["frac_of_measured"] = round(max(out[-1]["GBps"], out[-1]["GBps_programmatic"]) / peak, 3)
            continue
        es = 4 if dt == "f32" else 2
        tdt = torch.float32 if dt == "f32" else torch.bfloat16
        code = nm.F32 if dt == "f32" else nm.BF16
        nbytes = K * N * es
        R = max(2, min(512, (1 << 29) // nbytes + 1))        # copies of B that together exceed 512 MB (4 x the L2)
        Bs = (torch.randn(R, K * N, device=device) * 0.02).to(tdt)
        A = torch.randn(M * K, device=device).to(tdt)
        C = torch.empty(R, M * N, device=device, dtype=tdt)
        ws = nm.new_workspace(nm.nm_matmul_workspace_bytes(M, N, K), device=device)
        s = torch.cuda.Stream(device)
        row = {"M": M, "K": K, "N": N, "dtype": dt, "layout_B": ("row", "col", "fractal_nz")[layout], "copies_of_B": R}
        algo = (K * N + M * K + M * N) * es
        for mode in ("serial", "programmatic"):
            nm.nm_set_programmatic_launch(mode == "programmatic")
            with torch.cuda.stream(s):
                for i in range(R):
                    nm.nm_matmul_ws(A, Bs[i], C[i], M, N, K, code, layout, ws, s)
                s.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=s):
                    for i in range(R):
                        nm.nm_matmul_ws(A, Bs[i], C[i], M, N, K, code, layout, ws, s)
                g.replay(); s.synchronize()
                ts = []
                for _ in range(21):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(s); g.replay(); b.record(s); s.synchronize()
                    ts.append(a.elapsed_time(b) * 1e3 / R)
            ts.sort()
            us = statistics.median(ts)
            key = "" if mode == "serial" else "_programmatic"
            row["us" + key] = round(us, 2)
            row["us_mean_p5_p95" + key] = [round(statistics.mean(ts), 2), round(ts[1], 2), round(ts[-2], 2)]
            row["GBps" + key] = round(algo / us / 1e3, 1)
            del g
        nm.nm_set_programmatic_launch(False)
        row["pct_of_8TBs"] = round(max(row["GBps"], row["GBps_programmatic"]) / 80.0, 1)
        row["pct_of_8TBs_serial"] = round(row["GBps"] / 80.0, 1)
        if peak:
            row["frac_of_measured"] = round(max(row["GBps"], row["GBps_programmatic"]) / peak, 3)
            row["frac_of_measured_serial"] = round(row["GBps"] / peak, 3)
        if compact:
            out.append(row)
            del Bs, C
            continue
        # the paper's own schedule (its evaluation section): 100 runs of 100 iterations, the first iteration of
        # every run dropped; direct launches in stream order, B rotating through the copies (cold L2)
        with torch.cuda.stream(s):
            runs = []
            for r in range(100):
                nm.nm_matmul_ws(A, Bs[r % R], C[r % R], M, N, K, code, layout, ws, s)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s)
                for i in range(1, 100):
                    nm.nm_matmul_ws(A, Bs[(r + i) % R], C[(r + i) % R], M, N, K, code, layout, ws, s)
                b.record(s); s.synchronize()
                runs.append(a.elapsed_time(b) * 1e3 / 99)
            runs.sort()
            row["us_100x100"] = round(statistics.mean(runs), 2)
            row["us_100x100_p5_p95"] = [round(runs[5], 2), round(runs[94], 2)]
            # the same weights on every launch: what a matrix that fits the 126 MB L2 costs when it is already there
            if nbytes < 100e6:
                for i in range(5):
                    nm.nm_matmul_ws(A, Bs[0], C[0], M, N, K, code, layout, ws, s)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(s)
                for i in range(100):
                    nm.nm_matmul_ws(A, Bs[0], C[0], M, N, K, code, layout, ws, s)
                b.record(s); s.synchronize()
                row["us_warm_l2"] = round(a.elapsed_time(b) * 1e3 / 100, 2)
        # the oracle's time for the same product on the host cores (all it may use, and one thread), best of three
        # after a warm-up pass; for M > 1 on the large matrices a bounded sample: the first row only
        if not args_no_cpu:
            import oracle
            threads = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
            Mo = M if (M * K * N <= 3e8) else 1
            An = (np.random.default_rng(1).standard_normal((Mo, K)).astype(np.float32))
            Bn = (np.random.default_rng(2).standard_normal(K * N).astype(np.float32) * 0.02)
            if dt == "bf16":
                An = (An.view(np.uint32) >> 16).astype(np.uint16); Bn = (Bn.view(np.uint32) >> 16).astype(np.uint16)
            odt = oracle.F32 if dt == "f32" else oracle.BF16
            def run(th):
                best = 1e9
                for rep in range(4):
                    t0 = time.perf_counter()
                    oracle.matmul(An, Bn, Mo, N, K, odt, odt, layout, threads=th)
                    if rep: best = min(best, time.perf_counter() - t0)
                return best * 1e3
            row["oracle_ms"] = {"rows": Mo, "cores": threads, "all_cores": round(run(threads), 2),
                                "one_thread": round(run(1), 2) if Mo * K * N <= 5e7 else None}
        out.append(row)
        del Bs, C
    return out


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                if r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
# CPU oracle arm
# --------------------------------------------------------------------------------------------------
_ORACLE_INPUTS = {}


def oracle_sample(threads, kind="mla", seq_len=16384):
    """One pass of the oracle, as it stands, on the host cores over the same workload: the naive
    decode step at `seq_len` (kind "mla") or the six narrow products alone (kind "projections").
    Returns (seconds, algorithmic bytes, description)."""
    import oracle
    specs = projection_specs()
    key = (kind, seq_len)
    if key not in _ORACLE_INPUTS:
        w = gen.mla_weights(DIMS, seed=4000, with_wo=True)
        oracle.lib()
        if kind == "mla":
            _ORACLE_INPUTS[key] = (w, gen.mla_token(DIMS, seed=4100), gen.mla_cache(seq_len, DIMS, seed=4200))
        else:
            _ORACLE_INPUTS[key] = (w, {name: gen.normal_bf16((H * K,), 1.0, 4200 + i) for i, (name, K, N, H) in enumerate(specs)}, None)
    w, x, cache = _ORACLE_INPUTS[key]
    t0 = time.perf_counter()
    if kind == "mla":
        oracle.mla_decode_step(DIMS, w, x, cache, seq_len, threads=threads)
        dt = time.perf_counter() - t0
        nbytes = algorithmic_bytes(specs) + (seq_len + 1) * (DIMS["kv_lora"] + DIMS["rope"]) * 2
        return dt, nbytes, f"the whole naive decode step at seq_len {seq_len} (374 MB of bf16 weights + cache), one pass"
    for name, K, N, H in specs:
        if H == 1:
            oracle.matmul(x[name], w[name], 1, N, K, oracle.BF16, oracle.BF16, oracle.ROW_MAJOR, threads=threads)
        else:
            oracle.matmul_batched(x[name], w[name], 1, N, K, H, H * K, K, K * N, H * N, N, H * N,
                                  oracle.BF16, oracle.BF16, oracle.ROW_MAJOR, threads=threads)
    dt = time.perf_counter() - t0
    return dt, algorithmic_bytes(specs), "all six narrow products of one decode step at M=1 (374 MB of bf16 weights), one pass"


def run_reference(args, rank):
    if rank != 0:
        return
    import oracle
    # every core this process may run on: under torchrun the other ranks do no work, and its OMP_NUM_THREADS=1 default would
    # otherwise put the whole oracle on one core (14 s per step instead of 0.6)
    threads = len(os.sched_getaffinity(0))
    steps = min(args.steps, 20)              # bounded: the oracle is slow by design
    for _ in range(min(args.warmup, 2)):
        oracle_sample(threads, args.workload, args.seq_len)
    times, nbytes, what = [], 0, ""
    for _ in range(steps):
        dt, nbytes, what = oracle_sample(threads, args.workload, args.seq_len)
        times.append(dt)
    total = sum(times)
    value = nbytes * len(times) / total / 1e9
    line = {"impl": "reference", "metric": "narrow MatMul HBM GB/s (% of 8 TB/s) vs M; MLA single-token decode \u00b5s", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": total / len(times) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "CPU oracle (fp64 triple loop) on a bounded sample: " + what},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": what},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# main arm
# --------------------------------------------------------------------------------------------------
def reduce_over_ranks(values, dist, device):
    """Max over ranks of per-rank timings (every rank runs an independent replica; the job's step
    time is that of the slowest rank).  `dist` is torch.distributed or None for a single process."""
    if dist is None:
        return list(values)
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput_gbs(bytes_per_step, steps, world, ms):
    """Whole-job GB/s: every rank moves bytes_per_step per step; time is the slowest rank's."""
    return bytes_per_step * steps * world / (ms * 1e-3) / 1e9


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mla", choices=["mla", "projections", "matmul", "attention"])
    ap.add_argument("--mkn", default="1,16384,7168", help="M,K,N of --workload matmul")
    ap.add_argument("--layout", default="row", choices=["row", "col"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"], help="operand type of --workload matmul")
    ap.add_argument("--schedule", default="fused", choices=["fused", "two-stream", "kv-beside-attention"],
                    help="decode step: down-projections as one concatenated product on one stream, or W_DKV|KR on a side stream")
    ap.add_argument("--timeline", action="store_true", help="print the kernel timeline of one step and exit")
    ap.add_argument("--sweep", action="store_true", help="the full product sweep: more cases, the paper's 100 x 100 schedule, warm-L2 figures, oracle times")
    ap.add_argument("--seq-len", type=int, default=16384, help="cache rows of the headline step (default: the largest configuration)")
    ap.add_argument("--single-length", action="store_true", help="skip the step at the other sequence lengths (1024, 4096, 16384)")
    ap.add_argument("--no-sweep", action="store_true", help="skip the narrow-product-vs-M measurements")
    ap.add_argument("--single-block", action="store_true", help="time one block of --steps steps only (no repetition up to half a second): for traces")
    ap.add_argument("--no-extras", action="store_true", help="skip graph replay, the small-batch step and the step without W_O")
    ap.add_argument("--batch", type=int, default=1, help="sequences of the small-batch step (2-16) to run instead of the single-token step (captures, --timeline)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--weights", default="row", choices=["row", "fractal"],
                    help="storage of the step's dense weights: row-major (default) or the paper's FRACTAL_NZ tiling")
    ap.add_argument("--attention", default="auto", choices=["auto", "64", "128", "cuda-cores"],
                    help="attention kernel: chosen by length (default), tensor cores with 64 or 128 heads per CTA, CUDA cores")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    import paper_2609_16009_b200 as nm
    nm.nm_debug_set_attention({"auto": 0, "cuda-cores": 1, "128": 2, "64": 3}[args.attention])
    wl = make_workload(args, nm, device)
    stream = torch.cuda.Stream(device)
    if args.batch > 1 and not args.timeline:
        # the small-batch step as the workload (for kernel-level captures; extras and the other lengths are skipped)
        if args.workload != "mla" or args.weights != "row":
            raise SystemExit("--batch goes with --workload mla and row-major weights")
        fn, keep = wl.batch_step(args.batch, stream)

        def _batch_step(stream_, dom_events=None):       # the batch call has no event hooks: the "dominant kernel" is the whole step
            if dom_events is not None:
                dom_events[0].record(stream_)
            fn()
            if dom_events is not None:
                dom_events[1].record(stream_)
        wl.step = _batch_step
        wl.step_e2e = lambda stream_: fn()               # device operands only: no host leg in this mode
        wl.h2d = wl.d2h = 0
        wl.extra_measurements = lambda stream_: {}
        wl.launches_per_step = 9 if args.batch >= 3 else 7     # T >= 3: RoPE, the per-head products and the merge as kernels of their own
        wl.bytes_per_step = wl.bytes_per_step - wl.kv_bytes + args.batch * wl.kv_bytes      # weights once, every sequence's cache rows
        single = wl.describe()
        single["workload"] = (f"small-batch MLA decode step (nm_mla_decode_batch): {args.batch} sequences of seq_len {wl.S}, one new token each, "
                              "DeepSeek-V3 dims, bf16 weights row-major, W_O included; GB/s = weights once + every sequence's cache rows")
        single["batch"] = args.batch
        wl.describe = lambda: single
        wl.dominant = "the whole batch step (nm_mla_decode_batch has no per-kernel event hooks)"
        wl.dominant_bytes = wl.bytes_per_step
        wl.dominant_traffic = wl.dominant_traffic_source = None
        args.single_length = args.no_sweep = True
    if args.timeline:
        with torch.cuda.stream(stream):
            if args.batch > 1:                # the timeline of the small-batch step instead of the single-token step
                if args.workload != "mla" or args.weights != "row":
                    raise SystemExit("--batch goes with --workload mla and row-major weights")
                fn, keep = wl.batch_step(args.batch, stream)
                wl.step = lambda stream_, dom_events=None: fn()
            for _ in range(max(args.warmup, 10)):
                wl.step(stream)
            torch.cuda.synchronize()
            print_timeline(wl, stream)
        return

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_block(fn, n):
        """Device time (ms) of n calls of fn, bracketed by a barrier + synchronize on both sides."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        barrier()
        return e0.elapsed_time(e1)

    # the clock sampler covers everything from the warm-up to the last extra measurement
    sampler = ClockSampler(local_rank)
    sampler.start()
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            wl.step(stream)
        barrier()
        # ---- device-timed region: blocks of exactly `steps` steps, inputs resident in HBM.  A block shorter than
        #      half a second is repeated until half a second of device time has gone by (the same count on every
        #      rank), and the MEDIAN block is reported; nothing but the steps is enqueued inside a block ------------
        first = timed_block(lambda: wl.step(stream), args.steps)
        (first_max,) = reduce_over_ranks([first], dist, device)
        n_blocks = 1 if (first_max >= 500.0 or args.single_block) else int(min(200, max(3, -(-500.0 // max(first_max, 1e-3)))))
        blocks = [first] + [timed_block(lambda: wl.step(stream), args.steps) for _ in range(n_blocks - 1)]
        # ---- the dominant kernel, in a SEPARATE pass after the timed region: events around it on the launching
        #      stream in every step (the events switch off that kernel's programmatic launch, which is why they are
        #      kept out of the timed region) ---------------------------------------------------------------------
        n_dom = 64
        dom = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_dom)]
        for a, b in dom:                      # events get their handles on first record
            a.record(stream); b.record(stream)
        barrier()
        for i in range(n_dom):
            wl.step(stream, dom[i])
        barrier()
        dom_ms = statistics.mean(a.elapsed_time(b) for a, b in dom[8:])
        # ---- end-to-end region: host token in, host result out, every step -----------------------------
        for _ in range(3):
            wl.step_e2e(stream)
        barrier()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(args.steps):
            wl.step_e2e(stream)
            stream.synchronize()              # the host reads the result of every step
        t1.record(stream)
        barrier()
        e2e_ms = t0.elapsed_time(t1)
        extras = wl.extra_measurements(stream) if (hasattr(wl, "extra_measurements") and not args.no_extras) else {}
        # ---- the step at the other sequence lengths of the configuration (same resident weights) ------------------
        per_len = []
        if args.workload == "mla" and not args.single_length:
            for S in sorted({1024, 4096, 16384, args.seq_len}):
                w2 = wl if S == args.seq_len else MlaStep(nm, device, S, schedule=args.schedule, weights=args.weights, share=wl)
                if w2 is wl:
                    per_len.append((S, w2.bytes_per_step, None))
                    continue
                for _ in range(max(args.warmup, 20)):
                    w2.step(stream)
                n = max(args.steps, 200)
                per_len.append((S, w2.bytes_per_step, statistics.median(timed_block(lambda: w2.step(stream), n) for _ in range(3)) / n))
                del w2
    nm.nm_check_status(stream)

    blocks = [reduce_over_ranks([b], dist, device)[0] for b in blocks]
    ms = statistics.median(blocks)
    e2e_ms, dom_ms = reduce_over_ranks([e2e_ms, dom_ms], dist, device)
    per_len = [(S, nb, reduce_over_ranks([t], dist, device)[0] if t is not None else ms / args.steps) for S, nb, t in per_len]

    if rank == 0:
        peak, peak_kind = load_peaks()
        value = job_throughput_gbs(wl.bytes_per_step, args.steps, world, ms)
        e2e_value = job_throughput_gbs(wl.bytes_per_step, args.steps, world, e2e_ms)
        achieved = wl.dominant_bytes / (dom_ms * 1e-3) / 1e9
        line = {"metric": "narrow MatMul HBM GB/s (% of 8 TB/s) vs M; MLA single-token decode \u00b5s", "value": value, "unit": "GB/s",
                "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "decode_us": ms / args.steps * 1e3,
                "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": wl.describe(),
                "pct_of_8TBs": value / world / 8000.0,
                "frac_of_measured_peak": value / world / peak,
                "timed_blocks": {"blocks": len(blocks), "steps_per_block": args.steps, "reported": "median block",
                                 "ms_min_median_max": [min(blocks), ms, max(blocks)]},
                "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": wl.h2d, "d2h_bytes_per_step": wl.d2h,
                        "ms_per_step": e2e_ms / args.steps,
                        "launch": ("cuda graph replay" if getattr(wl, "graph", None) else "direct launches"),
                        "graph_error": getattr(wl, "graph_error", None)},
                "gpu_launches": wl.launches_per_step * args.steps * len(blocks),
                "roofline": {"bound": "hbm", "kernel": wl.dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                             "frac": achieved / peak, "peak_kind": peak_kind, "algorithmic_bytes": wl.dominant_bytes,
                             "traffic": getattr(wl, "dominant_traffic", None),
                             "traffic_source": getattr(wl, "dominant_traffic_source", None),
                             "us_per_launch": dom_ms * 1e3,
                             "measured": f"separate pass of {n_dom} steps after the timed region (first 8 dropped), CUDA events around the "
                                         "kernel on the launching stream; the events switch off that kernel's programmatic launch"}}
        if per_len:
            line["decode_vs_seq_len"] = [{"seq_len": S, "decode_us": t * 1e3, "GBps": nb / t / 1e6, "pct_of_8TBs": nb / t / 1e6 / 80.0,
                                          "frac_of_measured_peak": nb / t / 1e6 / peak, "algorithmic_bytes": nb} for S, nb, t in per_len]
        line.update(extras)
        if args.workload == "mla" and not args.no_sweep:
            # the metric's first half: narrow products vs M (GPU legs; --sweep adds the oracle's times and more cases)
            with torch.cuda.stream(stream):
                line["narrow_matmul_vs_M"] = matmul_sweep(nm, device, args.no_cpu_baseline, compact=not args.sweep, peak=peak)
                if args.sweep:
                    line["read_only_stream"] = read_only_stream(nm, device)
        elif args.sweep:
            line["narrow_matmul_vs_M"] = matmul_sweep(nm, device, args.no_cpu_baseline, peak=peak)
            line["read_only_stream"] = read_only_stream(nm, device)
        line["clocks"] = sampler.stop()
        if not args.no_cpu_baseline:
            import oracle
            threads = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
            oracle_sample(threads, args.workload, args.seq_len)                    # warm-up pass (page faults, thread pool)
            total, passes, nbytes, what = 0.0, 0, 0, ""
            while total < 10.0 and passes < 200:                                   # about ten seconds of CPU work
                dt, nbytes, what = oracle_sample(threads, args.workload, args.seq_len)
                total += dt
                passes += 1
            line["cpu_baseline"] = {"value": nbytes * passes / total / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                    "sample": f"{passes} passes of " + what.replace(", one pass", ""), "seconds": total,
                                    "ms_per_step": total / passes * 1e3}
        print(json.dumps(line), flush=True)
    else:
        sampler.stop()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
