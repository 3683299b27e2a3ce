#!/usr/bin/env python
"""Benchmark of the UniGist attention hot path on B200.

One step = one pass of the whole path over one synthetic batch, in the order a training /
prefill step runs it: gist shift of Q, K, V, dO -> forward (O, LSE) -> backward (dQ, dK, dV) ->
unshift of O, dQ, dK, dV -> KV compaction into the paged cache -> one decode query per sequence
over the compacted cache.  Where the tiles line up (ratio divides 128, head_dim 128, no sinks) the
shift and unshift are not separate launches: the attention kernels read the interleaved tensors
through tile maps that pick the raw rows or the gist row of each gist unit and store their results
at interleaved rows; the step with explicit shift launches is timed too and reported beside it.  The headline value is the effective TFLOP/s of forward + backward
counting only unmasked (visible) pairs: 14 * D * pairs * Hq * B FLOP per step / step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (launched by torchrun) every rank runs an independent replica of the workload (the
path has no exchange step); the value is the work of all ranks over the slowest rank's time.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
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
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "effective_tflops_fwd_bwd_unmasked"
UNIT = "TFLOP/s"

# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures
# summarised under profiles/, keyed by (kernel, workload); None until a capture exists.
NCU_TRAFFIC_BYTES = {
    ("attn_fwd_sm100_kernel", "llama8b_layer"): 353900000,
    ("attn_bwd_fused_sm100_kernel", "llama8b_layer"): 4827655000,
}

# FLOP per visible pair per query head that each attention kernel performs algorithmically,
# in units of head_dim (a QK^T- or PV-shaped product is 2 * D FLOP per pair).
KERNEL_FLOP_PER_PAIR_D = {
    "bwd_dq_simt_kernel": 6, "bwd_dkdv_simt_kernel": 8,
    "attn_fwd_sm100_kernel": 4, "attn_bwd_dq_sm100_kernel": 6, "attn_bwd_dkdv_sm100_kernel": 8,
    "attn_bwd_fused_sm100_kernel": 10,
}
CUDA_CORE_KERNELS = {"bwd_dq_simt_kernel", "bwd_dkdv_simt_kernel"}


def measured_peaks():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        d = json.loads(f.read_text())
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0]))
                mx.append(float(s[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample(w, seconds_hint: float = 20.0):
    """Time the oracle (as it stands) on a bounded sample of workload `w`: forward + backward of
    one KV group (G query heads) over the first T_s raw tokens.  -> (tflops, cores, description, s)."""
    import numpy as np

    from oracle import oracle
    from paper_2509_15763_b200 import synth

    T_s = min(w.raw_len, 8192 // w.ratio * w.ratio)
    G = w.num_q_heads // w.num_kv_heads
    ws = synth.Workload(w.name + "_sample", 1, T_s, w.ratio, w.window, G, 1, w.head_dim,
                        num_sinks=w.num_sinks, k_scale=w.k_scale, seed=w.seed)
    inp = synth.attention_inputs(ws)
    f = lambda t: t.to(dtype=__import__("torch").float64).numpy()
    q, k, v, do = f(inp["q"][0]), f(inp["k"][0, :, 0]), f(inp["v"][0, :, 0]), f(inp["dout"][0])
    ku = oracle.window_units(w.window, w.ratio)
    scale = w.head_dim ** -0.5
    t0 = time.perf_counter()
    oracle.attn_fwd_slice(ws.num_sinks, T_s, w.ratio, ku, scale, q, k, v)
    if not w.forward_only:
        oracle.attn_bwd_slice(ws.num_sinks, T_s, w.ratio, ku, scale, q, k, v, do)
    dt = time.perf_counter() - t0
    pairs = oracle.count_pairs(ws.num_sinks, T_s, w.ratio, ku)
    flops = (4.0 if w.forward_only else 14.0) * w.head_dim * pairs * G
    desc = (f"oracle {'fwd' if w.forward_only else 'fwd+bwd'} of one KV group ({G} query heads) over the first {T_s} raw tokens "
            f"(N={ws.total_len}) of {w.name}, {pairs} visible pairs per head")
    return flops / dt / 1e12, oracle.num_threads(), desc, dt


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(args.warmup):
        oracle_sample(w)
    t_tot = 0.0
    for _ in range(args.steps):
        tf, cores, desc, dt = oracle_sample(w)
        vals.append(tf)
        t_tot += dt
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "note": "each step is a bounded sample: " + desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


class Path_:
    """Device buffers of one workload and the step that runs the whole path on them."""

    def __init__(self, w, dev):
        import torch

        import paper_2509_15763_b200 as ug
        from paper_2509_15763_b200 import synth

        self.ug, self.torch, self.w, self.dev = ug, torch, w, dev
        self.p = ug.Problem(w.batch, w.raw_len, w.ratio, w.window, w.num_q_heads, w.num_kv_heads, w.head_dim,
                            num_sinks=w.num_sinks)
        p = self.p
        self.N = ug.unigist_total_len(p)
        self.pairs = ug.unigist_visible_pairs(p)
        host = synth.attention_inputs(w, with_grad=not w.forward_only)
        self.host_in = {k: v.pin_memory() for k, v in host.items()}
        self.inter = {k: v.to(dev) for k, v in host.items()}                      # interleaved inputs
        self.sh = {k: torch.empty_like(v) for k, v in self.inter.items()}         # shifted inputs
        self.o_s = torch.empty_like(self.sh["q"])
        self.lse = torch.empty(w.batch, w.num_q_heads, self.N, dtype=torch.float32, device=dev)
        self.dq_s, self.dk_s, self.dv_s = (torch.empty_like(self.sh[n]) for n in ("q", "k", "v"))
        self.out = {"o": torch.empty_like(self.o_s), "dq": torch.empty_like(self.dq_s),
                    "dk": torch.empty_like(self.dk_s), "dv": torch.empty_like(self.dv_s)}
        self.host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in self.out.items()
                         if k == "o" or not w.forward_only}
        self.ws = torch.empty(max(16, ug.unigist_workspace_bytes(p, ug.OP_BWD)), dtype=torch.uint8, device=dev)
        L = ug.unigist_compact_len(p)
        self.nb = -(-(L + 1) // ug.PAGE_TOKENS)
        nblocks = w.batch * self.nb
        self.kc = torch.zeros(nblocks, w.num_kv_heads, ug.PAGE_TOKENS, w.head_dim, dtype=torch.bfloat16, device=dev)
        self.vc = torch.zeros_like(self.kc)
        g = torch.Generator().manual_seed(w.seed)
        self.table = torch.randperm(nblocks, generator=g).to(torch.int32).reshape(w.batch, self.nb).to(dev)
        self.lens = torch.zeros(w.batch, dtype=torch.int32, device=dev)
        self.qd = torch.empty(w.batch, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
        self.od = torch.empty_like(self.qd)
        self.host_od = torch.empty(self.od.shape, dtype=self.od.dtype).pin_memory()
        self.wsd = torch.empty(max(16, ug.unigist_decode_workspace_bytes(w.batch, w.num_q_heads, w.num_kv_heads,
                                                                         w.head_dim, self.nb)),
                               dtype=torch.uint8, device=dev)
        self.flops = (4.0 if w.forward_only else 14.0) * w.head_dim * self.pairs * w.num_q_heads * w.batch
        # the gist shift as tile addressing inside the attention kernels (no shift / unshift launches)
        self.fused_shift = w.head_dim == 128 and 128 % w.ratio == 0
        self.p_il = ug.Problem(w.batch, w.raw_len, w.ratio, w.window, w.num_q_heads, w.num_kv_heads, w.head_dim,
                               num_sinks=w.num_sinks, flags=ug.FLAG_INTERLEAVED)

    def step(self, bufs=None):
        if self.fused_shift:
            return self.step_fused(bufs)
        return self.step_explicit(bufs)

    def step_fused(self, bufs=None):
        """Interleaved tensors in, interleaved results out: the shift is done by the kernels' tile loads."""
        ug, p = self.ug, self.p_il
        x, out, od = bufs or (self.inter, self.out, self.od)
        ug.unigist_attn_fwd(p, x["q"], x["k"], x["v"], out["o"], self.lse)
        if not self.w.forward_only:
            ug.unigist_attn_bwd(p, x["q"], x["k"], x["v"], out["o"], self.lse, x["dout"], out["dq"], out["dk"],
                                out["dv"], self.ws)
        ug.unigist_kv_compact(p, x["k"], x["v"], self.kc, self.vc, self.table, self.lens)
        self.qd.copy_(x["q"][:, -1])  # the last token (the last gist) in either order
        if self.w.head_dim == 128:  # the decode kernel is written for head_dim 128
            ug.unigist_decode(self.qd, self.kc, self.vc, self.table, self.lens, od, None, self.wsd)

    def step_explicit(self, bufs=None):
        ug, p = self.ug, self.p
        inter, out, od = bufs or (self.inter, self.out, self.od)
        for n in inter:
            ug.unigist_gist_shift(p, inter[n], self.sh[n])
        ug.unigist_attn_fwd(p, self.sh["q"], self.sh["k"], self.sh["v"], self.o_s, self.lse)
        outs = [("o", self.o_s)]
        if not self.w.forward_only:
            ug.unigist_attn_bwd(p, self.sh["q"], self.sh["k"], self.sh["v"], self.o_s, self.lse, self.sh["dout"],
                                self.dq_s, self.dk_s, self.dv_s, self.ws)
            outs += [("dq", self.dq_s), ("dk", self.dk_s), ("dv", self.dv_s)]
        for n, t in outs:
            ug.unigist_gist_unshift(p, t, out[n])
        ug.unigist_kv_compact(p, self.sh["k"], self.sh["v"], self.kc, self.vc, self.table, self.lens)
        self.qd.copy_(self.sh["q"][:, -1])
        if self.w.head_dim == 128:  # the decode kernel is written for head_dim 128
            ug.unigist_decode(self.qd, self.kc, self.vc, self.table, self.lens, od, None, self.wsd)

    def e2e_steps(self, steps):
        """`steps` end-to-end steps: every step copies its inputs from pinned host memory, runs the path and
        copies its results back.  The library only enqueues work on the stream it is given, so the copies of
        neighbouring steps run on two side streams under the kernels of the current one (two sets of device
        buffers, ordered by events); when this returns, the current stream waits for the last copy."""
        torch = self.torch
        cur = torch.cuda.current_stream()
        if not hasattr(self, "pipe"):
            sets = [(self.inter, self.out, self.od),
                    ({k: torch.empty_like(v) for k, v in self.inter.items()},
                     {k: torch.empty_like(v) for k, v in self.out.items()}, torch.empty_like(self.od))]
            self.pipe = {"h2d": torch.cuda.Stream(), "d2h": torch.cuda.Stream(), "sets": sets}
        h2d, d2h, sets = self.pipe["h2d"], self.pipe["d2h"], self.pipe["sets"]
        comp_done, d2h_done = [None, None], [None, None]
        start = cur.record_event()
        h2d.wait_event(start)
        d2h.wait_event(start)
        for i in range(steps):
            b = i % 2
            inter, out, od = sets[b]
            with torch.cuda.stream(h2d):
                if comp_done[b] is not None:
                    h2d.wait_event(comp_done[b])  # the step that read this input set is done
                for n in inter:
                    inter[n].copy_(self.host_in[n], non_blocking=True)
                h2d_done = h2d.record_event()
            cur.wait_event(h2d_done)
            if d2h_done[b] is not None:
                cur.wait_event(d2h_done[b])  # this output set has been copied out
            self.step(sets[b])
            comp_done[b] = cur.record_event()
            with torch.cuda.stream(d2h):
                d2h.wait_event(comp_done[b])
                for n in self.host_out:
                    self.host_out[n].copy_(out[n], non_blocking=True)
                self.host_od.copy_(od, non_blocking=True)
                d2h_done[b] = d2h.record_event()
        for e in d2h_done:
            if e is not None:
                cur.wait_event(e)

    def h2d_bytes(self):
        return sum(t.numel() * t.element_size() for t in self.host_in.values())

    def d2h_bytes(self):
        return sum(t.numel() * t.element_size() for t in self.host_out.values()) + \
            self.host_od.numel() * self.host_od.element_size()


def bench_decode(dev, iters=20):
    """Decode over the compressed-cache workload (64 sequences x 9216 cached tokens): GB/s of K+V."""
    import torch

    import paper_2509_15763_b200 as ug
    from paper_2509_15763_b200 import synth

    w = synth.DECODE_WORKLOADS["decode_cache"]
    d = {k: v.to(dev) for k, v in synth.decode_inputs(w).items()}
    ws = torch.empty(ug.unigist_decode_workspace_bytes(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                                       d["block_table"].shape[1]), dtype=torch.uint8, device=dev)
    o = torch.empty_like(d["q"])
    run = lambda: ug.unigist_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o, None, ws)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    ug.unigist_kernel_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    split_ms = [ug.unigist_kernel_timing_get(i)[1] for i in range(ug.unigist_kernel_timing_count())
                if ug.unigist_kernel_timing_get(i)[0] == "decode_split_kernel"]
    ug.unigist_kernel_timing(False)
    nbytes = w.num_seqs * w.seq_len * w.num_kv_heads * w.head_dim * 2 * 2
    return {"workload": w.name, "kv_bytes": nbytes, "us_per_call": 1e3 * ms, "gbs": nbytes / (ms * 1e-3) / 1e9,
            "split_kernel_us": 1e3 * statistics.mean(split_ms), "split_kernel_gbs": nbytes / (statistics.mean(split_ms) * 1e-3) / 1e9,
            "l2_policy": "K+V (2.4 GB) exceed L2, every call streams from HBM"}


def reduce_over_ranks(dist, times_ms, device):
    """Replicas share nothing on the data path; the job's time is that of the slowest rank.
    -> the element-wise MAX of `times_ms` over all ranks (the list itself without a process group)."""
    import torch

    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_value(world, flop_per_replica_step, steps, total_ms):
    """Whole-job effective TFLOP/s: every rank did `steps` steps of its own replica in `total_ms`."""
    return world * flop_per_replica_step * steps / (total_ms * 1e-3) / 1e12


def bench_chunked_prefill(path, chunk_units, iters=3):
    """The prefill workload fed in chunks of `chunk_units` gist units through unigist_prefill_chunk: each
    chunk attends to the compressed paged cache and advances it.  -> dict for the JSON line."""
    import torch

    ug, w, dev = path.ug, path.w, path.dev
    p, r, s, n = path.p, w.ratio, w.num_sinks, w.num_gists
    chunk_units = min(chunk_units, n)
    starts = list(range(0, n, chunk_units))
    chunks = []
    for u0 in starts:  # the chunk's tokens in shifted chunk order [sinks | raw | gists], sliced before timing
        c = min(chunk_units, n - u0)
        ar = torch.arange(u0, u0 + c, device=dev)
        raw = (s + ar[:, None] * (r + 1) + torch.arange(r, device=dev)[None, :]).reshape(-1)
        gist = s + ar * (r + 1) + r
        idx = torch.cat(([torch.arange(s, device=dev)] if u0 == 0 else []) + [raw, gist])
        chunks.append((u0, c, *(path.inter[k][:, idx].contiguous() for k in ("q", "k", "v"))))
    o = [torch.empty_like(c[2]) for c in chunks]
    lse = [torch.empty(w.batch, w.num_q_heads, c[2].shape[1], dtype=torch.float32, device=dev) for c in chunks]
    ws = torch.empty(max(ug.unigist_prefill_workspace_bytes(p, u0, c) for u0, c, *_ in chunks), dtype=torch.uint8,
                     device=dev)

    def run():
        for i, (u0, c, q, k, v) in enumerate(chunks):
            ug.unigist_prefill_chunk(p, u0, c, q, k, v, path.kc, path.vc, path.table, path.lens, o[i], lse[i], ws)

    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    flops = 4.0 * w.head_dim * path.pairs * w.num_q_heads * w.batch
    return {"chunk_units": chunk_units, "chunk_raw_tokens": chunk_units * r, "chunks": len(chunks), "ms": ms,
            "value": flops / (ms * 1e-3) / 1e12, "unit": UNIT,
            "note": "whole prompt through unigist_prefill_chunk: context gather + forward + cache advance per chunk"}


def bench_rope_and_docs(path, iters=3):
    """Two side measurements on the workload's own tensors: the rotary embedding with aligned position ids
    fused with the gist shift (HBM-bound), and the attention step under cross-document masking, with the
    sample cut into documents of T/2, T/4, ... raw tokens.  -> (rope dict, cross_doc dict)."""
    import torch

    ug, w, dev, p = path.ug, path.w, path.dev, path.p

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    x, y = path.inter["q"], path.sh["q"]
    ms = timed(lambda: ug.unigist_rope(p, x, y, 500000.0, ug.ROPE_TO_SHIFTED))
    nbytes = 2 * x.numel() * x.element_size()
    rope = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "bytes": nbytes,
            "note": "unigist_rope on Q, interleaved in, shifted out (read + write once)"}
    if w.batch != 1 or w.forward_only or not path.fused_shift:
        return rope, None
    # documents of T/2, T/4, ... raw tokens; what is left at 1024 tokens or fewer is the last document
    doc_T, left = [], w.raw_len
    while left > 0:
        t = left if left <= 1024 else (left // 2) // w.ratio * w.ratio
        doc_T.append(t)
        left -= t
    p1 = ug.Problem(1, doc_T[0], w.ratio, w.window, w.num_q_heads, w.num_kv_heads, w.head_dim, num_sinks=w.num_sinks,
                    flags=ug.FLAG_INTERLEAVED)
    n_tot = ug.unigist_docs_total_len(p1, doc_T)
    q, k, v, do = (path.inter[n][0, :n_tot] for n in ("q", "k", "v", "dout"))
    if n_tot > path.inter["q"].shape[1]:  # every document carries its own sinks: more rows than the one-document sample
        pad = lambda t: torch.cat([t, t[: n_tot - t.shape[0]]])
        q, k, v, do = pad(q), pad(k), pad(v), pad(do)
    o, dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    lse = torch.empty(w.num_q_heads * n_tot, dtype=torch.float32, device=dev)
    ws = torch.empty(max(16, ug.unigist_docs_workspace_bytes(p1, ug.OP_BWD, doc_T)), dtype=torch.uint8, device=dev)

    def run():
        ug.unigist_attn_fwd_docs(p1, doc_T, q, k, v, o, lse)
        ug.unigist_attn_bwd_docs(p1, doc_T, q, k, v, o, lse, do, dq, dk, dv, ws)

    ms = timed(run)
    pairs = 0
    for t in doc_T:
        pairs += ug.unigist_visible_pairs(ug.Problem(1, t, w.ratio, w.window, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                                     num_sinks=w.num_sinks))
    flops = 14.0 * w.head_dim * pairs * w.num_q_heads
    docs = {"doc_raw_len": doc_T, "ms": ms, "value": flops / (ms * 1e-3) / 1e12, "unit": UNIT,
            "note": "forward + backward of the sample cut into documents (one batched launch set per run of equal "
                    "documents, spread over the library's side streams)"}
    return rope, docs


def run_ours(args, w):
    import torch

    import paper_2509_15763_b200 as ug

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    ug.binding.lib()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_

        dist = dist_
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    path = Path_(w, dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)  # > 126 MB L2
    for _ in range(max(args.warmup, 3)):
        path.step()
    barrier()

    # ---- device-resident timing
    ug.unigist_kernel_timing(True)
    launches0 = ug.unigist_launch_count()
    evs = []
    barrier()
    with ClockSampler(local) as clocks:
        for _ in range(args.steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            path.step()
            e1.record()
            evs.append((e0, e1))
        barrier()
    launches = ug.unigist_launch_count() - launches0
    step_ms = [a.elapsed_time(b) for a, b in evs]
    total_ms = sum(step_ms)
    per_kernel = {}
    for i in range(ug.unigist_kernel_timing_count()):
        name, ms = ug.unigist_kernel_timing_get(i)
        cnt, tot = per_kernel.get(name, (0, 0.0))
        per_kernel[name] = (cnt + 1, tot + ms)
    ug.unigist_kernel_timing(False)

    # ---- the same step with the gist shift as separate launches (context for the fused number)
    explicit_ms = None
    if path.fused_shift and rank == 0:
        for _ in range(2):
            path.step_explicit()
        ev2 = []
        for _ in range(args.steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            path.step_explicit()
            e1.record()
            ev2.append((e0, e1))
        torch.cuda.synchronize()
        explicit_ms = sum(a.elapsed_time(b) for a, b in ev2) / args.steps
    # ---- the same step replayed from a CUDA graph (the tensor maps are kernel arguments, so a captured step
    # needs no host work at all); context for the launch gaps inside the eager number
    graph_ms = None
    if rank == 0 and world == 1:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            path.step()
            with torch.cuda.graph(graph, stream=side):
                path.step()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        ev3 = []
        for _ in range(args.steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            ev3.append((e0, e1))
        torch.cuda.synchronize()
        graph_ms = sum(a.elapsed_time(b) for a, b in ev3) / args.steps
    rope_line, docs_line = bench_rope_and_docs(path) if rank == 0 and world == 1 else (None, None)
    barrier()

    # ---- end to end: host buffers in, host buffers out
    path.e2e_steps(2)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    path.e2e_steps(args.steps)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)

    total_ms, e2e_ms = reduce_over_ranks(dist, [total_ms, e2e_ms], dev)
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    value = job_value(world, path.flops, args.steps, total_ms)
    e2e_value = job_value(world, path.flops, args.steps, e2e_ms)
    attn = {k: v for k, v in per_kernel.items() if k in KERNEL_FLOP_PER_PAIR_D}
    top = max(attn, key=lambda k: attn[k][1])
    cnt, tot = attn[top]
    top_flops = KERNEL_FLOP_PER_PAIR_D[top] * w.head_dim * path.pairs * w.num_q_heads * w.batch
    achieved = top_flops / (tot / cnt * 1e-3) / 1e12
    if top in CUDA_CORE_KERNELS:
        # fp32 FMA pipe: 148 SMs x 128 lanes x 2 FLOP x 1.965 GHz
        bound, peak, peak_src = "alu", 148 * 128 * 2 * 1.965e9 / 1e12, "derived from unit counts and max clock"
    else:
        bound, peak, peak_src = "tensor", peaks["bf16_tflops_sustained"], peaks["source"] + " sustained bf16"
    kernel_share = {k: {"launches": c, "ms": round(m, 4), "share": round(m / sum(x[1] for x in per_kernel.values()), 4)}
                    for k, (c, m) in sorted(per_kernel.items(), key=lambda kv: -kv[1][1])}
    decode = bench_decode(dev)
    cpu_tf, cores, desc, _ = oracle_sample(w)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "raw_len": w.raw_len, "ratio": w.ratio, "window": w.window,
                   "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads, "head_dim": w.head_dim,
                   "total_len": path.N, "visible_pairs_per_head": path.pairs, "flop_per_step": path.flops,
                   "l2": "256 MB buffer written between timed steps", "parallelism": f"replicas x{world}",
                   "gist_shift": ("done by the attention kernels' tile loads and row-mapped stores on interleaved "
                                  "tensors (UNIGIST_FLAG_INTERLEAVED), no shift / unshift launch") if path.fused_shift
                   else "shift_rows_kernel / unshift_rows_kernel launches inside the step"},
        "roofline": {"kernel": top, "bound": bound, "achieved": achieved, "peak": peak, "unit": UNIT,
                     "frac": achieved / peak, "peak_source": peak_src,
                     "traffic": NCU_TRAFFIC_BYTES.get((top, w.name))},
        "pct_of_nominal_bf16_peak": 100.0 * value / world / 2250.0,
        "kernels": kernel_share,
        "decode": dict(decode, frac_of_measured_hbm=decode["split_kernel_gbs"] / peaks["hbm_gbs"],
                       frac_of_nominal_8tbs=decode["split_kernel_gbs"] / 8000.0),
        "cpu_baseline": {"value": cpu_tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": path.h2d_bytes(),
                "d2h_bytes_per_step": path.d2h_bytes(), "ms_per_step": e2e_ms / args.steps,
                "how": "every step copies its inputs from pinned host memory and its results back; the copies of "
                       "neighbouring steps run on two side streams under the kernels (two device buffer sets)"},
        "chunked_prefill": bench_chunked_prefill(path, 1024) if w.forward_only else None,
        "rope": rope_line, "cross_doc": docs_line,
        "graph_step": None if graph_ms is None else {
            "ms_per_step": graph_ms, "value": path.flops / (graph_ms * 1e-3) / 1e12, "unit": UNIT,
            "note": "the timed step captured once in a CUDA graph and replayed"},
        "explicit_shift_step": None if explicit_ms is None else {
            "ms_per_step": explicit_ms, "value": path.flops / (explicit_ms * 1e-3) / 1e12, "unit": UNIT,
            "note": "the same step with 4 shift and 4 unshift launches around shifted-order attention calls"},
        "gpu_launches": launches,
        "clocks": clocks.summary(),
    }
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    from paper_2509_15763_b200 import synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_layer", choices=sorted(synth.WORKLOADS))
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
