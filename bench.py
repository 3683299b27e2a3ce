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

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--only] [--impl reference]

The headline workload is the largest forward + backward one that fits one GPU (`train_batch`: batch 4,
32768 raw tokens, ratio 4, window 2048).  On one GPU the same run also times decode over the compressed
cache and, with fewer steps, the one-layer and the long-prefill workloads; they are reported as extra
keys (`decode`, `workloads`) of the one JSON line.
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

# FLOP per visible pair per query head that each attention kernel performs algorithmically,
# in units of head_dim (a QK^T- or PV-shaped product is 2 * D FLOP per pair).
KERNEL_FLOP_PER_PAIR_D = {
    "attn_fwd_sm100_kernel": 4, "attn_bwd_dq_sm100_kernel": 6, "attn_bwd_dkdv_sm100_kernel": 8,
    "attn_bwd_fused_sm100_kernel": 10,
}
# The source files whose change makes a committed ncu capture of the kernel stale.
KERNEL_SOURCES = {
    "attn_fwd_sm100_kernel": ("attn_fwd_sm100.cu", "sm100_ptx.cuh", "ug_common.cuh"),
    "attn_bwd_fused_sm100_kernel": ("attn_bwd_sm100.cu", "sm100_ptx.cuh", "ug_common.cuh"),
    "attn_bwd_dkdv_sm100_kernel": ("attn_bwd_sm100.cu", "sm100_ptx.cuh", "ug_common.cuh"),
    "attn_bwd_dq_sm100_kernel": ("attn_bwd_sm100.cu", "sm100_ptx.cuh", "ug_common.cuh"),
    "decode_split_kernel": ("decode.cu", "sm100_ptx.cuh", "ug_common.cuh"),
}
HEADLINE = "train_batch"                       # the largest single-GPU forward + backward workload
ALSO = ("llama8b_layer", "long_prefill")       # timed as well (fewer steps), reported under "workloads"


def kernel_source_digest(kernel: str) -> str:
    """Short sha256 over the sources that define `kernel` (what an ncu summary records)."""
    import hashlib

    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        h.update((ROOT / "paper_2509_15763_b200" / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def ncu_traffic(kernel: str, workload: str, batch: int):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of `kernel` on `workload`, from the
    committed ncu summary profiles/<kernel>_<workload>.md.  The summary states the batch size of the captured
    slice (the traffic of these kernels grows in proportion to the batch: every batch index is an independent
    set of thread blocks over its own tensors) and a digest of the kernel's sources.
    -> (bytes scaled to `batch`, note); (None, why) without a capture or once the sources changed."""
    import re

    f = ROOT / "profiles" / f"{kernel}_{workload}.md"
    if not f.exists():
        return None, "no ncu capture committed for this kernel and workload"
    text = f.read_text()
    m_bytes = re.search(r"DRAM traffic per launch = ([0-9.eE+]+) bytes", text)
    m_batch = re.search(r"captured batch: (\d+)", text)
    m_src = re.search(r"kernel sources sha256: ([0-9a-f]+)", text)
    if not (m_bytes and m_batch and m_src):
        return None, f"{f.name} lacks the traffic, batch or source-digest line"
    if kernel not in KERNEL_SOURCES or m_src.group(1) != kernel_source_digest(kernel):
        return None, f"the kernel's sources changed since {f.name} was captured"
    cap_b = int(m_batch.group(1))
    return float(m_bytes.group(1)) * batch / cap_b, f"{f.name}: captured at batch {cap_b}, scaled x{batch / cap_b:g}"


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


def oracle_decode_sample(num_seqs: int = 4):
    """Time the oracle's decode (as it stands) on `num_seqs` of the 64 sequences of the decode workload, all
    heads.  -> (GB/s of K+V, cores, description)."""
    import torch

    from oracle import oracle
    from paper_2509_15763_b200 import synth

    w = synth.DECODE_WORKLOADS["decode_cache"]
    ws = synth.DecodeWorkload(w.name + "_sample", num_seqs, w.num_gists, w.window_raw, w.num_q_heads, w.num_kv_heads,
                              w.head_dim, seed=w.seed)
    d = synth.decode_inputs(ws)
    f = lambda t: t.to(dtype=torch.float64).numpy()
    view = lambda c, i: c[d["block_table"][i].long()].permute(0, 2, 1, 3).reshape(-1, c.shape[1], c.shape[3])[: ws.seq_len]
    k_list = [f(view(d["k_cache"], i)) for i in range(num_seqs)]
    v_list = [f(view(d["v_cache"], i)) for i in range(num_seqs)]
    q = f(d["q"])
    t0 = time.perf_counter()
    oracle.decode(w.head_dim ** -0.5, q, k_list, v_list)
    dt = time.perf_counter() - t0
    nbytes = num_seqs * ws.seq_len * w.num_kv_heads * w.head_dim * 2 * 2  # the bf16 K and V the query attends to
    desc = (f"oracle decode of {num_seqs} of the {w.num_seqs} sequences ({ws.seq_len} cache entries each, all "
            f"{w.num_q_heads} query heads); the whole workload is {w.num_seqs // num_seqs}x this")
    return nbytes / dt / 1e9, oracle.num_threads(), desc


def pick_tensor_peak(peaks, clocks, timed_seconds):
    """The measured bf16 rate the timed kernel is held against: the burst figure for a short region at full
    clock, the sustained one for a region of a second or more or one the power cap held below full clock."""
    sm, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    capped = "sw_power_cap" in clocks.get("reasons", []) or (sm is not None and mx and sm < 0.9 * mx)
    if capped or timed_seconds >= 1.0:
        why = ("power cap active / SM clock below 0.9 of max during the timed region" if capped else
               "timed region of a second or more")
        return peaks["bf16_tflops_sustained"], f"{peaks['source']} sustained bf16 ({why})"
    return peaks["bf16_tflops"], f"{peaks['source']} burst bf16 (timed region {timed_seconds:.2f} s at full clock)"


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

    def __init__(self, w, dev, host_buffers=True):
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
        self.host_in = {k: v.pin_memory() for k, v in host.items()} if host_buffers else {}
        self.inter = {k: v.to(dev) for k, v in host.items()}                      # interleaved inputs
        self.sh = {k: torch.empty_like(v) for k, v in self.inter.items()}         # shifted inputs
        self.o_s = torch.empty_like(self.sh["q"])
        self.lse = torch.empty(w.batch, w.num_q_heads, self.N, dtype=torch.float32, device=dev)
        self.dq_s, self.dk_s, self.dv_s = (torch.empty_like(self.sh[n]) for n in ("q", "k", "v"))
        self.out = {"o": torch.empty_like(self.o_s), "dq": torch.empty_like(self.dq_s),
                    "dk": torch.empty_like(self.dk_s), "dv": torch.empty_like(self.dv_s)}
        self.host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in self.out.items()
                         if host_buffers and (k == "o" or not w.forward_only)}
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
    """Decode over the compressed-cache workload (64 sequences x 9216 cached tokens): GB/s of K+V.
    The calls alternate between two independent copies of the cache (2.4 GB each), so nothing a call reads
    can still sit in the 126 MB L2 from the call before."""
    import torch

    import paper_2509_15763_b200 as ug
    from paper_2509_15763_b200 import synth

    w = synth.DECODE_WORKLOADS["decode_cache"]
    d = {k: v.to(dev) for k, v in synth.decode_inputs(w).items()}
    sets = [(d["k_cache"], d["v_cache"]), (d["k_cache"].clone(), d["v_cache"].clone())]
    ws = torch.empty(ug.unigist_decode_workspace_bytes(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                                       d["block_table"].shape[1]), dtype=torch.uint8, device=dev)
    o = torch.empty_like(d["q"])
    run = lambda i: ug.unigist_decode(d["q"], sets[i & 1][0], sets[i & 1][1], d["block_table"], d["seq_lens"], o, None, ws)
    for i in range(4):
        run(i)
    torch.cuda.synchronize()
    ug.unigist_kernel_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        run(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    split_ms = [ug.unigist_kernel_timing_get(i)[1] for i in range(ug.unigist_kernel_timing_count())
                if ug.unigist_kernel_timing_get(i)[0] == "decode_split_kernel"]
    ug.unigist_kernel_timing(False)
    nbytes = w.num_seqs * w.seq_len * w.num_kv_heads * w.head_dim * 2 * 2
    traffic, traffic_note = ncu_traffic("decode_split_kernel", w.name, 1)
    return {"workload": w.name, "kv_bytes": nbytes, "us_per_call": 1e3 * ms, "gbs": nbytes / (ms * 1e-3) / 1e9,
            "split_kernel_us": 1e3 * statistics.mean(split_ms), "split_kernel_gbs": nbytes / (statistics.mean(split_ms) * 1e-3) / 1e9,
            "traffic": traffic, "traffic_source": traffic_note,
            "l2_policy": "consecutive calls read two different copies of the cache (2.4 GB each, L2 is 126 MB)"}


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

    def timed(fn, iters=iters):
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
    # one launch of tens of microseconds: enough of them in a row that the host's launch cost hides under the kernels
    ms = timed(lambda: ug.unigist_rope(p, x, y, 500000.0, ug.ROPE_TO_SHIFTED), iters=20)
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
            "note": "forward + backward of the sample cut into documents of different lengths: one launch of each "
                    "kernel for all of them (every block finds its document from its block index)"}
    return rope, docs


def timed_steps(torch, ug, path, steps, flush, barrier, local):
    """`steps` device-resident steps of `path`, L2 flushed before each, CUDA events around each step and (inside
    the library) around each kernel.  -> (step times ms, {kernel: (launches, total ms)}, launches, clock summary)."""
    ug.unigist_kernel_timing(True)
    launches0 = ug.unigist_launch_count()
    evs = []
    barrier()
    with ClockSampler(local) as clocks:
        for _ in range(steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            path.step()
            e1.record()
            evs.append((e0, e1))
        barrier()
    launches = ug.unigist_launch_count() - launches0
    per_kernel = {}
    for i in range(ug.unigist_kernel_timing_count()):
        name, ms = ug.unigist_kernel_timing_get(i)
        cnt, tot = per_kernel.get(name, (0, 0.0))
        per_kernel[name] = (cnt + 1, tot + ms)
    ug.unigist_kernel_timing(False)
    return [a.elapsed_time(b) for a, b in evs], per_kernel, launches, clocks.summary()


def roofline_of(w, path, per_kernel, clocks, timed_seconds, peaks):
    """The roofline object of the attention kernel with the largest share of the step."""
    attn = {k: v for k, v in per_kernel.items() if k in KERNEL_FLOP_PER_PAIR_D}
    top = max(attn, key=lambda k: attn[k][1])
    cnt, tot = attn[top]
    top_flops = KERNEL_FLOP_PER_PAIR_D[top] * w.head_dim * path.pairs * w.num_q_heads * w.batch
    achieved = top_flops / (tot / cnt * 1e-3) / 1e12
    peak, peak_src = pick_tensor_peak(peaks, clocks, timed_seconds)
    traffic, traffic_note = ncu_traffic(top, w.name, w.batch)
    sm, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    return {"kernel": top, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": UNIT, "frac": achieved / peak,
            "peak_source": peak_src, "kernel_ms": tot / cnt, "algorithmic_flop_per_launch": top_flops,
            "frac_of_burst": achieved / peaks["bf16_tflops"], "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
            "frac_of_nominal_2250": achieved / 2250.0,
            # the same rate carried to the maximum SM clock: how much of the gap to the peak is the clock
            "achieved_at_max_clock": achieved * mx / sm if sm and mx else None,
            "traffic": traffic, "traffic_source": traffic_note}


def kernel_shares(per_kernel):
    total = sum(x[1] for x in per_kernel.values())
    return {k: {"launches": c, "ms": round(m, 4), "share": round(m / total, 4)}
            for k, (c, m) in sorted(per_kernel.items(), key=lambda kv: -kv[1][1])}


def config_of(w, path, world):
    return {"workload": w.name, "batch": w.batch, "raw_len": w.raw_len, "ratio": w.ratio, "window": w.window,
            "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads, "head_dim": w.head_dim,
            "total_len": path.N, "visible_pairs_per_head": path.pairs, "flop_per_step": path.flops,
            "l2": "256 MB buffer written between timed steps", "parallelism": f"replicas x{world}",
            "gist_shift": ("done by the attention kernels' tile loads and row-mapped stores on interleaved "
                           "tensors (UNIGIST_FLAG_INTERLEAVED), no shift / unshift launch") if path.fused_shift
            else "shift_rows_kernel / unshift_rows_kernel launches inside the step"}


def side_workload(torch, ug, name, dev, steps, flush, barrier, local, peaks):
    """One of the other workloads, device-resident timing only (rank 0, one GPU): a dict for the JSON line."""
    from paper_2509_15763_b200 import synth

    w = synth.WORKLOADS[name]
    path = Path_(w, dev, host_buffers=False)
    for _ in range(3):
        path.step()
    step_ms, per_kernel, _, clocks = timed_steps(torch, ug, path, steps, flush, barrier, local)
    ms = sum(step_ms) / steps
    out = {"config": config_of(w, path, 1), "steps": steps, "ms_per_step": ms,
           "value": path.flops / (ms * 1e-3) / 1e12, "unit": UNIT,
           "what": "forward only (prefill)" if w.forward_only else "forward + backward",
           "pct_of_nominal_bf16_peak": 100.0 * path.flops / (ms * 1e-3) / 1e12 / 2250.0,
           "roofline": roofline_of(w, path, per_kernel, clocks, sum(step_ms) * 1e-3, peaks),
           "kernels": kernel_shares(per_kernel), "clocks": clocks}
    if w.forward_only:
        out["chunked_prefill"] = bench_chunked_prefill(path, 1024)
    else:
        out["rope"], out["cross_doc"] = bench_rope_and_docs(path)
    del path
    torch.cuda.empty_cache()
    return out


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

    warmup = max(args.warmup, 3)
    path = Path_(w, dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)  # > 126 MB L2
    for _ in range(warmup):
        path.step()
    barrier()

    # ---- device-resident timing
    step_ms, per_kernel, launches, clocks = timed_steps(torch, ug, path, args.steps, flush, barrier, local)
    total_ms = sum(step_ms)
    median_ms = statistics.median(step_ms)  # this rank's; the line's ms_per_step is the mean of the slowest rank

    # ---- the same step with the gist shift as separate launches (context for the fused number)
    explicit_ms = None
    if path.fused_shift and rank == 0:
        for _ in range(2):
            path.step_explicit()
        ev2 = []
        for _ in range(min(args.steps, 5)):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            path.step_explicit()
            e1.record()
            ev2.append((e0, e1))
        torch.cuda.synchronize()
        explicit_ms = sum(a.elapsed_time(b) for a, b in ev2) / len(ev2)
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
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": total_ms / args.steps, "ms_per_step_median": median_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(w, path, world),
        "roofline": roofline_of(w, path, per_kernel, clocks, total_ms * 1e-3, peaks),
        "pct_of_nominal_bf16_peak": 100.0 * value / world / 2250.0,
        "kernels": kernel_shares(per_kernel),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": path.h2d_bytes(),
                "d2h_bytes_per_step": path.d2h_bytes(), "ms_per_step": e2e_ms / args.steps,
                "how": "every step copies its inputs from pinned host memory and its results back; the copies of "
                       "neighbouring steps run on two side streams under the kernels (two device buffer sets)"},
        "explicit_shift_step": None if explicit_ms is None else {
            "ms_per_step": explicit_ms, "value": path.flops / (explicit_ms * 1e-3) / 1e12, "unit": UNIT,
            "shift_unshift_ms": explicit_ms - total_ms / args.steps,
            "note": "the same step with 4 shift and 4 unshift launches around shifted-order attention calls; "
                    "shift_unshift_ms is what those 8 launches add"},
        "gpu_launches": launches,
        "clocks": clocks,
        # clock-normalised step: milliseconds x median SM MHz = thousands of SM cycles per step
        "kcycles_per_step": None if not clocks.get("sm_mhz") else total_ms / args.steps * clocks["sm_mhz"],
    }
    if w.forward_only:
        line["chunked_prefill"] = bench_chunked_prefill(path, 1024)
    elif world == 1:
        line["rope"], line["cross_doc"] = bench_rope_and_docs(path)
    del path
    torch.cuda.empty_cache()
    # ---- the metric's other parts (one GPU): decode over the compressed cache, and the other workloads
    decode = bench_decode(dev)
    line["decode"] = dict(decode, frac_of_measured_hbm=decode["split_kernel_gbs"] / peaks["hbm_gbs"],
                          frac_of_nominal_8tbs=decode["split_kernel_gbs"] / 8000.0)
    torch.cuda.empty_cache()
    line["workloads"] = {}
    if world == 1 and not args.only:
        for name in ALSO:
            if name != w.name:
                line["workloads"][name] = side_workload(torch, ug, name, dev, min(args.steps, 5), flush, barrier, local, peaks)
    cpu_tf, cores, desc, _ = oracle_sample(w)
    line["cpu_baseline"] = {"value": cpu_tf, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}
    dec_gbs, dec_cores, dec_desc = oracle_decode_sample()
    line["decode"]["cpu_baseline"] = {"value": dec_gbs, "unit": "GB/s", "cores": dec_cores, "kind": "oracle",
                                      "sample": dec_desc}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    from paper_2509_15763_b200 import synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--only", action="store_true", help="time the named workload alone, not the other workloads beside it")
    ap.add_argument("--batch", type=int, default=0,
                    help="run a slice of the workload with this batch size (what the ncu captures under profiles/ use)")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.batch > 0:
        w = w.scaled(batch=args.batch)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
