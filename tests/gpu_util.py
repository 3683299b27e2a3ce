"""Helpers for the GPU parity tests: run the library on seeded inputs, hand results back in the
interleaved order the oracle works in."""
from __future__ import annotations

import numpy as np
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth

# Tolerances of the bf16 path against the fp64 oracle: O max-abs and mean-abs, LSE, gradients.
TOL_O_MAX, TOL_O_MEAN, TOL_LSE, TOL_GRAD = 2e-2, 2e-3, 1e-3, 5e-2


def problem_of(w: synth.Workload, flags: int = 0, softmax_scale: float = 0.0) -> ug.Problem:
    return ug.Problem(w.batch, w.raw_len, w.ratio, w.window, w.num_q_heads, w.num_kv_heads,
                      w.head_dim, num_sinks=w.num_sinks, softmax_scale=softmax_scale, flags=flags)


def run_attention_interleaved(w: synth.Workload, backward: bool = True, inputs=None, dout_fp32: bool = False,
                              softmax_scale: float = 0.0):
    """The same results as run_attention, computed with UNIGIST_FLAG_INTERLEAVED: the library reads the
    interleaved tensors as they are and writes o, dq, dk, dv interleaved; no shift / unshift call."""
    dev = torch.device("cuda:0")
    inp = inputs or synth.attention_inputs(w, with_grad=backward, dout_fp32=dout_fp32)
    p = problem_of(w, ug.FLAG_INTERLEAVED | (ug.FLAG_DOUT_FP32 if (backward and dout_fp32) else 0), softmax_scale)
    N = ug.unigist_total_len(p)
    d = {k: v.to(dev) for k, v in inp.items()}
    o = torch.full_like(d["q"], float("nan"))
    lse_s = torch.full((w.batch, w.num_q_heads, N), float("nan"), device=dev, dtype=torch.float32)
    ug.unigist_attn_fwd(p, d["q"], d["k"], d["v"], o, lse_s)
    up = torch.empty(N, dtype=torch.int32, device=dev)
    ug.unigist_layout(p, None, up, None)
    out = {"inputs": inp, "o": o, "lse": lse_s[:, :, up.long()], "lse_shifted": lse_s}
    if backward:
        ws = torch.empty(max(ug.unigist_workspace_bytes(p, ug.OP_BWD), 16), dtype=torch.uint8, device=dev)
        out["dq"] = torch.full_like(d["q"], float("nan"))
        out["dk"] = torch.full_like(d["k"], float("nan"))
        out["dv"] = torch.full_like(d["v"], float("nan"))
        ug.unigist_attn_bwd(p, d["q"], d["k"], d["v"], o, lse_s, d["dout"], out["dq"], out["dk"], out["dv"], ws)
    ug.unigist_device_status()
    return out


def run_attention(w: synth.Workload, backward: bool = True, dout_fp32: bool = False, inputs=None,
                  softmax_scale: float = 0.0, flags: int = 0):
    """-> dict of CUDA tensors in INTERLEAVED order: o, lse [B,Hq,N], dq, dk, dv, plus inputs."""
    dev = torch.device("cuda:0")
    inp = inputs or synth.attention_inputs(w, with_grad=backward, dout_fp32=dout_fp32)
    p = problem_of(w, flags | (ug.FLAG_DOUT_FP32 if (backward and dout_fp32) else 0), softmax_scale)
    N = ug.unigist_total_len(p)
    d = {k: v.to(dev) for k, v in inp.items()}
    sh = {}
    for name in ("q", "k", "v") + (("dout",) if backward else ()):
        sh[name] = torch.empty_like(d[name])
        ug.unigist_gist_shift(p, d[name], sh[name])
    o_s = torch.full_like(sh["q"], float("nan"))
    lse_s = torch.full((w.batch, w.num_q_heads, N), float("nan"), device=dev, dtype=torch.float32)
    ug.unigist_attn_fwd(p, sh["q"], sh["k"], sh["v"], o_s, lse_s)
    out = {"inputs": inp, "shifted": sh, "o_shifted": o_s, "lse_shifted": lse_s}
    o = torch.empty_like(o_s)
    ug.unigist_gist_unshift(p, o_s, o)
    # lse is [B,Hq,N]: unshift through a [B,N,Hq,1]-shaped view would break the 16-byte row rule,
    # so permute it on the host side of the test with the library's own index array.
    up = torch.empty(N, dtype=torch.int32, device=dev)
    ug.unigist_layout(p, None, up, None)
    out["o"] = o
    out["lse"] = lse_s[:, :, up.long()]
    if backward:
        ws = torch.empty(max(ug.unigist_workspace_bytes(p, ug.OP_BWD), 16), dtype=torch.uint8, device=dev)
        dq_s = torch.full_like(sh["q"], float("nan"))
        dk_s = torch.full_like(sh["k"], float("nan"))
        dv_s = torch.full_like(sh["v"], float("nan"))
        ug.unigist_attn_bwd(p, sh["q"], sh["k"], sh["v"], o_s, lse_s, sh["dout"], dq_s, dk_s, dv_s, ws)
        for name, t in (("dq", dq_s), ("dk", dk_s), ("dv", dv_s)):
            out[name] = torch.empty_like(t)
            ug.unigist_gist_unshift(p, t, out[name])
            out[name + "_shifted"] = t
    ug.unigist_device_status()  # synchronises; raises if a bounded device wait gave up
    return out


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def check_close(name, got: np.ndarray, want: np.ndarray, tol_max: float, tol_mean: float | None = None):
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    err = np.abs(got - want)
    assert err.max() <= tol_max, f"{name}: max-abs {err.max():.4g} > {tol_max}"
    if tol_mean is not None:
        assert err.mean() <= tol_mean, f"{name}: mean-abs {err.mean():.4g} > {tol_mean}"


def edge_positions(s, T, r, k):
    """SHIFTED positions of the rows / keys the 128-row tile kernels branch on: the first and last row of the first
    tile of each segment, of the tile in which the window starts to clip (raw row (k + 1) r, gist k + 1), of a middle
    tile and of the last tile, the rows on either side of the clipping point, a row inside a tile, and the sinks' ends."""
    n = T // r
    pos = set()

    def tiles(base, length, first_clipped):
        last_tile = (length - 1) // 128
        for j in {0, min(first_clipped // 128, last_tile), last_tile // 2, last_tile}:
            pos.update(base + x for x in (128 * j, min(128 * j + 127, length - 1)))
        for x in (first_clipped - 1, first_clipped, length // 3 + 5):
            if 0 <= x < length:
                pos.add(base + x)

    tiles(s, T, (k + 1) * r)      # raw rows: unit k + 1 is the first whose window no longer reaches unit 0
    tiles(s + T, n, k + 1)        # gist rows
    if s:
        pos.update((0, s - 1))
    return np.array(sorted(pos), dtype=np.int64)
