"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth
from oracle import oracle

from gpu_util import (TOL_GRAD, TOL_LSE, TOL_O_MAX, TOL_O_MEAN, check_close, edge_positions, f64, problem_of,
                      run_attention, run_attention_interleaved)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


# ------------------------------------------------------------------ layout and shift (bit-exact)
@pytest.mark.parametrize("s,T,r", [(0, 448, 7), (5, 64, 4), (128, 4096, 8), (0, 16, 16), (3, 9, 1),
                                   (0, 131072, 16)])
def test_layout_device_matches_oracle(s, T, r):
    p = ug.Problem(1, T, r, 64, 1, 1, 64, num_sinks=s)
    N = ug.unigist_total_len(p)
    sp, up, pos = (torch.full((N,), -1, dtype=torch.int32, device=DEV) for _ in range(3))
    ug.unigist_layout(p, sp, up, pos)
    a, b, c = oracle.layout(s, T, r)
    assert np.array_equal(sp.cpu().numpy(), a)
    assert np.array_equal(up.cpu().numpy(), b)
    assert np.array_equal(pos.cpu().numpy(), c)
    hs, hu, hp = (torch.empty(N, dtype=torch.int32) for _ in range(3))
    ug.unigist_layout(p, hs, hu, hp)  # host variant
    assert np.array_equal(hs.numpy(), a) and np.array_equal(hu.numpy(), b) and np.array_equal(hp.numpy(), c)


@pytest.mark.parametrize("B,s,T,r,H,D,dtype", [(2, 0, 448, 7, 1, 64, torch.bfloat16),
                                               (1, 5, 640, 4, 8, 128, torch.bfloat16),
                                               (3, 2, 90, 9, 3, 64, torch.float32),
                                               (1, 0, 16384, 8, 32, 128, torch.bfloat16)])
def test_shift_unshift_bit_exact(B, s, T, r, H, D, dtype):
    p = ug.Problem(B, T, r, 64, H, H, D, num_sinks=s)
    N = ug.unigist_total_len(p)
    g = torch.Generator().manual_seed(7)
    x = torch.randn(B, N, H, D, generator=g).to(dtype)
    sp, up, _ = oracle.layout(s, T, r)
    xd = x.to(DEV)
    y = torch.full_like(xd, float("nan"))
    ug.unigist_gist_shift(p, xd, y)
    assert torch.equal(y.cpu(), x[:, torch.from_numpy(sp).long()])
    z = torch.full_like(xd, float("nan"))
    ug.unigist_gist_unshift(p, y, z)
    assert torch.equal(z.cpu(), x)


# ------------------------------------------------------------------ forward + backward, whole problem
SMALL = [
    synth.WORKLOADS["tiny"],
    synth.Workload("sinks_ragged", 2, 330, 5, 48, 4, 2, 64, num_sinks=7, seed=101),
    synth.Workload("gqa_128", 1, 1536, 4, 256, 8, 2, 128, seed=102),
    synth.Workload("full_window", 1, 384, 8, 4096, 2, 2, 128, seed=103),
    synth.Workload("ratio_one", 1, 200, 1, 16, 2, 1, 64, seed=104),
    synth.Workload("no_window", 1, 512, 16, 0, 2, 1, 128, num_sinks=3, seed=105),
    synth.Workload("one_unit", 1, 12, 12, 12, 1, 1, 64, seed=106),
    synth.Workload("odd_tiles", 1, 1000, 8, 200, 4, 4, 128, num_sinks=1, k_scale=0.5, seed=107),
    # tensor-core paths (no sinks) with ragged last tiles in both segments, batch > 1, odd and even group sizes
    synth.Workload("ragged_128", 2, 1000, 8, 200, 4, 2, 128, k_scale=0.5, seed=108),
    synth.Workload("ragged_mha_128", 1, 1096, 4, 300, 3, 3, 128, seed=109),
    synth.Workload("ragged_group3_128", 1, 777, 7, 77, 6, 2, 128, seed=110),
    synth.Workload("ragged_64", 2, 1000, 8, 200, 4, 2, 64, seed=111),
    synth.Workload("tiny_window_128", 1, 2048, 16, 16, 2, 1, 128, seed=112),
    # sink prefixes on the tensor-core paths: one full sink tile (the paper's default 128), several ragged ones
    synth.Workload("sinks_128", 1, 1024, 8, 128, 4, 2, 128, num_sinks=128, seed=113),
    synth.Workload("sinks_300", 2, 640, 4, 64, 2, 2, 128, num_sinks=300, seed=114),
    synth.Workload("sinks_64_d64", 1, 512, 8, 64, 2, 1, 64, num_sinks=64, seed=115),
    # gist units longer than a tile: plain causal attention as a single unit, and two-tile units with a one-unit window
    synth.Workload("single_unit_causal", 1, 640, 640, 640, 2, 2, 128, seed=116),
    synth.Workload("long_units", 2, 1024, 256, 256, 4, 2, 128, num_sinks=5, seed=117),
    # 32 query heads on one KV head: the rows one KV head's blocks sweep (133 MB) exceed the L2, so the backward cuts
    # the walks of the sink and gist key tiles (2 + 4 tiles, 34 query tiles) into two chunks and adds partial dK / dV
    # (dO scaled down: 32 heads add into one KV head, and the gradient tolerance is absolute)
    synth.Workload("cut_walks_sinks", 2, 3584, 8, 256, 32, 1, 128, num_sinks=130, dout_scale=0.25, seed=118),
]


# Logits with a standard deviation of 4 to 6 instead of 1: the row maximum moves by many powers of two from key tile to
# key tile (every rescale branch of the online softmax is taken), the probabilities are close to one-hot and most
# exponentials underflow.  dO is scaled down because K is scaled up and the gradient tolerance is absolute; V is halved
# because O is then close to single rows of V, and the bf16 rounding of a |v| >= 4 alone is most of the O tolerance.
PEAKY = [
    synth.Workload("peaky_128", 2, 1536, 4, 256, 8, 2, 128, num_sinks=5, k_scale=6.0, v_scale=0.5, dout_scale=0.125, seed=120),
    synth.Workload("peaky_ragged_128", 1, 1000, 8, 200, 4, 4, 128, k_scale=4.0, v_scale=0.5, dout_scale=0.25, seed=121),
    synth.Workload("peaky_64", 1, 1000, 8, 200, 4, 2, 64, num_sinks=3, k_scale=5.0, v_scale=0.5, dout_scale=0.125, seed=122),
]


@pytest.mark.parametrize("w", SMALL + PEAKY, ids=lambda w: w.name)
def test_attention_matches_oracle(w):
    fp32_dout = w.name == "tiny"  # the tiny workload states an fp32 dO
    out = run_attention(w, backward=True, dout_fp32=fp32_dout)
    inp = out["inputs"]
    k = oracle.window_units(w.window, w.ratio)
    scale = w.head_dim ** -0.5
    q, kk, v, do = (f64(inp[n]) for n in ("q", "k", "v", "dout"))
    o, lse = oracle.attn_fwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v)
    check_close("O", f64(out["o"]), o, TOL_O_MAX, TOL_O_MEAN)
    check_close("LSE", f64(out["lse"]), lse, TOL_LSE)
    dq, dk, dv = oracle.attn_bwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v, do)
    check_close("dQ", f64(out["dq"]), dq, TOL_GRAD)
    check_close("dK", f64(out["dk"]), dk, TOL_GRAD)
    check_close("dV", f64(out["dv"]), dv, TOL_GRAD)


INTERLEAVED = [w for w in SMALL + PEAKY if w.head_dim == 128 and 128 % w.ratio == 0]


@pytest.mark.parametrize("w", INTERLEAVED, ids=lambda w: w.name)
def test_interleaved_tensors_match_oracle(w):
    """UNIGIST_FLAG_INTERLEAVED: the shift happens inside the tile addressing, no shift / unshift pass."""
    out = run_attention_interleaved(w)
    inp = out["inputs"]
    k = oracle.window_units(w.window, w.ratio)
    scale = w.head_dim ** -0.5
    q, kk, v, do = (f64(inp[n]) for n in ("q", "k", "v", "dout"))
    o, lse = oracle.attn_fwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v)
    check_close("O", f64(out["o"]), o, TOL_O_MAX, TOL_O_MEAN)
    check_close("LSE", f64(out["lse"]), lse, TOL_LSE)
    dq, dk, dv = oracle.attn_bwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v, do)
    check_close("dQ", f64(out["dq"]), dq, TOL_GRAD)
    check_close("dK", f64(out["dk"]), dk, TOL_GRAD)
    check_close("dV", f64(out["dv"]), dv, TOL_GRAD)
    # and bit for bit what the explicit shift -> attention -> unshift route gives (dQ: up to its summation order)
    ref = run_attention(w, inputs=inp)
    for n in ("o", "lse", "dk", "dv"):
        assert torch.equal(out[n], ref[n]), n
    assert (out["dq"].float() - ref["dq"].float()).abs().max().item() <= 2.0 ** -7


@pytest.mark.parametrize("name", ["gqa_128", "sinks_300", "ragged_group3_128", "ragged_64"])
def test_fp32_dout_is_rounded_to_bf16_on_load(name):
    """UNIGIST_FLAG_DOUT_FP32: the gradients are those of the same dO rounded to bf16 (round to nearest even), bit
    for bit, on both backward paths and in both tensor orders; and they match the oracle on the rounded dO."""
    w = next(x for x in SMALL if x.name == name)
    inp32 = synth.attention_inputs(w, dout_fp32=True)
    assert inp32["dout"].dtype == torch.float32
    inp16 = dict(inp32, dout=inp32["dout"].to(torch.bfloat16))
    routes = [run_attention] + ([run_attention_interleaved] if w in INTERLEAVED else [])
    for run in routes:
        a = run(w, inputs=inp32, dout_fp32=True)
        b = run(w, inputs=inp16)
        for n in ("dk", "dv"):
            assert torch.equal(a[n], b[n]), (run.__name__, n)
        assert (a["dq"].float() - b["dq"].float()).abs().max().item() <= 2.0 ** -7
    k = oracle.window_units(w.window, w.ratio)
    dq, dk, dv = oracle.attn_bwd(w.num_sinks, w.raw_len, w.ratio, k, w.head_dim ** -0.5,
                                 *(f64(inp16[n]) for n in ("q", "k", "v", "dout")))
    check_close("dQ", f64(a["dq"]), dq, TOL_GRAD)
    check_close("dK", f64(a["dk"]), dk, TOL_GRAD)
    check_close("dV", f64(a["dv"]), dv, TOL_GRAD)


@pytest.mark.parametrize("name", ["gqa_128", "sinks_300", "ragged_group3_128", "long_units", "cut_walks_sinks", "peaky_128"])
def test_deterministic_dq_flag(name):
    """UNIGIST_FLAG_DETERMINISTIC_DQ (head_dim 128): the gradients match the oracle, and two runs give the same bits
    in dq as well; dk, dv and the forward are what the default backward gives."""
    w = next(x for x in SMALL + PEAKY if x.name == name)
    assert w.head_dim == 128
    a = run_attention(w, flags=ug.FLAG_DETERMINISTIC_DQ)
    b = run_attention(w, inputs=a["inputs"], flags=ug.FLAG_DETERMINISTIC_DQ)
    for n in ("o", "lse", "dq", "dk", "dv"):
        assert torch.equal(a[n], b[n]), n
    inp = a["inputs"]
    k = oracle.window_units(w.window, w.ratio)
    dq, dk, dv = oracle.attn_bwd(w.num_sinks, w.raw_len, w.ratio, k, w.head_dim ** -0.5,
                                 *(f64(inp[n]) for n in ("q", "k", "v", "dout")))
    check_close("dQ", f64(a["dq"]), dq, TOL_GRAD)
    check_close("dK", f64(a["dk"]), dk, TOL_GRAD)
    check_close("dV", f64(a["dv"]), dv, TOL_GRAD)
    p = problem_of(w, ug.FLAG_DETERMINISTIC_DQ | ug.FLAG_INTERLEAVED)
    x = torch.zeros(w.batch, w.total_len, w.num_q_heads, 128, dtype=torch.bfloat16, device=DEV)
    kv = torch.zeros(w.batch, w.total_len, w.num_kv_heads, 128, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(w.batch, w.num_q_heads, w.total_len, device=DEV)
    ws = torch.empty(max(16, ug.unigist_workspace_bytes(p, ug.OP_BWD)), dtype=torch.uint8, device=DEV)
    with pytest.raises(ug.UnigistError):  # the flag's kernels take shifted tensors
        ug.unigist_attn_bwd(p, x, kv, kv, x, lse, x, torch.empty_like(x), torch.empty_like(kv), torch.empty_like(kv), ws)


def test_interleaved_flag_is_refused_where_the_tiles_do_not_line_up():
    for w in (SMALL[0], synth.Workload("r7", 1, 448, 7, 64, 2, 1, 128, seed=1)):
        p = problem_of(w, ug.FLAG_INTERLEAVED)
        N = ug.unigist_total_len(p)
        q = torch.zeros(w.batch, N, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=DEV)
        kv = torch.zeros(w.batch, N, w.num_kv_heads, w.head_dim, dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros(w.batch, w.num_q_heads, N, dtype=torch.float32, device=DEV)
        with pytest.raises(ug.UnigistError):
            ug.unigist_attn_fwd(p, q, kv, kv, torch.empty_like(q), lse)


def test_forward_is_deterministic():
    w = SMALL[2]
    a = run_attention(w, backward=True)
    b = run_attention(w, backward=True)
    for n in ("o", "lse", "dk", "dv"):
        assert torch.equal(a[n], b[n]), n
    # dQ of a query tile is summed over its key tiles with floating-point atomics in the fused
    # backward (head_dim 128): the order, hence the last bit, may differ between runs
    assert (a["dq"].float() - b["dq"].float()).abs().max().item() <= 2.0 ** -7


# ------------------------------------------------------------------ full-size workloads, sampled outputs
@pytest.mark.parametrize("name,backward,route", [("llama8b_layer", True, "explicit"), ("train_batch", True, "explicit"),
                                                 ("long_prefill", False, "explicit"),
                                                 # the route bench.py times: interleaved tensors, no shift launches
                                                 ("llama8b_layer", True, "interleaved"),
                                                 ("train_batch", True, "interleaved"),
                                                 ("long_prefill", False, "interleaved"),
                                                 ("table4_16k_r8", True, "interleaved"),
                                                 # the two-kernel backward at head_dim 128 (a fixed dQ summation order)
                                                 ("llama8b_layer", True, "deterministic")])
def test_full_size_sampled(name, backward, route):
    w = synth.WORKLOADS[name]
    if route == "interleaved":
        out = run_attention_interleaved(w, backward=backward)
    else:
        out = run_attention(w, backward=backward, flags=ug.FLAG_DETERMINISTIC_DQ if route == "deterministic" else 0)
    inp = out["inputs"]
    s, T, r = w.num_sinks, w.raw_len, w.ratio
    k = oracle.window_units(w.window, r)
    N, G = w.total_len, w.num_q_heads // w.num_kv_heads
    scale = w.head_dim ** -0.5
    rng = np.random.default_rng(w.seed)
    sp, _, _ = oracle.layout(s, T, r)
    edge = sp[edge_positions(s, T, r, min(k, T // r))].astype(np.int64)  # interleaved indices of the edge rows
    hk0 = int(rng.integers(0, w.num_kv_heads))
    kv_heads = sorted({hk0, (hk0 + max(1, w.num_kv_heads // 2)) % w.num_kv_heads})
    # no row anywhere was left unwritten
    assert torch.isfinite(out["lse_shifted"]).all()
    assert torch.isfinite(out["o_shifted" if route != "interleaved" else "o"].float()).all()
    if backward:
        for n in ("dq", "dk", "dv"):
            assert torch.isfinite(out[n + "_shifted" if route != "interleaved" else n].float()).all(), n
    # forward: every batch index, two KV heads; the edge rows one by one and three blocks of 16 consecutive rows
    for b in range(w.batch):
        for hk in kv_heads:
            hs = slice(hk * G, (hk + 1) * G)
            q, kk, v = f64(inp["q"][b, :, hs]), f64(inp["k"][b, :, hk]), f64(inp["v"][b, :, hk])
            o_gpu, lse_gpu = f64(out["o"][b, :, hs]), f64(out["lse"][b, hs])
            blocks = [(int(t), int(t) + 1) for t in edge]
            blocks += [(r0, r0 + 16) for r0 in (0, int(rng.integers(16, N - 32)), N - 16)]
            for r0, r1 in blocks:
                o, lse = oracle.attn_fwd_slice(s, T, r, k, scale, q, kk, v, r0, r1)
                check_close(f"O b{b} hk{hk} rows {r0}:{r1}", o_gpu[r0:r1], o, TOL_O_MAX, TOL_O_MEAN if r1 - r0 > 1 else None)
                check_close(f"LSE b{b} hk{hk} rows {r0}:{r1}", lse_gpu[:, r0:r1].T, lse, TOL_LSE)
    if not backward:
        return
    # backward: first and last batch index, the same two KV heads; dQ of the edge rows, dK / dV of the edge keys (among
    # them gist keys, which every later row sees: the oracle walks all rows of the slice)
    keys = np.unique(np.concatenate([edge, [0, 1, r, N // 2, N - 2, N - 1]])).astype(np.int64)
    rows = np.unique(np.concatenate([edge, np.arange(0, 8), np.arange(N - 8, N)])).astype(np.int64)
    for b in sorted({0, w.batch - 1}):
        for hk in kv_heads:
            hs = slice(hk * G, (hk + 1) * G)
            q, kk, v = f64(inp["q"][b, :, hs]), f64(inp["k"][b, :, hk]), f64(inp["v"][b, :, hk])
            do = f64(inp["dout"][b, :, hs])
            dq, dk, dv = oracle.attn_bwd_sample(s, T, r, k, scale, q, kk, v, do, rows, keys)
            check_close(f"dQ rows b{b} hk{hk}", f64(out["dq"][b, rows][:, hs]), dq, TOL_GRAD)
            check_close(f"dK keys b{b} hk{hk}", f64(out["dk"][b, keys, hk]), dk, TOL_GRAD)
            check_close(f"dV keys b{b} hk{hk}", f64(out["dv"][b, keys, hk]), dv, TOL_GRAD)
