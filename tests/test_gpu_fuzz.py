"""Seeded random shapes: the closed-form tile intervals and masks of the CUDA path against the oracle's explicit
mask on problems nobody picked by hand (ratios that do and do not divide the tile, windows shorter and longer than
a unit or a tile, sink prefixes that end inside a tile, odd group sizes, several batch entries)."""
import numpy as np
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth
from oracle import oracle

from gpu_util import (TOL_GRAD, TOL_LSE, TOL_O_MAX, TOL_O_MEAN, check_close, f64, run_attention,
                      run_attention_interleaved)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PG = synth.PAGE


def _random_workloads(count, seed, max_len=1700):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        r = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 16, 32, 64, 128, 256]))
        n = int(rng.integers(1, max(2, (max_len - 300) // (r + 1)) + 1))
        T = n * r
        s = int(rng.choice([0, 0, 1, 7, 64, 128, 129, 300]))
        if s + T + n > max_len or s + T + n < max_len // 8:
            continue
        W = int(rng.choice([0, max(r - 1, 0), r, 3 * r + 1, 128, 130, 700, 1024, 10 ** 6]))
        Hkv = int(rng.choice([1, 2, 3]))
        G = int(rng.choice([1, 2, 3, 4, 8]))
        D = int(rng.choice([64, 128]))
        B = int(rng.choice([1, 1, 2, 3]))
        if B * Hkv * G > 24:
            continue
        # dO scaled down with the group size: G heads add into one dK / dV row and the gradient tolerance is absolute
        out.append(synth.Workload(f"fuzz{len(out)}_s{s}_T{T}_r{r}_W{W}_h{Hkv * G}x{Hkv}_d{D}_b{B}", B, T, r, W, Hkv * G, Hkv, D,
                                  num_sinks=s, k_scale=float(rng.choice([0.5, 1.0])), dout_scale=1.0 / max(1, G // 2),
                                  seed=int(rng.integers(1, 2 ** 31))))
    return out


@pytest.mark.parametrize("w", _random_workloads(40, 20250915) + _random_workloads(12, 99, max_len=5200), ids=lambda w: w.name)
def test_random_attention_problems(w):
    k = oracle.window_units(w.window, w.ratio)
    scale = w.head_dim ** -0.5
    inp = synth.attention_inputs(w)
    q, kk, v, do = (f64(inp[n]) for n in ("q", "k", "v", "dout"))
    o, lse = oracle.attn_fwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v)
    dq, dk, dv = oracle.attn_bwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v, do)
    runs = [run_attention]
    if w.head_dim == 128 and 128 % w.ratio == 0:
        runs.append(run_attention_interleaved)
    for run in runs:
        out = run(w, inputs=inp)
        check_close("O", f64(out["o"]), o, TOL_O_MAX, TOL_O_MEAN)
        check_close("LSE", f64(out["lse"]), lse, TOL_LSE)
        check_close("dQ", f64(out["dq"]), dq, TOL_GRAD)
        check_close("dK", f64(out["dk"]), dk, TOL_GRAD)
        check_close("dV", f64(out["dv"]), dv, TOL_GRAD)


def _random_doc_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(count):
        r = int(rng.choice([1, 2, 4, 8, 16]))
        s = int(rng.choice([0, 0, 3, 8]))
        W = int(rng.choice([0, r, 2 * r, 64, 10 ** 6]))
        docs = [int(rng.choice([1, 1, 2, 3, 5, 9, 17, 40])) * r for _ in range(int(rng.integers(1, 20)))]
        while sum(s + T + T // r for T in docs) > 1500:
            docs.pop()
        Hkv = int(rng.choice([1, 2]))
        G = int(rng.choice([1, 2, 4]))
        D = int(rng.choice([64, 128]))
        il = bool(D == 128 and 128 % r == 0 and rng.integers(0, 2))
        out.append((s, r, W, docs or [r], Hkv * G, Hkv, D, il, int(rng.integers(1, 2 ** 31))))
    return out


@pytest.mark.parametrize("case", _random_doc_cases(16, 7), ids=lambda c: f"s{c[0]}_r{c[1]}_W{c[2]}_{len(c[3])}docs_d{c[6]}_il{int(c[7])}")
def test_random_packed_samples(case):
    s, r, W, doc_T, Hq, Hkv, D, il, seed = case
    k_units = (W + r - 1) // r
    p = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED if il else 0)
    n_tot = ug.unigist_docs_total_len(p, doc_T)
    g = torch.Generator().manual_seed(seed)
    q, k, v, do = (torch.randn(n_tot, h, D, generator=g).to(torch.bfloat16) for h in (Hq, Hkv, Hkv, Hq))  # interleaved
    scale = D ** -0.5
    o_ref, lse_ref = oracle.docs_attn_fwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v))
    dq_ref, dk_ref, dv_ref = oracle.docs_attn_bwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v), f64(do))
    perm, base = [], 0
    for T in doc_T:  # per-document shift permutation of the packed rows
        sp, _, _ = oracle.layout(s, T, r)
        perm.append(base + sp.astype(np.int64))
        base += len(sp)
    perm = torch.from_numpy(np.concatenate(perm))
    to_lib = (lambda t: t.to(DEV)) if il else (lambda t: t[perm].contiguous().to(DEV))
    qd, kd, vd, dod = to_lib(q), to_lib(k), to_lib(v), to_lib(do)
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((Hq * n_tot,), float("nan"), device=DEV)
    ug.unigist_attn_fwd_docs(p, doc_T, qd, kd, vd, o, lse)
    ws = torch.empty(max(ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T), 16), dtype=torch.uint8, device=DEV)
    dq, dk, dv = (torch.full_like(t, float("nan")) for t in (qd, kd, vd))
    ug.unigist_attn_bwd_docs(p, doc_T, qd, kd, vd, o, lse, dod, dq, dk, dv, ws)
    ug.unigist_device_status()

    def from_lib(t):
        t = t.cpu()
        if il:
            return t
        out = torch.empty_like(t)
        out[perm] = t
        return out

    check_close("o", f64(from_lib(o)), o_ref, TOL_O_MAX, TOL_O_MEAN)
    check_close("dq", f64(from_lib(dq)), dq_ref, TOL_GRAD)
    check_close("dk", f64(from_lib(dk)), dk_ref, TOL_GRAD)
    check_close("dv", f64(from_lib(dv)), dv_ref, TOL_GRAD)
    lse_h, base = lse.cpu().double().numpy(), 0
    for T in doc_T:
        sp, _, _ = oracle.layout(s, T, r)
        blk = lse_h[Hq * base: Hq * (base + len(sp))].reshape(Hq, len(sp))
        check_close("lse", blk, lse_ref[:, base + sp], TOL_LSE)
        base += len(sp)


def test_random_decode_batches():
    rng = np.random.default_rng(11)
    for it in range(12):
        Hkv = int(rng.choice([1, 2, 8]))
        G = int(rng.choice([1, 2, 3, 4, 8]))
        S = int(rng.integers(1, 9))
        w = synth.DecodeWorkload("fuzz", S, int(rng.integers(1, 1200)), int(rng.integers(0, 300)), Hkv * G, Hkv, 128,
                                 seed=int(rng.integers(1, 2 ** 31)))
        inp = synth.decode_inputs(w, spare_blocks=int(rng.integers(0, 4)))
        lens = [int(rng.integers(0, w.seq_len + 1)) for _ in range(S)]
        lens[int(rng.integers(0, S))] = w.seq_len
        d = {k: v.to(DEV) for k, v in inp.items()}
        d["seq_lens"] = torch.tensor(lens, dtype=torch.int32, device=DEV)
        ws = torch.empty(ug.unigist_decode_workspace_bytes(S, w.num_q_heads, Hkv, 128, d["block_table"].shape[1]),
                         dtype=torch.uint8, device=DEV)
        o = torch.full_like(d["q"], float("nan"))
        lse = torch.full((S, w.num_q_heads), float("nan"), dtype=torch.float32, device=DEV)
        ug.unigist_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o, lse, ws)
        ug.unigist_device_status()
        for i in range(S):
            if lens[i] == 0:
                assert not o[i].float().any() and torch.isinf(lse[i]).all()
                continue
            rows = lambda c: c[inp["block_table"][i].long()].permute(0, 2, 1, 3).reshape(-1, Hkv, 128)[:lens[i]]
            oo, ll = oracle.decode(128 ** -0.5, f64(inp["q"][i:i + 1]), [f64(rows(inp["k_cache"]))], [f64(rows(inp["v_cache"]))])
            check_close(f"decode O batch {it} seq {i}", f64(o[i:i + 1]), oo, TOL_O_MAX, TOL_O_MEAN)
            check_close(f"decode LSE batch {it} seq {i}", f64(lse[i:i + 1]), ll, TOL_LSE)
