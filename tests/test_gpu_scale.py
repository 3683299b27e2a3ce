"""A caller-given softmax scale (the problem's `softmax_scale`, decode's argument) instead of the default
1 / sqrt(head_dim): every entry point that takes one, against the oracle at the same scale."""
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


@pytest.mark.parametrize("w,scale,route", [
    (synth.Workload("scale_128", 2, 1024, 8, 128, 4, 2, 128, num_sinks=3, seed=501), 0.031, "explicit"),
    (synth.Workload("scale_128", 2, 1024, 8, 128, 4, 2, 128, num_sinks=3, seed=501), 0.2, "interleaved"),
    (synth.Workload("scale_64", 1, 770, 7, 70, 4, 2, 64, num_sinks=2, seed=502), 0.25, "explicit"),
], ids=lambda x: x.name if isinstance(x, synth.Workload) else str(x))
def test_attention_with_a_given_scale(w, scale, route):
    run = run_attention if route == "explicit" else run_attention_interleaved
    out = run(w, softmax_scale=scale)
    inp = out["inputs"]
    k = oracle.window_units(w.window, w.ratio)
    q, kk, v, do = (f64(inp[n]) for n in ("q", "k", "v", "dout"))
    o, lse = oracle.attn_fwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v)
    check_close("O", f64(out["o"]), o, TOL_O_MAX, TOL_O_MEAN)
    check_close("LSE", f64(out["lse"]), lse, TOL_LSE)
    dq, dk, dv = oracle.attn_bwd(w.num_sinks, w.raw_len, w.ratio, k, scale, q, kk, v, do)
    check_close("dQ", f64(out["dq"]), dq, TOL_GRAD)
    check_close("dK", f64(out["dk"]), dk, TOL_GRAD)
    check_close("dV", f64(out["dv"]), dv, TOL_GRAD)
    # the scale is not ignored: the default one gives another O
    assert (f64(run(w, backward=False, inputs=inp)["o"]) - o).__abs__().max() > TOL_O_MAX


def test_packed_documents_with_a_given_scale():
    s, r, W, doc_T, Hq, Hkv, D, scale = 2, 4, 8, [64, 132, 64, 64, 8], 4, 2, 128, 0.15
    k_units = (W + r - 1) // r
    p = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, softmax_scale=scale, flags=ug.FLAG_INTERLEAVED)
    n_tot = ug.unigist_docs_total_len(p, doc_T)
    g = torch.Generator().manual_seed(503)
    q, k, v, do = (torch.randn(n_tot, h, D, generator=g).to(torch.bfloat16) for h in (Hq, Hkv, Hkv, Hq))
    o_ref, lse_ref = oracle.docs_attn_fwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v))
    dq_ref, dk_ref, dv_ref = oracle.docs_attn_bwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v), f64(do))
    qd, kd, vd, dod = (t.to(DEV) for t in (q, k, v, do))
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((Hq * n_tot,), float("nan"), device=DEV)
    ug.unigist_attn_fwd_docs(p, doc_T, qd, kd, vd, o, lse)
    ws = torch.empty(max(ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T), 16), dtype=torch.uint8, device=DEV)
    dq, dk, dv = (torch.full_like(t, float("nan")) for t in (qd, kd, vd))
    ug.unigist_attn_bwd_docs(p, doc_T, qd, kd, vd, o, lse, dod, dq, dk, dv, ws)
    ug.unigist_device_status()
    check_close("o", f64(o), o_ref, TOL_O_MAX, TOL_O_MEAN)
    check_close("dq", f64(dq), dq_ref, TOL_GRAD)
    check_close("dk", f64(dk), dk_ref, TOL_GRAD)
    check_close("dv", f64(dv), dv_ref, TOL_GRAD)
    lse_h, base = lse.cpu().double().numpy(), 0
    for T in doc_T:  # one [Hq, N_d] block per document, shifted order inside
        sp, _, _ = oracle.layout(s, T, r)
        blk = lse_h[Hq * base: Hq * (base + len(sp))].reshape(Hq, len(sp))
        check_close("lse", blk, lse_ref[:, base + sp], TOL_LSE)
        base += len(sp)


@pytest.mark.parametrize("static", [False, True])
def test_decode_with_a_given_scale(static):
    w = synth.DecodeWorkload("scale", 3, 300, 45, 8, 2, 128, seed=504)
    inp = synth.decode_inputs(w, spare_blocks=1)
    d = {k: v.to(DEV) for k, v in inp.items()}
    lens = [w.seq_len, w.seq_len - 70, 5]
    d["seq_lens"] = torch.tensor(lens, dtype=torch.int32, device=DEV)
    o = torch.full_like(d["q"], float("nan"))
    lse = torch.full((w.num_seqs, w.num_q_heads), float("nan"), dtype=torch.float32, device=DEV)
    scale = 0.04
    if static:
        ug.unigist_decode_static(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o, lse,
                                 softmax_scale=scale)
    else:
        ws = torch.empty(ug.unigist_decode_workspace_bytes(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                                           d["block_table"].shape[1]), dtype=torch.uint8, device=DEV)
        ug.unigist_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o, lse, ws,
                          softmax_scale=scale)
    ug.unigist_device_status()
    for i in range(w.num_seqs):
        rows = lambda c: c[inp["block_table"][i].long()].permute(0, 2, 1, 3).reshape(-1, w.num_kv_heads, w.head_dim)[:lens[i]]
        oo, ll = oracle.decode(scale, f64(inp["q"][i:i + 1]), [f64(rows(inp["k_cache"]))], [f64(rows(inp["v_cache"]))])
        check_close(f"decode O seq {i}", f64(o[i:i + 1]), oo, TOL_O_MAX, TOL_O_MEAN)
        check_close(f"decode LSE seq {i}", f64(lse[i:i + 1]), ll, TOL_LSE)
