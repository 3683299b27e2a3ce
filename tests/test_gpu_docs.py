"""Cross-document masking (Section 5.1): packed documents through the library against the dense oracle."""
import numpy as np
import pytest
import torch

import paper_2509_15763_b200 as ug
from oracle import oracle
from gpu_util import TOL_GRAD, TOL_LSE, TOL_O_MAX, TOL_O_MEAN, check_close, f64

pytestmark = pytest.mark.gpu

CASES = [
    # s, r, W, doc_T, Hq, Hkv, D, interleaved
    (0, 4, 8, [256, 64, 64, 132], 4, 2, 128, False),   # a run of two equal documents, a ragged one
    (0, 4, 8, [256, 64, 64, 132], 4, 2, 128, True),
    (8, 8, 16, [40, 304, 8], 2, 1, 128, False),         # sinks in every document; a one-unit document
    (8, 8, 16, [40, 304, 8], 2, 1, 128, True),
    (0, 2, 4, [66, 130], 2, 2, 64, False),              # head_dim 64 (two-kernel backward)
    (0, 4, 8, [64, 128, 64, 192, 64, 256], 2, 2, 128, True),  # six units of different lengths in one launch
    # fifteen units: more than one launch holds (twelve), with sinks, a batch of three equal documents and a tiny one
    (4, 4, 8, [64, 32, 96, 32, 32, 32, 160, 8, 64, 128, 36, 72, 40, 44, 48, 52, 56], 4, 2, 128, False),
    (0, 8, 16, [64, 32, 96, 32, 32, 32, 160, 8, 64, 128, 16, 72, 40, 24, 48, 56, 80], 2, 2, 128, True),
]


def _packed_inputs(n_tot, Hq, Hkv, D, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda h: torch.randn(n_tot, h, D, generator=g).to(torch.bfloat16)
    return mk(Hq), mk(Hkv), mk(Hkv), mk(Hq)


@pytest.mark.parametrize("case", CASES)
def test_docs_match_oracle(case):
    s, r, W, doc_T, Hq, Hkv, D, il = case
    k_units = (W + r - 1) // r
    p = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED if il else 0)
    n_tot = ug.unigist_docs_total_len(p, doc_T)
    assert n_tot == sum(oracle.total_len(s, T, r) for T in doc_T)
    q, k, v, do = _packed_inputs(n_tot, Hq, Hkv, D, 77 + len(doc_T) + s)  # interleaved order, packed
    scale = 1.0 / np.sqrt(D)
    o_ref, lse_ref = oracle.docs_attn_fwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v))
    dq_ref, dk_ref, dv_ref = oracle.docs_attn_bwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v), f64(do))

    # per-document shift permutation of the packed rows (shifted position -> interleaved row)
    perm, base = [], 0
    for T in doc_T:
        sp, _, _ = oracle.layout(s, T, r)
        perm.append(base + sp.astype(np.int64))
        base += len(sp)
    perm = torch.from_numpy(np.concatenate(perm))
    dev = torch.device("cuda:0")
    to_lib = (lambda t: t.to(dev)) if il else (lambda t: t[perm].contiguous().to(dev))
    qd, kd, vd, dod = to_lib(q), to_lib(k), to_lib(v), to_lib(do)
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((Hq * n_tot,), float("nan"), device=dev)
    ug.unigist_attn_fwd_docs(p, doc_T, qd, kd, vd, o, lse)
    ws = torch.empty(max(ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T), 16), dtype=torch.uint8, device=dev)
    dq, dk, dv = (torch.full_like(t, float("nan")) for t in (qd, kd, vd))
    ug.unigist_attn_bwd_docs(p, doc_T, qd, kd, vd, o, lse, dod, dq, dk, dv, ws)
    ug.unigist_device_status()

    def from_lib(t):  # back to interleaved packed order on the host
        t = t.cpu()
        if il:
            return t
        out = torch.empty_like(t)
        out[perm] = t
        return out

    check_close("o", f64(from_lib(o)), o_ref, TOL_O_MAX, TOL_O_MEAN)
    # lse: one [Hq, N_d] block per document, shifted order inside
    lse_h = lse.cpu().double().numpy()
    base = 0
    for T in doc_T:
        sp, _, _ = oracle.layout(s, T, r)
        n = len(sp)
        blk = lse_h[Hq * base: Hq * (base + n)].reshape(Hq, n)
        check_close("lse", blk, lse_ref[:, base + sp], TOL_LSE)
        base += n
    check_close("dq", f64(from_lib(dq)), dq_ref, TOL_GRAD)
    check_close("dk", f64(from_lib(dk)), dk_ref, TOL_GRAD)
    check_close("dv", f64(from_lib(dv)), dv_ref, TOL_GRAD)


@pytest.mark.parametrize("D,il", [(128, True), (128, False), (64, False)])
def test_docs_backward_takes_an_fp32_dout(D, il):
    """UNIGIST_FLAG_DOUT_FP32 on a packed sample: the gradients of the same dO rounded to bf16, bit for bit."""
    s, r, W, doc_T, Hq, Hkv = 4, 4, 8, [64, 132, 64, 64, 8], 4, 2
    flags = ug.FLAG_INTERLEAVED if il else 0
    p16 = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=flags)
    p32 = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=flags | ug.FLAG_DOUT_FP32)
    n_tot = ug.unigist_docs_total_len(p16, doc_T)
    dev = torch.device("cuda:0")
    q, k, v, _ = (t.to(dev) for t in _packed_inputs(n_tot, Hq, Hkv, D, 31))
    do32 = torch.randn(n_tot, Hq, D, generator=torch.Generator().manual_seed(32)).to(dev)
    o = torch.empty_like(q)
    lse = torch.empty(Hq * n_tot, device=dev)
    ug.unigist_attn_fwd_docs(p16, doc_T, q, k, v, o, lse)
    got = {}
    for p, do in ((p16, do32.to(torch.bfloat16)), (p32, do32)):
        ws = torch.empty(max(ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T), 16), dtype=torch.uint8, device=dev)
        dq, dk, dv = (torch.full_like(t, float("nan")) for t in (q, k, v))
        ug.unigist_attn_bwd_docs(p, doc_T, q, k, v, o, lse, do, dq, dk, dv, ws)
        ug.unigist_device_status()
        got[p is p32] = (dq, dk, dv)
    assert torch.isfinite(got[True][0].float()).all()
    assert torch.equal(got[True][1], got[False][1]) and torch.equal(got[True][2], got[False][2])
    assert (got[True][0].float() - got[False][0].float()).abs().max().item() <= 2.0 ** -7


def test_docs_backward_with_a_fixed_dq_order():
    """UNIGIST_FLAG_DETERMINISTIC_DQ on a packed sample (head_dim 128): against the oracle, and the same bits twice."""
    s, r, W, doc_T, Hq, Hkv, D = 4, 4, 8, [64, 132, 64, 64, 8, 256], 4, 2, 128
    k_units = (W + r - 1) // r
    p = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=ug.FLAG_DETERMINISTIC_DQ)
    n_tot = ug.unigist_docs_total_len(p, doc_T)
    q, k, v, do = _packed_inputs(n_tot, Hq, Hkv, D, 41)  # interleaved order, packed
    scale = 1.0 / np.sqrt(D)
    dq_ref, dk_ref, dv_ref = oracle.docs_attn_bwd(s, doc_T, r, k_units, scale, f64(q), f64(k), f64(v), f64(do))
    perm, base = [], 0
    for T in doc_T:
        sp, _, _ = oracle.layout(s, T, r)
        perm.append(base + sp.astype(np.int64))
        base += len(sp)
    perm = torch.from_numpy(np.concatenate(perm))
    dev = torch.device("cuda:0")
    qd, kd, vd, dod = (t[perm].contiguous().to(dev) for t in (q, k, v, do))
    o = torch.empty_like(qd)
    lse = torch.empty(Hq * n_tot, device=dev)
    ug.unigist_attn_fwd_docs(p, doc_T, qd, kd, vd, o, lse)
    ws = torch.empty(max(ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T), 16), dtype=torch.uint8, device=dev)
    got = []
    for _ in range(2):
        dq, dk, dv = (torch.full_like(t, float("nan")) for t in (qd, kd, vd))
        ug.unigist_attn_bwd_docs(p, doc_T, qd, kd, vd, o, lse, dod, dq, dk, dv, ws)
        ug.unigist_device_status()
        got.append((dq, dk, dv))
    for a, b in zip(*got):
        assert torch.equal(a, b)

    def from_lib(t):
        out = torch.empty_like(t.cpu())
        out[perm] = t.cpu()
        return out

    check_close("dq", f64(from_lib(got[0][0])), dq_ref, TOL_GRAD)
    check_close("dk", f64(from_lib(got[0][1])), dk_ref, TOL_GRAD)
    check_close("dv", f64(from_lib(got[0][2])), dv_ref, TOL_GRAD)


def test_docs_reject_bad_lists():
    p = ug.Problem(1, 16, 4, 8, 2, 2, 128)
    x = torch.zeros(64, 2, 128, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(2 * 64, device="cuda")
    with pytest.raises(ug.UnigistError):
        ug.unigist_attn_fwd_docs(p, [16, 6], x, x, x, x, lse)  # 6 is not a multiple of the ratio
    assert ug.unigist_docs_total_len(p, [16, 6]) == -1
    p2 = ug.Problem(2, 16, 4, 8, 2, 2, 128)
    with pytest.raises(ug.UnigistError):
        ug.unigist_attn_fwd_docs(p2, [16], x, x, x, x, lse)  # batch must be 1


def test_docs_calls_can_be_captured_in_a_cuda_graph():
    """A packed sample's forward + backward only enqueues kernels on the caller's stream (the documents' tensor
    maps are kernel parameters), so it is capturable; a replay gives what the eager calls gave."""
    s, r, W, doc_T, Hq, Hkv, D = 0, 4, 8, [256, 128, 64, 64, 192], 4, 2, 128
    p = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED)
    n_tot = ug.unigist_docs_total_len(p, doc_T)
    dev = torch.device("cuda:0")
    q, k, v, do = (t.to(dev) for t in _packed_inputs(n_tot, Hq, Hkv, D, 5))
    o = torch.empty_like(q)
    lse = torch.empty(Hq * n_tot, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(max(ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T), 16), dtype=torch.uint8, device=dev)

    def run():
        ug.unigist_attn_fwd_docs(p, doc_T, q, k, v, o, lse)
        ug.unigist_attn_bwd_docs(p, doc_T, q, k, v, o, lse, do, dq, dk, dv, ws)

    run()
    torch.cuda.synchronize()
    want = [t.clone() for t in (o, lse, dk, dv)]
    want_dq = dq.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            run()
    for t in (o, lse, dq, dk, dv):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ug.unigist_device_status()
    for got, ref in zip((o, lse, dk, dv), want):
        assert torch.equal(got, ref)
    assert (dq.float() - want_dq.float()).abs().max().item() <= 2.0 ** -7  # dQ: up to its summation order
