"""Every call is asynchronous on the caller's stream and on nothing else: issued on a side stream behind work
that is still running, it must see the inputs that work produces.  Each case fills its inputs on a non-blocking
side stream after a spin of a tenth of a second, calls the library there without any synchronisation in between, and
compares with the same call on settled inputs; a kernel launched on another stream would read the buffers before
they are filled."""
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth

from gpu_util import problem_of

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SPIN = 200_000_000  # clocks the side stream is kept busy before the inputs appear


def _late(side, host_tensors):
    """Device buffers (NaN for floating point, zero for indices, so that a premature reader stays in bounds) that
    receive their values on `side` only after the spin."""
    bufs = [torch.full(t.shape, float("nan") if t.is_floating_point() else 0, dtype=t.dtype, device=DEV)
            for t in host_tensors]
    srcs = [t.to(DEV) for t in host_tensors]
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        torch.cuda._sleep(SPIN)
        for b, s in zip(bufs, srcs):
            b.copy_(s, non_blocking=True)
            s.record_stream(side)  # the allocator must not hand the source to anyone before the copy has run
    return bufs


@pytest.mark.parametrize("w,flags", [
    (synth.Workload("stream_128", 2, 1024, 8, 128, 4, 2, 128, num_sinks=3, seed=601), ug.FLAG_INTERLEAVED),
    (synth.Workload("stream_64", 1, 770, 7, 70, 4, 2, 64, num_sinks=2, seed=602), 0),
], ids=lambda x: x.name if isinstance(x, synth.Workload) else str(x))
def test_attention_on_a_side_stream(w, flags):
    inp = synth.attention_inputs(w)
    p = problem_of(w, flags)
    N = w.total_len

    def call(make_inputs, stream):
        o, dq = (torch.full(inp["q"].shape, float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(2))
        dk, dv = (torch.full(inp["k"].shape, float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(2))
        lse = torch.full((w.batch, w.num_q_heads, N), float("nan"), device=DEV)
        ws = torch.empty(max(16, ug.unigist_workspace_bytes(p, ug.OP_BWD)), dtype=torch.uint8, device=DEV)
        torch.cuda.synchronize()  # the outputs above are settled; nothing below waits for anything
        q, k, v, do = make_inputs()
        ug.unigist_attn_fwd(p, q, k, v, o, lse, stream=stream)
        ug.unigist_attn_bwd(p, q, k, v, o, lse, do, dq, dk, dv, ws, stream=stream)
        return o, lse, dk, dv, dq

    want = call(lambda: [inp[n].to(DEV) for n in ("q", "k", "v", "dout")], torch.cuda.current_stream())
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    got = call(lambda: _late(side, [inp[n] for n in ("q", "k", "v", "dout")]), side)
    side.synchronize()
    ug.unigist_device_status()
    for a, b in zip(got[:4], want[:4]):
        assert torch.equal(a, b)
    assert (got[4].float() - want[4].float()).abs().max().item() <= 2.0 ** -7


def test_packed_documents_on_a_side_stream():
    s, r, W, doc_T, Hq, Hkv, D = 0, 4, 8, [256, 128, 64, 64, 192], 4, 2, 128
    p = ug.Problem(1, doc_T[0], r, W, Hq, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED)
    n_tot = ug.unigist_docs_total_len(p, doc_T)
    g = torch.Generator().manual_seed(603)
    host = [torch.randn(n_tot, h, D, generator=g).to(torch.bfloat16) for h in (Hq, Hkv, Hkv, Hq)]

    def call(make_inputs, stream):
        o, dq = (torch.full(host[0].shape, float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(2))
        dk, dv = (torch.full(host[1].shape, float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(2))
        lse = torch.full((Hq * n_tot,), float("nan"), device=DEV)
        ws = torch.empty(max(16, ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, doc_T)), dtype=torch.uint8, device=DEV)
        torch.cuda.synchronize()
        q, k, v, do = make_inputs()
        ug.unigist_attn_fwd_docs(p, doc_T, q, k, v, o, lse, stream=stream)
        ug.unigist_attn_bwd_docs(p, doc_T, q, k, v, o, lse, do, dq, dk, dv, ws, stream=stream)
        return o, lse, dk, dv, dq

    want = call(lambda: [t.to(DEV) for t in host], torch.cuda.current_stream())
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    got = call(lambda: _late(side, host), side)
    side.synchronize()
    ug.unigist_device_status()
    for a, b in zip(got[:4], want[:4]):
        assert torch.equal(a, b)
    assert (got[4].float() - want[4].float()).abs().max().item() <= 2.0 ** -7


def test_cache_calls_on_a_side_stream():
    """Compaction into the paged cache, then decode over it (both variants), then the gist shift and the rotary
    embedding: all issued back to back on the side stream."""
    B, s, T, r, W, Hq, Hkv, D = 2, 3, 1024, 8, 128, 8, 2, 128
    w = synth.Workload("stream_cache", B, T, r, W, Hq, Hkv, D, num_sinks=s, seed=604)
    inp = synth.attention_inputs(w, with_grad=False)
    p, p_shifted = problem_of(w, ug.FLAG_INTERLEAVED), problem_of(w)
    L = ug.unigist_compact_len(p)
    per_seq = -(-L // synth.PAGE)
    nb = B * per_seq + 1
    table_h = torch.randperm(nb, generator=torch.Generator().manual_seed(5))[:B * per_seq].to(torch.int32).reshape(B, per_seq)
    qd_h = inp["q"][:, -1].contiguous()

    def call(make_inputs, stream):
        kc = torch.zeros(nb, Hkv, synth.PAGE, D, dtype=torch.bfloat16, device=DEV)
        vc = torch.zeros_like(kc)
        lens = torch.zeros(B, dtype=torch.int32, device=DEV)
        o1, o2 = (torch.full(qd_h.shape, float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(2))
        ws = torch.empty(ug.unigist_decode_workspace_bytes(B, Hq, Hkv, D, per_seq), dtype=torch.uint8, device=DEV)
        k_sh, k_rot = (torch.full(inp["k"].shape, float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(2))
        torch.cuda.synchronize()
        k, v, qd, table = make_inputs()
        ug.unigist_kv_compact(p, k, v, kc, vc, table, lens, stream=stream)
        ug.unigist_decode(qd, kc, vc, table, lens, o1, None, ws, stream=stream)
        ug.unigist_decode_static(qd, kc, vc, table, lens, o2, stream=stream)
        ug.unigist_gist_shift(p_shifted, k, k_sh, stream=stream)
        ug.unigist_rope(p_shifted, k, k_rot, 10000.0, ug.ROPE_TO_SHIFTED, stream=stream)
        return kc, vc, lens, o1, o2, k_sh, k_rot

    want = call(lambda: [inp["k"].to(DEV), inp["v"].to(DEV), qd_h.to(DEV), table_h.to(DEV)], torch.cuda.current_stream())
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    got = call(lambda: _late(side, [inp["k"], inp["v"], qd_h, table_h]), side)
    side.synchronize()
    ug.unigist_device_status()
    for a, b in zip(got, want):
        assert torch.equal(a, b)
    assert got[2].tolist() == [L] * B and torch.isfinite(got[3].float()).all()
