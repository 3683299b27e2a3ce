"""Maximum sizes: tensors of more than 2^32 bytes and 2^31 elements, so that an element or byte offset kept in 32
bits anywhere in the CUDA path (tile coordinates, row bases of LSE / Delta, the fp32 dQ accumulator, cache block
addresses) would land in the wrong place.  Each case is checked two ways: sampled outputs against the fp64
oracle at the far end of the tensors, and every batch index (or sequence) against the others by a property that
holds at any size (equal inputs give bit-equal outputs wherever they sit)."""
import numpy as np
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth
from oracle import oracle

from gpu_util import TOL_GRAD, TOL_LSE, TOL_O_MAX, TOL_O_MEAN, check_close, edge_positions, f64, problem_of

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PG = synth.PAGE


def _spread(t, B):
    """[2, ...] on the host -> [B, ...] on the device: sample 0 at every batch index but the last, sample 1 there."""
    out = torch.empty((B,) + tuple(t.shape[1:]), dtype=t.dtype, device=DEV)
    out[:B - 1] = t[0].to(DEV)
    out[B - 1] = t[1].to(DEV)
    return out


@pytest.mark.parametrize("D,B", [(128, 16), (64, 32)])
def test_attention_on_tensors_beyond_four_gib(D, B):
    """Forward + backward of B sequences of the training workload's geometry; Q, O, dO and dQ hold 2.7 G elements
    (5.4 GB) each, the fp32 dQ accumulator of head_dim 128 10.7 GB.  head_dim 128 runs on interleaved tensors (the
    route the benchmark times, fused backward), head_dim 64 on shifted ones (two-kernel backward)."""
    base = synth.WORKLOADS["train_batch"]
    w2 = base.scaled(batch=2, head_dim=D, seed=base.seed + 500 + D)
    inp = synth.attention_inputs(w2)
    s, T, r, Hq, Hkv = w2.num_sinks, w2.raw_len, w2.ratio, w2.num_q_heads, w2.num_kv_heads
    N, G = w2.total_len, Hq // Hkv
    assert B * N * Hq * D > 2 ** 31 and B * N * Hq * D * 2 > 2 ** 32
    interleaved = D == 128
    sp, up, _ = oracle.layout(s, T, r)
    up_d = torch.from_numpy(up).long().to(DEV)
    if not interleaved:  # hand the library shifted tensors
        inp_lib = {n: t[:, torch.from_numpy(sp).long()].contiguous() for n, t in inp.items()}
    else:
        inp_lib = inp
    flags = ug.FLAG_INTERLEAVED if interleaved else 0

    def run(p, d):
        o = torch.full_like(d["q"], float("nan"))
        lse = torch.full((p.batch, Hq, N), float("nan"), device=DEV, dtype=torch.float32)
        ug.unigist_attn_fwd(p, d["q"], d["k"], d["v"], o, lse)
        ws = torch.empty(max(16, ug.unigist_workspace_bytes(p, ug.OP_BWD)), dtype=torch.uint8, device=DEV)
        dq, dk, dv = (torch.full_like(d[n], float("nan")) for n in ("q", "k", "v"))
        ug.unigist_attn_bwd(p, d["q"], d["k"], d["v"], o, lse, d["dout"], dq, dk, dv, ws)
        ug.unigist_device_status()
        return {"o": o, "lse": lse, "dq": dq, "dk": dk, "dv": dv}

    big = run(problem_of(w2.scaled(batch=B), flags), {n: _spread(t, B) for n, t in inp_lib.items()})

    # (1) the last batch index (every offset at its largest) against the oracle: rows and keys at the tile edges
    k_units = oracle.window_units(w2.window, r)
    scale = D ** -0.5
    edge = sp[edge_positions(s, T, r, min(k_units, T // r))].astype(np.int64)  # interleaved indices
    hk = Hkv - 1
    hs = slice(hk * G, (hk + 1) * G)
    q, kk, v = f64(inp["q"][1, :, hs]), f64(inp["k"][1, :, hk]), f64(inp["v"][1, :, hk])
    do = f64(inp["dout"][1, :, hs])

    def tokens(name, idx):  # rows of a [B, N, H, D] result of the last batch index, by interleaved token index
        at = torch.from_numpy(np.asarray(idx)).long().to(DEV)
        return big[name][B - 1, at if interleaved else up_d[at]]

    lse_gpu = f64(big["lse"][B - 1, hs][:, up_d])  # shifted -> interleaved order
    for t in list(edge) + [0, N - 1]:
        o, lse = oracle.attn_fwd_slice(s, T, r, k_units, scale, q, kk, v, int(t), int(t) + 1)
        check_close(f"O row {t}", f64(tokens("o", [t])[:, hs]), o, TOL_O_MAX)
        check_close(f"LSE row {t}", lse_gpu[:, t:t + 1].T, lse, TOL_LSE)
    keys = np.unique(np.concatenate([edge, [0, r, N - 1]])).astype(np.int64)
    rows = np.unique(np.concatenate([edge, [0, N - 1]])).astype(np.int64)
    dq, dk, dv = oracle.attn_bwd_sample(s, T, r, k_units, scale, q, kk, v, do, rows, keys)
    check_close("dQ rows", f64(tokens("dq", rows)[:, hs]), dq, TOL_GRAD)
    check_close("dK keys", f64(tokens("dk", keys)[:, hk]), dk, TOL_GRAD)
    check_close("dV keys", f64(tokens("dv", keys)[:, hk]), dv, TOL_GRAD)

    # (2) every batch index: the same two samples as a batch of two give the same bits wherever the sample sits
    # (dQ of the fused backward: up to the order of its fp32 additions)
    small = run(problem_of(w2, flags), {n: t.to(DEV) for n, t in inp_lib.items()})
    for b in range(B):
        src = 1 if b == B - 1 else 0
        for n in ("o", "lse", "dk", "dv"):
            assert torch.equal(big[n][b], small[n][src]), (n, b)
        a, c = big["dq"][b].float(), small["dq"][src].float()
        assert ((a - c).abs() <= 2.0 ** -7 * c.abs().clamp(min=1.0)).all(), ("dq", b)


def test_shift_of_a_tensor_beyond_four_gib():
    B, s, T, r, H, D = 16, 0, 32768, 4, 32, 128
    p = ug.Problem(B, T, r, 2048, H, H, D, num_sinks=s)
    N = ug.unigist_total_len(p)
    assert B * N * H * D * 2 > 2 ** 32
    g = torch.Generator().manual_seed(11)
    two = torch.randn(2, N, H, D, generator=g).to(torch.bfloat16)
    x = _spread(two, B)
    sp, _, _ = oracle.layout(s, T, r)
    perm = torch.from_numpy(sp).long().to(DEV)
    y = torch.full_like(x, float("nan"))
    ug.unigist_gist_shift(p, x, y)
    for b in range(B):
        assert torch.equal(y[b], x[b, perm]), b
    x.fill_(float("nan"))
    ug.unigist_gist_unshift(p, y, x)
    torch.cuda.synchronize()
    assert torch.equal(x[0].cpu(), two[0]) and torch.equal(x[B - 1].cpu(), two[1])
    for b in range(1, B - 1):
        assert torch.equal(x[b], x[0]), b


def test_decode_over_a_cache_beyond_four_gib():
    """Eight sequences whose blocks are scattered over a cache of 36 000 blocks (4.7 GB per tensor): the blocks
    past 2^32 bytes are reached through the block table like any other."""
    S, Hq, Hkv, D, pool_blocks, copies = 8, 32, 8, 128, 3000, 12
    nb = pool_blocks * copies
    assert nb * Hkv * PG * D * 2 > 2 ** 32 and (2 ** 32 // (Hkv * PG * D * 2)) % pool_blocks != 0
    g = torch.Generator().manual_seed(synth.BASE_SEED + 77)
    q = torch.randn(S, Hq, D, generator=g).to(torch.bfloat16)
    k_pool = torch.randn(pool_blocks, Hkv, PG, D, generator=g).to(torch.bfloat16)
    v_pool = torch.randn(pool_blocks, Hkv, PG, D, generator=g).to(torch.bfloat16)
    # physical block p holds pool block p mod pool_blocks, scaled by (1 + copy / 16) so that no two copies are equal
    kc = torch.empty(nb, Hkv, PG, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.empty_like(kc)
    for c in range(copies):
        f = 1.0 + c / 16.0  # product in fp32, rounded to bf16: the host rebuilds the same values below
        kc[c * pool_blocks:(c + 1) * pool_blocks] = (k_pool.to(DEV).float() * f).to(torch.bfloat16)
        vc[c * pool_blocks:(c + 1) * pool_blocks] = (v_pool.to(DEV).float() * f).to(torch.bfloat16)
    per_seq = 150
    perm = torch.randperm(nb, generator=g)
    table = perm[:S * per_seq].reshape(S, per_seq).clone()
    # the last blocks of the cache and the two on either side of the 4 GiB line (a block listed twice is harmless: decode only reads)
    table[0, :4] = torch.tensor([nb - 1, nb - 2, 2 ** 32 // (Hkv * PG * D * 2), 2 ** 32 // (Hkv * PG * D * 2) - 1])
    table = table.to(torch.int32)
    lens = [per_seq * PG - 17 * i for i in range(S)]
    ws = torch.empty(ug.unigist_decode_workspace_bytes(S, Hq, Hkv, D, per_seq), dtype=torch.uint8, device=DEV)
    o = torch.full((S, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((S, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ug.unigist_decode(q.to(DEV), kc, vc, table.to(DEV), torch.tensor(lens, dtype=torch.int32, device=DEV), o, lse, ws)
    ug.unigist_device_status()
    assert (table.long() * Hkv * PG * D * 2 >= 2 ** 32).any(dim=1).all()  # every sequence reaches past 4 GiB

    def rows_of(pool, i):  # the sequence's cache rows, rebuilt on the host from the pool
        blocks = table[i].long()
        f = (1.0 + (blocks // pool_blocks).float() / 16.0).reshape(-1, 1, 1, 1)
        x = (pool[blocks % pool_blocks].float() * f).to(torch.bfloat16)  # [blocks, Hkv, PG, D]
        return x.permute(0, 2, 1, 3).reshape(-1, Hkv, D)[:lens[i]]

    for i in range(S):
        oo, ll = oracle.decode(D ** -0.5, f64(q[i:i + 1]), [f64(rows_of(k_pool, i))], [f64(rows_of(v_pool, i))])
        check_close(f"decode O seq {i}", f64(o[i:i + 1]), oo, TOL_O_MAX, TOL_O_MEAN)
        check_close(f"decode LSE seq {i}", f64(lse[i:i + 1]), ll, TOL_LSE)


def test_compaction_of_tensors_beyond_four_gib():
    """Sixteen prompts of the long-prefill geometry (K and V 4.6 GB each) gathered into their compressed caches:
    the kept rows of the last batch index, bit for bit, are the oracle's kept set of its sample."""
    B = 16
    w = synth.WORKLOADS["long_prefill"]
    s, T, r, Hkv, D = w.num_sinks, w.raw_len, w.ratio, w.num_kv_heads, w.head_dim
    p = ug.Problem(B, T, r, w.window, Hkv, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED)
    N, L = ug.unigist_total_len(p), ug.unigist_compact_len(p)
    assert B * N * Hkv * D * 2 > 2 ** 32
    g = torch.Generator().manual_seed(w.seed + 2000)
    k2 = torch.randn(2, N, Hkv, D, generator=g).to(torch.bfloat16)  # interleaved order (Eq. 2)
    v2 = torch.randn(2, N, Hkv, D, generator=g).to(torch.bfloat16)
    kept = torch.from_numpy(oracle.kept_set(s, T, r, oracle.window_units(w.window, r))).long()  # interleaved indices
    assert len(kept) == L
    per_seq = -(-L // PG)
    nb = B * per_seq + 7
    table = torch.randperm(nb, generator=g)[:B * per_seq].to(torch.int32).reshape(B, per_seq)
    kc = torch.zeros(nb, Hkv, PG, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    lens = torch.zeros(B, dtype=torch.int32, device=DEV)
    ug.unigist_kv_compact(p, _spread(k2, B), _spread(v2, B), kc, vc, table.to(DEV), lens)
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [L] * B

    def rows(cache, b):
        return cache[table[b].long().to(DEV)].permute(0, 2, 1, 3).reshape(-1, Hkv, D)[:L]

    for cache, src in ((kc, k2), (vc, v2)):
        assert torch.equal(rows(cache, B - 1).cpu(), src[1, kept])
        first = rows(cache, 0)
        assert torch.equal(first.cpu(), src[0, kept])
        for b in range(1, B - 1):
            assert torch.equal(rows(cache, b), first), b
