"""GPU parity for KV compaction (bit-exact) and decode over the paged compressed cache."""
import numpy as np
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth
from oracle import oracle

from gpu_util import TOL_LSE, TOL_O_MAX, TOL_O_MEAN, check_close, f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PG = ug.PAGE_TOKENS


def read_cache(cache, table_row, length):
    """Logical view [length, Hkv, D] of a paged cache."""
    blocks = cache[table_row[: -(-length // PG)].long()]           # [nb, Hkv, PG, D]
    return blocks.permute(0, 2, 1, 3).reshape(-1, cache.shape[1], cache.shape[3])[:length]


COMPACT_CASES = [
    # B, s, T, r, W, Hkv, D
    (2, 0, 448, 7, 64, 1, 64),
    (1, 5, 330, 5, 48, 2, 128),
    (1, 64, 1024, 8, 512, 2, 128),     # page aligned: in place is a table edit
    (2, 0, 2048, 16, 4096, 2, 128),    # window covers everything
    (1, 3, 640, 4, 0, 1, 64),          # no window
]


def _random_compact_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        r = int(rng.choice([1, 2, 3, 4, 7, 8, 16, 64, 128]))
        T = int(rng.integers(1, 2400 // r + 1)) * r
        s = int(rng.choice([0, 0, 1, 63, 64, 65, 128, 200]))
        W = int(rng.choice([0, r, 2 * r + 1, 64, 128, 500, 10 ** 6]))
        out.append((int(rng.choice([1, 2, 3])), s, T, r, W, int(rng.choice([1, 2, 8])), int(rng.choice([64, 128]))))
    return out


COMPACT_CASES += _random_compact_cases(12, 5)


@pytest.mark.parametrize("B,s,T,r,W,Hkv,D", COMPACT_CASES)
@pytest.mark.parametrize("mode", ["gather", "gather_interleaved", "inplace"])
def test_compaction_matches_oracle(B, s, T, r, W, Hkv, D, mode):
    interleaved = mode == "gather_interleaved"  # K, V handed over in interleaved order (UNIGIST_FLAG_INTERLEAVED)
    if interleaved:
        mode = "gather"
    p = ug.Problem(B, T, r, W, Hkv, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED if interleaved else 0)
    N, L = ug.unigist_total_len(p), ug.unigist_compact_len(p)
    k_units = oracle.window_units(W, r)
    kept = oracle.kept_set(s, T, r, k_units)              # interleaved indices, cache order
    sp, up, _ = oracle.layout(s, T, r)
    assert len(kept) == L
    g = torch.Generator().manual_seed(11)
    k_sh = torch.randn(B, N, Hkv, D, generator=g).to(torch.bfloat16)  # shifted order
    v_sh = torch.randn(B, N, Hkv, D, generator=g).to(torch.bfloat16)
    nbN, nbL = -(-N // PG), -(-L // PG)
    per_seq = nbN if mode == "inplace" else nbL
    nblocks = B * per_seq + 3
    table = torch.randperm(nblocks, generator=g)[: B * per_seq].to(torch.int32).reshape(B, per_seq)
    kc = torch.randn(nblocks, Hkv, PG, D, generator=g).to(torch.bfloat16)
    vc = torch.randn(nblocks, Hkv, PG, D, generator=g).to(torch.bfloat16)
    if mode == "inplace":  # the cache holds the whole shifted sequence
        for b in range(B):
            pad = torch.zeros(nbN * PG - N, Hkv, D, dtype=torch.bfloat16)
            for src, dst in ((k_sh, kc), (v_sh, vc)):
                full = torch.cat([src[b], pad]).reshape(nbN, PG, Hkv, D).permute(0, 2, 1, 3)
                dst[table[b].long()] = full
    kc_d, vc_d, table_d = kc.to(DEV), vc.to(DEV), table.to(DEV)
    lens = torch.zeros(B, dtype=torch.int32, device=DEV)
    kept_idx = torch.full((B, L), -1, dtype=torch.int32, device=DEV)
    ws = torch.empty(max(ug.unigist_workspace_bytes(p, ug.OP_COMPACT), 16), dtype=torch.uint8, device=DEV)
    if mode == "gather":
        src_k, src_v = k_sh, v_sh
        if interleaved:  # the same tokens, in the order of Eq. 2
            src_k, src_v = k_sh[:, torch.from_numpy(up).long()], v_sh[:, torch.from_numpy(up).long()]
        ug.unigist_kv_compact(p, src_k.contiguous().to(DEV), src_v.contiguous().to(DEV), kc_d, vc_d, table_d, lens,
                              kept_idx, ws)
    else:
        ug.unigist_kv_compact(p, None, None, kc_d, vc_d, table_d, lens, kept_idx, ws)
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [L] * B
    # indices: bit-exact against the oracle's kept set (mapped into shifted positions)
    want_idx = up[kept]
    assert np.array_equal(kept_idx.cpu().numpy(), np.tile(want_idx, (B, 1)))
    new_table = table_d.cpu()
    for b in range(B):
        assert sorted(new_table[b].tolist()) == sorted(table[b].tolist())  # a permutation of the row
        for cache, src in ((kc_d, k_sh), (vc_d, v_sh)):
            got = read_cache(cache.cpu(), new_table[b], L)
            assert torch.equal(got, src[b, torch.from_numpy(want_idx).long()])
    if mode == "gather":  # blocks outside the tables are untouched
        spare = sorted(set(range(nblocks)) - set(table.flatten().tolist()))
        assert torch.equal(kc_d.cpu()[spare], kc[spare])


@pytest.mark.parametrize("mode", ["gather_interleaved", "inplace"])
def test_compaction_of_the_long_prefill_at_full_size(mode):
    """The prefill workload's second half (Section 4.3): after the 131072-token prompt, the cache keeps the 8192
    gists and the last 4096 raw tokens of 139264.  Both routes a caller has at that size: the gather out of the
    interleaved K / V tensors (what the benchmark step does) and the in-place compaction of a paged cache that
    holds the whole shifted sequence (every segment is page aligned: a block-table edit).  Indices bit-exact
    against the oracle's brute-force kept set, pages byte-equal to the source rows."""
    w = synth.WORKLOADS["long_prefill"]
    s, T, r, Hkv, D = w.num_sinks, w.raw_len, w.ratio, w.num_kv_heads, w.head_dim
    il = mode == "gather_interleaved"
    p = ug.Problem(1, T, r, w.window, w.num_q_heads, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED if il else 0)
    N, L = ug.unigist_total_len(p), ug.unigist_compact_len(p)
    assert (N, L) == (139264, 12288)
    kept = oracle.kept_set(s, T, r, oracle.window_units(w.window, r))  # interleaved indices, cache order
    sp, up, _ = oracle.layout(s, T, r)
    want_idx = torch.from_numpy(up[kept]).long()
    assert len(kept) == L
    g = torch.Generator().manual_seed(w.seed + 1000)
    k_il = torch.randn(1, N, Hkv, D, generator=g).to(torch.bfloat16)  # interleaved order (Eq. 2)
    v_il = torch.randn(1, N, Hkv, D, generator=g).to(torch.bfloat16)
    k_sh, v_sh = k_il[:, torch.from_numpy(sp).long()], v_il[:, torch.from_numpy(sp).long()]
    nbN, nbL = N // PG, L // PG
    per_seq = nbL if il else nbN
    nblocks = per_seq + 5
    table = torch.randperm(nblocks, generator=g)[:per_seq].to(torch.int32).reshape(1, per_seq)
    kc = torch.zeros(nblocks, Hkv, PG, D, dtype=torch.bfloat16)
    vc = torch.zeros_like(kc)
    if not il:  # the cache holds the whole shifted sequence, logical position = shifted position
        for src, dst in ((k_sh, kc), (v_sh, vc)):
            dst[table[0].long()] = src[0].reshape(nbN, PG, Hkv, D).permute(0, 2, 1, 3)
    kc_d, vc_d, table_d = kc.to(DEV), vc.to(DEV), table.to(DEV)
    lens = torch.zeros(1, dtype=torch.int32, device=DEV)
    kept_idx = torch.full((1, L), -1, dtype=torch.int32, device=DEV)
    before = ug.unigist_launch_count()
    if il:
        ug.unigist_kv_compact(p, k_il.to(DEV), v_il.to(DEV), kc_d, vc_d, table_d, lens, kept_idx)
    else:
        ug.unigist_kv_compact(p, None, None, kc_d, vc_d, table_d, lens, kept_idx)
    torch.cuda.synchronize()
    assert ug.unigist_launch_count() == before + 1
    assert lens.cpu().tolist() == [L]
    assert np.array_equal(kept_idx.cpu().numpy()[0], want_idx.numpy())
    new_table = table_d.cpu()
    assert sorted(new_table[0].tolist()) == sorted(table[0].tolist())  # a permutation of the row
    for cache, src in ((kc_d, k_sh), (vc_d, v_sh)):
        assert torch.equal(read_cache(cache.cpu(), new_table[0], L), src[0, want_idx])
    if not il:  # no token moved: the cache bytes are what they were, and the freed blocks are listed after the kept ones
        assert torch.equal(kc_d.cpu(), kc) and torch.equal(vc_d.cpu(), vc)
        assert len(set(new_table[0, nbL:].tolist()) & set(new_table[0, :nbL].tolist())) == 0


def run_decode(inp, lens=None):
    d = {k: v.to(DEV) for k, v in inp.items()}
    if lens is not None:
        d["seq_lens"] = torch.tensor(lens, dtype=torch.int32, device=DEV)
    S, Hq, D = d["q"].shape
    Hkv = d["k_cache"].shape[1]
    ws = torch.empty(ug.unigist_decode_workspace_bytes(S, Hq, Hkv, D, d["block_table"].shape[1]),
                     dtype=torch.uint8, device=DEV)
    o = torch.full_like(d["q"], float("nan"))
    lse = torch.full((S, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ug.unigist_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o, lse, ws)
    torch.cuda.synchronize()
    return o, lse, d["seq_lens"].cpu().tolist()


def check_decode(inp, o, lse, lens, seqs):
    Hq, D = inp["q"].shape[1:]
    for i in seqs:
        kl = read_cache(inp["k_cache"], inp["block_table"][i], lens[i])
        vl = read_cache(inp["v_cache"], inp["block_table"][i], lens[i])
        oo, ll = oracle.decode(D ** -0.5, f64(inp["q"][i:i + 1]), [f64(kl)], [f64(vl)])
        check_close(f"decode O seq {i}", f64(o[i:i + 1]), oo, TOL_O_MAX, TOL_O_MEAN)
        check_close(f"decode LSE seq {i}", f64(lse[i:i + 1]), ll, TOL_LSE)


@pytest.mark.parametrize("S,Hq,Hkv,gists,window", [(3, 8, 2, 100, 37), (2, 4, 4, 1, 0), (5, 32, 8, 600, 128),
                                                   (1, 8, 1, 64, 64), (2, 2, 1, 700, 1)])
def test_decode_matches_oracle(S, Hq, Hkv, gists, window):
    w = synth.DecodeWorkload("t", S, gists, window, Hq, Hkv, 128, seed=300 + S)
    inp = synth.decode_inputs(w, spare_blocks=2)
    inp["k_cache"][inp["block_table"][0, -1].long(), :, (w.seq_len - 1) % PG + 1:] = float("nan")  # unused slots
    lens = [max(1, w.seq_len - 13 * i) for i in range(S)]  # ragged lengths
    o, lse, lens = run_decode(inp, lens)
    check_decode(inp, o, lse, lens, range(S))


def test_decode_of_an_empty_sequence_is_zero_not_nan():
    """A padding slot of a decode batch (length 0) attends to nothing: O = 0 and LSE = -inf there, and the
    other sequences of the batch are not disturbed."""
    w = synth.DecodeWorkload("pad", 3, 200, 30, 8, 2, 128, seed=310)
    inp = synth.decode_inputs(w, spare_blocks=1)
    o, lse, lens = run_decode(inp, [w.seq_len, 0, 77])
    assert torch.equal(o[1].float(), torch.zeros_like(o[1].float()))
    assert torch.isinf(lse[1]).all() and (lse[1] < 0).all()
    check_decode(inp, o, lse, lens, [0, 2])


def test_decode_full_size_sampled():
    w = synth.DECODE_WORKLOADS["decode_cache"]
    inp = synth.decode_inputs(w)
    o, lse, lens = run_decode(inp)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    check_decode(inp, o, lse, lens, [0, 21, 42, 63])


def test_compact_then_decode_equals_forward_row():
    """Sections 4.1 and 4.3 jointly, on the GPU path: the query of the next token over the
    compacted cache (plus its own K/V) reproduces its row of the uncompacted forward."""
    s, T, r, W, Hq, Hkv, D = 0, 512, 8, 128, 8, 2, 128
    w = synth.Workload("ext", 1, T + r, r, W, Hq, Hkv, D, seed=400)
    inp = synth.attention_inputs(w, with_grad=False)
    k_units = oracle.window_units(W, r)
    N = oracle.total_len(s, T, r)
    # prefix of T raw tokens, in shifted order
    sp, _, _ = oracle.layout(s, T, r)
    p = ug.Problem(1, T, r, W, Hq, Hkv, D)
    L = ug.unigist_compact_len(p)
    k_sh = inp["k"][:, torch.from_numpy(sp).long()].contiguous().to(DEV)
    v_sh = inp["v"][:, torch.from_numpy(sp).long()].contiguous().to(DEV)
    nb = -(-(L + 1) // PG)
    kc = torch.zeros(nb + 1, Hkv, PG, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    table = torch.arange(nb, dtype=torch.int32, device=DEV).flip(0).reshape(1, nb).contiguous()
    lens = torch.zeros(1, dtype=torch.int32, device=DEV)
    ug.unigist_kv_compact(p, k_sh, v_sh, kc, vc, table, lens)
    # append the next token (interleaved index N of the extended sequence)
    blk, slot = table[0, L // PG].item(), L % PG
    kc[blk, :, slot] = inp["k"][0, N].to(DEV)
    vc[blk, :, slot] = inp["v"][0, N].to(DEV)
    lens += 1
    q = inp["q"][:, N].contiguous().to(DEV)
    ws = torch.empty(ug.unigist_decode_workspace_bytes(1, Hq, Hkv, D, nb), dtype=torch.uint8, device=DEV)
    o = torch.empty_like(q)
    lse = torch.empty(1, Hq, dtype=torch.float32, device=DEV)
    ug.unigist_decode(q, kc, vc, table, lens, o, lse, ws)
    torch.cuda.synchronize()
    G = Hq // Hkv
    for hk in range(Hkv):
        oo, ll = oracle.attn_fwd_slice(s, T + r, r, k_units, D ** -0.5, f64(inp["q"][0, :, hk * G:(hk + 1) * G]),
                                       f64(inp["k"][0, :, hk]), f64(inp["v"][0, :, hk]), N, N + 1)
        check_close("O", f64(o[0, hk * G:(hk + 1) * G]), oo[0], TOL_O_MAX, TOL_O_MEAN)
        check_close("LSE", f64(lse[0, hk * G:(hk + 1) * G]), ll[0], TOL_LSE)
