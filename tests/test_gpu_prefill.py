"""GPU parity of chunk-wise prefill (Section 4.3): chunks of gist units are encoded against the compressed
paged cache; every chunk's outputs must equal the rows of the oracle's one-pass forward over the whole
prompt, and after every chunk the cache must hold exactly the oracle's kept set of the prefix."""
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

CASES = [
    # B, s, T, r, W, Hq, Hkv, D, chunk sizes in gist units
    (1, 0, 1024, 8, 128, 4, 2, 128, [32, 32, 64]),
    (2, 128, 1024, 8, 128, 2, 2, 128, [16, 48, 64]),     # the paper's default sinks and window
    (1, 5, 330, 5, 48, 2, 1, 64, [7, 20, 39]),           # ragged everything, head_dim 64
    (1, 0, 2048, 16, 4096, 2, 1, 128, [64, 64]),         # the window covers the whole prompt
    (1, 3, 640, 4, 0, 2, 2, 128, [100, 60]),             # no window: gists and sinks only
    (1, 0, 512, 8, 64, 2, 1, 128, [64]),                 # one chunk = the whole prompt
]
def _random_prefill_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        r = int(rng.choice([1, 2, 4, 5, 8, 16, 32]))
        n = int(rng.integers(2, 1200 // (r + 1) + 1))
        s = int(rng.choice([0, 0, 3, 64, 130]))
        W = int(rng.choice([0, r, 3 * r, 100, 10 ** 6]))
        cuts = sorted(set(rng.integers(1, n, size=int(rng.integers(0, 5))).tolist()))
        chunks = [b - a for a, b in zip([0] + cuts, cuts + [n])]
        Hkv = int(rng.choice([1, 2]))
        out.append((int(rng.choice([1, 2])), s, n * r, r, W, Hkv * int(rng.choice([1, 2, 4])), Hkv,
                    int(rng.choice([64, 128])), chunks))
    return out


CASES += _random_prefill_cases(10, 3)
CASES = [c + (0.0,) for c in CASES] + [
    # a caller-given softmax scale instead of 1 / sqrt(head_dim)
    (2, 4, 768, 8, 64, 4, 2, 128, [24, 40, 32], 0.05),
    (1, 0, 330, 5, 48, 2, 1, 64, [30, 36], 0.3),
]


def read_cache(cache, table_row, length):
    blocks = cache[table_row[: -(-length // PG)].long()]           # [nb, Hkv, PG, D]
    return blocks.permute(0, 2, 1, 3).reshape(-1, cache.shape[1], cache.shape[3])[:length]


@pytest.mark.parametrize("B,s,T,r,W,Hq,Hkv,D,chunks,given_scale", CASES)
def test_chunked_prefill_matches_the_one_pass_forward(B, s, T, r, W, Hq, Hkv, D, chunks, given_scale):
    assert sum(chunks) == T // r
    w = synth.Workload("prefill", B, T, r, W, Hq, Hkv, D, num_sinks=s, seed=4242 + T + r)
    inp = synth.attention_inputs(w, with_grad=False)
    k_units = oracle.window_units(W, r)
    scale = given_scale or D ** -0.5
    o_ref, lse_ref = oracle.attn_fwd(s, T, r, k_units, scale, *(f64(inp[n]) for n in ("q", "k", "v")))
    p = ug.Problem(B, T, r, W, Hq, Hkv, D, num_sinks=s, softmax_scale=given_scale)
    L_max = s + T // r + min(k_units, T // r) * r
    per_seq = -(-L_max // PG)
    nblocks = B * per_seq + 2
    g = torch.Generator().manual_seed(7)
    table = torch.randperm(nblocks, generator=g)[: B * per_seq].to(torch.int32).reshape(B, per_seq)
    kc = torch.zeros(nblocks, Hkv, PG, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    table_d = table.to(DEV)
    lens = torch.zeros(B, dtype=torch.int32, device=DEV)
    u0 = 0
    for c in chunks:
        # the chunk's tokens: interleaved indices, listed in shifted chunk order [sinks | raw | gists]
        raw_idx = [s + u * (r + 1) + t for u in range(u0, u0 + c) for t in range(r)]
        gist_idx = [s + u * (r + 1) + r for u in range(u0, u0 + c)]
        idx = torch.tensor((list(range(s)) if u0 == 0 else []) + raw_idx + gist_idx)
        qc, kk, vv = (inp[n][:, idx].contiguous().to(DEV) for n in ("q", "k", "v"))
        o = torch.full_like(qc, float("nan"))
        lse = torch.full((B, Hq, len(idx)), float("nan"), dtype=torch.float32, device=DEV)
        ws = torch.empty(max(16, ug.unigist_prefill_workspace_bytes(p, u0, c)), dtype=torch.uint8, device=DEV)
        ug.unigist_prefill_chunk(p, u0, c, qc, kk, vv, kc, vc, table_d, lens, o, lse, ws)
        ug.unigist_device_status()
        check_close(f"O of units [{u0}, {u0 + c})", f64(o), o_ref[:, idx.numpy()], TOL_O_MAX, TOL_O_MEAN)
        check_close(f"LSE of units [{u0}, {u0 + c})", f64(lse), lse_ref[:, :, idx.numpy()], TOL_LSE)
        # the cache now holds the compressed prefix: bit for bit the oracle's kept set, in cache order
        u0 += c
        kept = oracle.kept_set(s, u0 * r, r, min(k_units, u0))
        assert lens.cpu().tolist() == [len(kept)] * B
        for b in range(B):
            for cache, src in ((kc, inp["k"]), (vc, inp["v"])):
                got = read_cache(cache.cpu(), table[b], len(kept))
                assert torch.equal(got, src[b, torch.from_numpy(kept).long()])
    if D != 128:
        return
    # and a decode step over the cache the prefill left behind
    qd = torch.randn(B, Hq, D, generator=g).to(torch.bfloat16)
    od = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=DEV)
    wsd = torch.empty(ug.unigist_decode_workspace_bytes(B, Hq, Hkv, D, per_seq), dtype=torch.uint8, device=DEV)
    ug.unigist_decode(qd.to(DEV), kc, vc, table_d, lens, od, None, wsd, softmax_scale=given_scale)
    kept = torch.from_numpy(oracle.kept_set(s, T, r, min(k_units, T // r))).long()
    od_ref, _ = oracle.decode(scale, f64(qd), [f64(inp["k"][b, kept]) for b in range(B)],
                              [f64(inp["v"][b, kept]) for b in range(B)])
    check_close("decode after prefill", f64(od), od_ref, TOL_O_MAX, TOL_O_MEAN)


def test_prefill_rejects_chunks_outside_the_prompt():
    p = ug.Problem(1, 64, 8, 16, 1, 1, 128)
    assert ug.unigist_prefill_workspace_bytes(p, 6, 4) == 0   # 8 units in all
    assert ug.unigist_prefill_workspace_bytes(p, 0, 0) == 0
    assert ug.unigist_prefill_workspace_bytes(p, 2, 6) > 0
