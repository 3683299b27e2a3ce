"""GPU parity of the decoding loop (Section 4.3): the compressed cache is grown token by token with
unigist_cache_append -- raw tokens leave it at compression points, nothing moves -- and after every
append it must hold exactly the tokens the new query sees, so that unigist_decode over it equals the row
of the oracle's forward over the whole sequence."""
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
    # B, s, T, r, W, Hq, Hkv, units prefilled before decoding starts
    (2, 4, 96, 8, 16, 4, 2, 3),
    (1, 0, 64, 4, 0, 2, 1, 0),        # no window: every unit's raw tokens go as soon as its gist arrives
    (1, 3, 40, 1, 3, 2, 2, 5),        # ratio 1
    (2, 0, 120, 8, 1000, 8, 2, 2),    # the window never fills: nothing is ever evicted
    (1, 130, 70, 7, 15, 4, 4, 1),     # sinks over two pages, window of ceil(15 / 7) = 3 units
]


def _random_loop_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        r = int(rng.choice([1, 2, 3, 4, 8, 16]))
        n = int(rng.integers(2, 160 // (r + 1) + 2))
        Hkv = int(rng.choice([1, 2]))
        out.append((int(rng.choice([1, 2])), int(rng.choice([0, 0, 2, 65])), n * r, r, int(rng.choice([0, r, 2 * r + 1, 40, 10 ** 6])),
                    Hkv * int(rng.choice([1, 2, 4])), Hkv, int(rng.integers(0, n))))
    return out


CASES += _random_loop_cases(6, 9)
CASES = [c + (0.0,) for c in CASES] + [(2, 2, 64, 4, 8, 4, 2, 2, 0.05)]  # the last: a caller-given softmax scale


def read_cache(cache, table_row, length):
    blocks = cache[table_row[: -(-length // PG)].long()]
    return blocks.permute(0, 2, 1, 3).reshape(-1, cache.shape[1], cache.shape[3])[:length]


@pytest.mark.parametrize("B,s,T,r,W,Hq,Hkv,units0,given_scale", CASES)
def test_decode_loop_matches_the_one_pass_forward(B, s, T, r, W, Hq, Hkv, units0, given_scale):
    D = 128
    w = synth.Workload("loop", B, T, r, W, Hq, Hkv, D, num_sinks=s, seed=777 + T + r)
    inp = synth.attention_inputs(w, with_grad=False)
    k_units = oracle.window_units(W, r)
    scale = given_scale or D ** -0.5
    o_ref, lse_ref = oracle.attn_fwd(s, T, r, k_units, scale, *(f64(inp[n]) for n in ("q", "k", "v")))
    p = ug.Problem(B, T, r, W, Hq, Hkv, D, num_sinks=s, softmax_scale=given_scale)
    n = T // r
    per_seq = -(-(s + n + (k_units + 1) * r + 1) // PG)
    nblocks = B * per_seq + 1
    g = torch.Generator().manual_seed(3)
    table = torch.randperm(nblocks, generator=g)[: B * per_seq].to(torch.int32).reshape(B, per_seq)
    kc = torch.zeros(nblocks, Hkv, PG, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    table_d = table.to(DEV)
    lens = torch.zeros(B, dtype=torch.int32, device=DEV)
    # the prefix: sinks and units0 whole units, compacted into the cache (interleaved tensors handed over)
    n0 = s + units0 * (r + 1)
    if n0 > 0 and units0 > 0:
        pp = ug.Problem(B, units0 * r, r, W, Hq, Hkv, D, num_sinks=s, flags=ug.FLAG_INTERLEAVED)
        ug.unigist_kv_compact(pp, inp["k"][:, :n0].contiguous().to(DEV), inp["v"][:, :n0].contiguous().to(DEV), kc, vc,
                              table_d, lens)
    state = torch.zeros(ug.unigist_cache_state_bytes(p) // 4, dtype=torch.int32, device=DEV)
    ug.unigist_cache_state_init(p, units0, state)
    if units0 == 0:  # the sinks are appended like any other token before the first unit starts
        n0 = 0
    wsd = torch.empty(ug.unigist_decode_workspace_bytes(B, Hq, Hkv, D, per_seq), dtype=torch.uint8, device=DEV)
    od = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=DEV)
    lsed = torch.empty(B, Hq, dtype=torch.float32, device=DEV)
    kd, vd, qd = inp["k"].to(DEV), inp["v"].to(DEV), inp["q"].to(DEV)
    N = w.total_len
    ints = 8 + (k_units + 1) * r + r  # per-sequence state: 8 header ints, the window ring, the free list
    for t in range(n0, N):
        if t < s:   # a sink of a sequence that starts empty: plain append at the end
            is_gist = None
        else:
            is_gist = (t - s) % (r + 1) == r
        if is_gist is None:
            # sinks are not part of any unit: write them where compaction would (positions 0 .. s-1)
            pos = t
            blk = table_d[:, pos // PG].long()
            kc[blk, :, pos % PG] = kd[:, t]
            vc[blk, :, pos % PG] = vd[:, t]
            lens += 1
        else:
            ug.unigist_cache_append(p, kd[:, t].contiguous(), vd[:, t].contiguous(), is_gist, kc, vc, table_d, lens, state)
        ug.unigist_decode_step(p, qd[:, t].contiguous(), kc, vc, table_d, lens, state, od, lsed, wsd)
        torch.cuda.synchronize()
        assert state[: B * ints].view(B, ints)[:, 4].abs().sum().item() == 0
        check_close(f"decode O at token {t}", f64(od), o_ref[:, t], TOL_O_MAX, TOL_O_MEAN)
        check_close(f"decode LSE at token {t}", f64(lsed), lse_ref[:, :, t], TOL_LSE)
        if t % 7 == 0 or t == N - 1:  # the cache holds exactly what token t sees (as a set: its order is free)
            vis = np.nonzero(oracle.mask(s, T, r, k_units, t, t + 1)[0])[0]
            L = lens.cpu().tolist()
            st_host = state[: B * ints].view(B, ints).cpu()
            free_off = 8 + (k_units + 1) * r
            for b in range(B):
                holes = set(st_host[b, free_off: free_off + int(st_host[b, 2])].tolist())
                live = [i for i in range(L[b]) if i not in holes]
                assert len(live) == len(vis)
                got = read_cache(kc.cpu(), table[b], L[b])[live].reshape(len(live), -1).view(torch.int16)
                want = inp["k"][b, torch.from_numpy(vis).long()].reshape(len(vis), -1).view(torch.int16)
                assert sorted(map(tuple, got[:, :4].tolist())) == sorted(map(tuple, want[:, :4].tolist()))


def test_append_flags_misuse_and_leaves_the_cache_alone():
    B, r, D, Hkv = 1, 4, 128, 1
    p = ug.Problem(B, 8, r, 4, 1, Hkv, D)
    kc = torch.zeros(2, Hkv, PG, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    table = torch.arange(2, dtype=torch.int32, device=DEV).reshape(1, 2)
    lens = torch.zeros(B, dtype=torch.int32, device=DEV)
    state = torch.zeros(ug.unigist_cache_state_bytes(p) // 4, dtype=torch.int32, device=DEV)
    ug.unigist_cache_state_init(p, 0, state)
    x = torch.ones(B, Hkv, D, dtype=torch.bfloat16, device=DEV)
    ug.unigist_cache_append(p, x, x, True, kc, vc, table, lens, state)   # a gist with no raw token before it
    torch.cuda.synchronize()
    assert state[4].item() == 2 and lens.item() == 0 and kc.abs().sum().item() == 0
