"""The allocation-free decode entry point against the ordinary one.

`unigist_decode_static` serves callers that cannot supply scratch memory and are not allowed to
allocate (for example code running inside a server that owns the whole GPU memory pool).  It must
give the same answer as `unigist_decode`, also when it is called twice in a row on different
problems, because both calls share one built-in scratch array that keeps the previous contents.
This file sorts last on purpose: a failure here cannot hide the result of any other test.
"""
import pytest
import torch

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import synth
from oracle import oracle

from gpu_util import TOL_LSE, TOL_O_MAX, TOL_O_MEAN, check_close, f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PG = ug.PAGE_TOKENS


def against_oracle(inp, lens, o, lse):
    """The fp64 definition (softmax attention of the query over the sequence's cache entries)."""
    D = inp["q"].shape[2]
    for i, n in enumerate(lens):
        blocks = inp["block_table"][i, : -(-n // PG)].long()
        view = lambda c: c[blocks].permute(0, 2, 1, 3).reshape(-1, c.shape[1], c.shape[3])[:n]
        oo, ll = oracle.decode(D ** -0.5, f64(inp["q"][i:i + 1]), [f64(view(inp["k_cache"]))], [f64(view(inp["v_cache"]))])
        check_close(f"static decode O seq {i}", f64(o[i:i + 1]), oo, TOL_O_MAX, TOL_O_MEAN)
        check_close(f"static decode LSE seq {i}", f64(lse[i:i + 1]), ll, TOL_LSE)


def both_ways(w, lens):
    inp = synth.decode_inputs(w, spare_blocks=1)
    d = {k: v.to(DEV) for k, v in inp.items()}
    d["seq_lens"] = torch.tensor(lens, dtype=torch.int32, device=DEV)
    S, Hq, D = d["q"].shape
    nbytes = ug.unigist_decode_workspace_bytes(S, Hq, w.num_kv_heads, D, d["block_table"].shape[1])
    assert nbytes <= ug.DECODE_STATIC_SCRATCH_BYTES
    ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    o_ref = torch.full_like(d["q"], float("nan"))
    lse_ref = torch.full((S, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ug.unigist_decode(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o_ref, lse_ref, ws)
    o = torch.full_like(d["q"], float("nan"))
    lse = torch.full((S, Hq), float("nan"), dtype=torch.float32, device=DEV)
    ug.unigist_decode_static(d["q"], d["k_cache"], d["v_cache"], d["block_table"], d["seq_lens"], o, lse)
    torch.cuda.synchronize()
    against_oracle(inp, lens, o, lse)
    return o, lse, o_ref, lse_ref


def test_static_decode_matches_decode_on_two_calls_in_a_row():
    # first call: many splits fill the scratch array with partial results
    w1 = synth.DecodeWorkload("a", 6, 1500, 200, 32, 8, 128, seed=901)
    o, lse, o_ref, lse_ref = both_ways(w1, [w1.seq_len - 37 * i for i in range(6)])
    # both entry points run the same kernels with the same split count: not one bit may differ, so
    # stale partial results leaking out of the shared array cannot hide inside a tolerance
    assert torch.isfinite(o.float()).all()
    assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)
    # second call, straight after, on a smaller and differently shaped problem: the leftovers of
    # the first call sit in the same array and must not leak into the result
    w2 = synth.DecodeWorkload("b", 3, 90, 21, 8, 2, 128, seed=902)
    o, lse, o_ref, lse_ref = both_ways(w2, [111, 64, 1])
    assert torch.isfinite(o.float()).all()
    assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)
    # a group size that is not a power of two: accepted here exactly as by unigist_decode
    w3 = synth.DecodeWorkload("c", 2, 130, 9, 6, 2, 128, seed=904)
    o, lse, o_ref, lse_ref = both_ways(w3, [139, 70])
    assert torch.equal(o, o_ref) and torch.equal(lse, lse_ref)


def test_static_decode_rejects_problems_larger_than_its_scratch():
    w = synth.DecodeWorkload("big", 2, 64, 0, 8, 2, 128, seed=903)
    d = {k: v.to(DEV) for k, v in synth.decode_inputs(w).items()}
    S = 4096  # claims far more sequences than the built-in array can hold partials for
    assert ug.unigist_decode_workspace_bytes(S, 32, 8, 128, 4096) > ug.DECODE_STATIC_SCRATCH_BYTES
    before = ug.unigist_launch_count()
    rc = ug.binding.lib().unigist_decode_static(S, 32, 8, 128, 0.0, d["q"].data_ptr(), d["k_cache"].data_ptr(),
                                                d["v_cache"].data_ptr(), d["k_cache"].shape[0],
                                                d["block_table"].data_ptr(), 4096, d["seq_lens"].data_ptr(),
                                                d["q"].data_ptr(), None, None)
    assert rc == 4  # UNIGIST_ERR_WORKSPACE
    assert "built-in array" in ug.unigist_last_error_string()
    assert ug.unigist_launch_count() == before
