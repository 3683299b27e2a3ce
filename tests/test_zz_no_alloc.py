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

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def both_ways(w, lens):
    d = {k: v.to(DEV) for k, v in synth.decode_inputs(w, spare_blocks=1).items()}
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
    return o, lse, o_ref, lse_ref


def test_static_decode_matches_decode_on_two_calls_in_a_row():
    # first call: many splits fill the scratch array with partial results
    w1 = synth.DecodeWorkload("a", 6, 1500, 200, 32, 8, 128, seed=901)
    o, lse, o_ref, lse_ref = both_ways(w1, [w1.seq_len - 37 * i for i in range(6)])
    assert torch.isfinite(o.float()).all()
    assert (o.float() - o_ref.float()).abs().max().item() <= 2e-2
    assert (lse - lse_ref).abs().max().item() <= 1e-3
    # second call, straight after, on a smaller and differently shaped problem: the leftovers of
    # the first call sit in the same array and must not leak into the result
    w2 = synth.DecodeWorkload("b", 3, 90, 21, 8, 2, 128, seed=902)
    o, lse, o_ref, lse_ref = both_ways(w2, [111, 64, 1])
    assert torch.isfinite(o.float()).all()
    assert (o.float() - o_ref.float()).abs().max().item() <= 2e-2
    assert (lse - lse_ref).abs().max().item() <= 1e-3


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
