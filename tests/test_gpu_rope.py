"""Rotary embedding with aligned position ids (Section 4.1, step 3), alone and fused with the gist shift."""
import numpy as np
import pytest
import torch

import paper_2509_15763_b200 as ug
from oracle import oracle

pytestmark = pytest.mark.gpu

CASES = [
    # s, T, r, heads, D, B, theta
    (0, 64, 4, 8, 128, 2, 500000.0),
    (5, 96, 8, 3, 128, 1, 10000.0),   # odd head count: the last pass of a warp is ragged
    (128, 1024, 4, 2, 128, 1, 500000.0),
    (3, 120, 3, 5, 64, 2, 10000.0),
    (0, 7, 7, 1, 64, 1, 10000.0),     # a single unit
]


def _run(s, T, r, H, D, B, theta, flags, in_place=False):
    p = ug.Problem(batch=B, raw_len=T, num_sinks=s, ratio=r, window=r, num_q_heads=H, num_kv_heads=H, head_dim=D)
    N = ug.unigist_total_len(p)
    g = torch.Generator().manual_seed(1234 + T + H)
    x = torch.randn(B, N, H, D, generator=g).to(torch.bfloat16)
    xd = x.cuda()
    yd = xd if in_place else torch.empty_like(xd)
    ug.unigist_rope(p, xd, yd, theta, flags)
    torch.cuda.synchronize()
    return x, yd.cpu(), N


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("shifted", [False, True])
def test_rope_matches_oracle(case, shifted):
    s, T, r, H, D, B, theta = case
    x, y, N = _run(*case, flags=ug.ROPE_TO_SHIFTED if shifted else 0)
    sp, up, pos = oracle.layout(s, T, r)
    for b in range(B):
        want = oracle.rope(x[b].double().numpy(), pos, theta)
        if shifted:
            want = want[sp]
        got = y[b].double().numpy()
        # one bf16 rounding of a value of magnitude <= |x| sqrt(2): 2^-9 relative, plus the fp32 rotation
        tol = 2.0 ** -8 * np.maximum(np.abs(want), 1e-2) + 1e-6
        assert (np.abs(got - want) <= tol).all(), float(np.abs(got - want).max())


def test_rope_in_place():
    case = (2, 48, 4, 4, 128, 1, 10000.0)
    x, y0, _ = _run(*case, flags=0)
    _, y1, _ = _run(*case, flags=0, in_place=True)
    assert torch.equal(y0, y1)


def test_rope_rejects_overlap_with_shift():
    p = ug.Problem(batch=1, raw_len=16, num_sinks=0, ratio=4, window=4, num_q_heads=1, num_kv_heads=1, head_dim=128)
    x = torch.zeros(1, ug.unigist_total_len(p), 1, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ug.UnigistError):
        ug.unigist_rope(p, x, x, 10000.0, ug.ROPE_TO_SHIFTED)
