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


def test_rope_inverse_and_shifted_source():
    """The inverse flag is the transposed rotation (what a backward pass applies); a shifted source gives
    the same rows as an interleaved one."""
    s, T, r, H, D, B, theta = 3, 120, 4, 2, 128, 1, 500000.0
    p = ug.Problem(batch=B, raw_len=T, num_sinks=s, ratio=r, window=r, num_q_heads=H, num_kv_heads=H, head_dim=D)
    N = ug.unigist_total_len(p)
    g = torch.Generator().manual_seed(9)
    x = torch.randn(B, N, H, D, generator=g).to(torch.bfloat16)
    dy = torch.randn(B, N, H, D, generator=g).to(torch.bfloat16)
    sp, up, pos = oracle.layout(s, T, r)
    xd, dyd = x.cuda(), dy.cuda()
    # the transposed rotation against the oracle rotating by the negated ids
    dx = torch.empty_like(dyd)
    ug.unigist_rope(p, dyd, dx, theta, ug.ROPE_INVERSE)
    want = oracle.rope(dy[0].double().numpy(), -pos.astype(np.int64), theta)
    got = dx[0].cpu().double().numpy()
    assert (np.abs(got - want) <= 2.0 ** -8 * np.maximum(np.abs(want), 1e-2) + 1e-6).all()
    # <R x, dy> = <x, R^T dy> up to the bf16 rounding of the two results
    y = torch.empty_like(xd)
    ug.unigist_rope(p, xd, y, theta, 0)
    lhs = (y.double() * dyd.double()).sum().item()
    rhs = (xd.double() * dx.double()).sum().item()
    assert abs(lhs - rhs) <= 2e-3 * (y.double().abs() * dyd.double().abs()).sum().item() ** 0.5 + 1e-2 * abs(lhs)
    # shifted in, interleaved out (fused unshift), and shifted in, shifted out: the same rows as from interleaved input
    xs = xd[:, torch.from_numpy(sp.astype(np.int64)).cuda()].contiguous()
    a = torch.empty_like(xd)
    ug.unigist_rope(p, xs, a, theta, ug.ROPE_FROM_SHIFTED)
    assert torch.equal(a, y)
    b = torch.empty_like(xd)
    ug.unigist_rope(p, xs, b, theta, ug.ROPE_FROM_SHIFTED | ug.ROPE_TO_SHIFTED)
    assert torch.equal(b, y[:, torch.from_numpy(sp.astype(np.int64)).cuda()])
    ug.unigist_rope(p, xs, xs, theta, ug.ROPE_FROM_SHIFTED | ug.ROPE_TO_SHIFTED)  # in place: the order does not change
    assert torch.equal(xs, b)
