"""Pins for the oracle's forward, backward and decode arithmetic (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import oracle


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def dense_masked_attention(q, k, v, mask, scale):
    """Independent dense statement with torch fp64: q [N,G,D], k,v [N,D], mask [N,N]."""
    q_, k_, v_ = (torch.from_numpy(np.ascontiguousarray(a)) for a in (q, k, v))
    sc = scale * torch.einsum("tgd,jd->gtj", q_, k_)
    sc = sc.masked_fill(torch.from_numpy(mask == 0)[None], float("-inf"))
    lse = torch.logsumexp(sc, dim=-1)
    o = torch.einsum("gtj,jd->tgd", torch.softmax(sc, dim=-1), v_)
    return o.numpy(), lse.T.numpy()


def test_full_window_equals_library_causal_attention():
    s, T, r = 2, 24, 3
    N, G, D = oracle.total_len(s, T, r), 2, 8
    q, k, v = rnd((N, G, D), 1), rnd((N, D), 2), rnd((N, D), 3)
    o, lse = oracle.attn_fwd_slice(s, T, r, T // r + 1, 0.3, q, k, v)
    qt = torch.from_numpy(q).permute(1, 0, 2)[None]            # [1,G,N,D]
    kt = torch.from_numpy(k)[None, None].expand(1, G, N, D)
    vt = torch.from_numpy(v)[None, None].expand(1, G, N, D)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=0.3)
    assert np.allclose(o, ref[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


@pytest.mark.parametrize("s,T,r,k", [(0, 56, 7, 2), (5, 64, 4, 3), (1, 6, 2, 1), (0, 20, 5, 0)])
def test_forward_matches_dense_masked_softmax(s, T, r, k):
    from test_oracle_mask_layout import literal_visible_sets
    N, G, D = oracle.total_len(s, T, r), 3, 16
    _, sets = literal_visible_sets(s, T, r, k)
    m = np.zeros((N, N), np.uint8)
    for t, vis in enumerate(sets):
        m[t, sorted(vis)] = 1
    q, kk, v = rnd((N, G, D), 4), rnd((N, D), 5), rnd((N, D), 6)
    o, lse = oracle.attn_fwd_slice(s, T, r, k, 0.25, q, kk, v)
    o2, lse2 = dense_masked_attention(q, kk, v, m, 0.25)
    assert np.allclose(o, o2, rtol=0, atol=1e-12)
    assert np.allclose(lse, lse2, rtol=0, atol=1e-12)


def test_zero_query_gives_log_count_and_mean_of_visible_values():
    s, T, r, k = 3, 40, 4, 2
    N, G, D = oracle.total_len(s, T, r), 2, 8
    kk, v = rnd((N, D), 7), rnd((N, D), 8)
    o, lse = oracle.attn_fwd_slice(s, T, r, k, 1.0, np.zeros((N, G, D)), kk, v)
    m = oracle.mask(s, T, r, k).astype(np.float64)
    cnt = m.sum(1)
    assert np.allclose(lse, np.log(cnt)[:, None], rtol=0, atol=1e-13)
    assert np.allclose(o, ((m @ v) / cnt[:, None])[:, None, :].repeat(G, 1), rtol=0, atol=1e-13)


def test_constant_values_are_reproduced_rows_sum_to_one():
    s, T, r, k = 0, 56, 7, 2
    N, G, D = oracle.total_len(s, T, r), 2, 8
    q, kk = rnd((N, G, D), 9), rnd((N, D), 10)
    row = rnd((D,), 11)
    o, _ = oracle.attn_fwd_slice(s, T, r, k, 0.5, q, kk, np.tile(row, (N, 1)))
    assert np.allclose(o, row[None, None], rtol=0, atol=1e-13)


def test_key_shift_moves_lse_only():
    s, T, r, k = 2, 30, 5, 1
    N, G, D = oracle.total_len(s, T, r), 2, 8
    q, kk, v, c = rnd((N, G, D), 12), rnd((N, D), 13), rnd((N, D), 14), rnd((D,), 15)
    o1, l1 = oracle.attn_fwd_slice(s, T, r, k, 0.4, q, kk, v)
    o2, l2 = oracle.attn_fwd_slice(s, T, r, k, 0.4, q, kk + c, v)
    assert np.allclose(o1, o2, rtol=0, atol=1e-12)
    assert np.allclose(l2 - l1, 0.4 * (q @ c), rtol=0, atol=1e-12)


def test_row_range_and_whole_problem_wrappers_agree():
    s, T, r, k = 1, 24, 4, 1
    N, Hq, Hkv, D = oracle.total_len(s, T, r), 4, 2, 8
    q, kk, v = rnd((2, N, Hq, D), 16), rnd((2, N, Hkv, D), 17), rnd((2, N, Hkv, D), 18)
    o, lse = oracle.attn_fwd(s, T, r, k, 0.35, q, kk, v)
    # q head 3 of batch 1 uses kv head 1
    o_s, l_s = oracle.attn_fwd_slice(s, T, r, k, 0.35, q[1, :, 2:4], kk[1, :, 1], v[1, :, 1], 5, 9)
    assert np.array_equal(o[1, 5:9, 2:4], o_s)
    assert np.array_equal(lse[1, 2:4, 5:9], l_s.T)


def test_shifted_layout_agrees_after_inverse_permutation():
    """Section 4.2: attention on the gist-shifted sequence, with the mask evaluated from the
    original token indexes, equals attention on the interleaved sequence."""
    s, T, r, k = 2, 36, 4, 2
    N, G, D = oracle.total_len(s, T, r), 2, 8
    q, kk, v = rnd((N, G, D), 19), rnd((N, D), 20), rnd((N, D), 21)
    o, lse = oracle.attn_fwd_slice(s, T, r, k, 0.3, q, kk, v)
    sp, up, _ = oracle.layout(s, T, r)
    m = oracle.mask(s, T, r, k)
    m_shift = m[np.ix_(sp, sp)]  # mask through the original indexes
    assert not (m_shift == np.tril(np.ones_like(m))).all()
    o_s, lse_s = dense_masked_attention(q[sp], kk[sp], v[sp], m_shift, 0.3)
    assert np.allclose(o_s[up], o, rtol=0, atol=1e-12)
    assert np.allclose(lse_s[up], lse, rtol=0, atol=1e-12)


def loss(s, T, r, k, scale, q, kk, v, dout):
    o, _ = oracle.attn_fwd_slice(s, T, r, k, scale, q, kk, v)
    return float((o * dout).sum())


@pytest.mark.parametrize("s,T,r,k", [(1, 6, 2, 1), (0, 12, 3, 1), (2, 8, 4, 0)])
def test_backward_matches_central_finite_differences(s, T, r, k):
    N, G, D, scale, h = oracle.total_len(s, T, r), 2, 4, 0.6, 1e-5
    q, kk, v, dout = rnd((N, G, D), 22), rnd((N, D), 23), rnd((N, D), 24), rnd((N, G, D), 25)
    dq, dk, dv = oracle.attn_bwd_slice(s, T, r, k, scale, q, kk, v, dout)
    for name, arr, grad in (("q", q, dq), ("k", kk, dk), ("v", v, dv)):
        num = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = arr[idx]
            arr[idx] = old + h
            lp = loss(s, T, r, k, scale, q, kk, v, dout)
            arr[idx] = old - h
            lm = loss(s, T, r, k, scale, q, kk, v, dout)
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        err = np.abs(num - grad).max() / max(1.0, np.abs(grad).max())
        assert err < 1e-7, (name, err)


def test_backward_full_window_matches_autograd_of_dense_causal():
    s, T, r = 1, 20, 4
    N, G, D, scale = oracle.total_len(s, T, r), 2, 8, 0.3
    q, kk, v, dout = rnd((N, G, D), 26), rnd((N, D), 27), rnd((N, D), 28), rnd((N, G, D), 29)
    dq, dk, dv = oracle.attn_bwd_slice(s, T, r, T // r, scale, q, kk, v, dout)
    qt, kt, vt = (torch.tensor(a, requires_grad=True) for a in (q, kk, v))
    sc = scale * torch.einsum("tgd,jd->gtj", qt, kt)
    sc = sc.masked_fill(~torch.tril(torch.ones(N, N, dtype=torch.bool))[None], float("-inf"))
    o = torch.einsum("gtj,jd->tgd", torch.softmax(sc, -1), vt)
    (o * torch.from_numpy(dout)).sum().backward()
    assert np.allclose(dq, qt.grad.numpy(), rtol=0, atol=1e-12)
    assert np.allclose(dk, kt.grad.numpy(), rtol=0, atol=1e-12)
    assert np.allclose(dv, vt.grad.numpy(), rtol=0, atol=1e-12)


def test_backward_invariants_and_gqa_sum():
    s, T, r, k = 0, 28, 7, 1
    N, G, D, scale = oracle.total_len(s, T, r), 3, 8, 0.5
    q, kk, v, dout = rnd((N, G, D), 30), rnd((N, D), 31), rnd((N, D), 32), rnd((N, G, D), 33)
    dq, dk, dv = oracle.attn_bwd_slice(s, T, r, k, scale, q, kk, v, dout)
    # each row of dS sums to zero => the key gradients sum to zero over keys
    assert np.abs(dk.sum(0)).max() < 1e-12
    # softmax rows sum to one => sum_j dV_j = sum over rows and heads of dO
    assert np.allclose(dv.sum(0), dout.sum((0, 1)), rtol=0, atol=1e-12)
    # dK, dV of a KV head are the sums over its query heads
    parts = [oracle.attn_bwd_slice(s, T, r, k, scale, q[:, g:g + 1], kk, v, dout[:, g:g + 1])
             for g in range(G)]
    assert np.allclose(dk, sum(p[1] for p in parts), rtol=0, atol=1e-12)
    assert np.allclose(dv, sum(p[2] for p in parts), rtol=0, atol=1e-12)
    assert np.allclose(dq, np.concatenate([p[0] for p in parts], 1), rtol=0, atol=1e-12)


def test_decode_over_compacted_cache_equals_row_of_full_forward():
    """Sections 4.1 and 4.3 jointly: the next token after a T-token prefix, attending to the
    compacted cache plus itself, gets the same output as its row in the uncompacted forward."""
    s, T, r, k = 2, 24, 4, 2
    G, D, scale = 2, 8, 0.4
    T_ext = T + r
    N, N_ext = oracle.total_len(s, T, r), oracle.total_len(s, T_ext, r)
    q, kk, v = rnd((N_ext, G, D), 34), rnd((N_ext, D), 35), rnd((N_ext, D), 36)
    o_full, lse_full = oracle.attn_fwd_slice(s, T_ext, r, k, scale, q, kk, v, N, N + 1)
    kept = oracle.kept_set(s, T, r, k)
    idx = np.concatenate([kept, [N]])  # the new token's own K/V is appended before decoding
    o_d, lse_d = oracle.decode_slice(scale, q[N], kk[idx], v[idx])
    assert np.allclose(o_d, o_full[0], rtol=0, atol=1e-12)
    assert np.allclose(lse_d, lse_full[0], rtol=0, atol=1e-12)


def test_decode_matches_library_softmax():
    L, G, D = 37, 4, 16
    qd, kc, vc = rnd((G, D), 37), rnd((L, D), 38), rnd((L, D), 39)
    o, lse = oracle.decode_slice(0.2, qd, kc, vc)
    sc = 0.2 * torch.from_numpy(qd) @ torch.from_numpy(kc).T
    assert np.allclose(o, (torch.softmax(sc, -1) @ torch.from_numpy(vc)).numpy(), atol=1e-13, rtol=0)
    assert np.allclose(lse, torch.logsumexp(sc, -1).numpy(), atol=1e-13, rtol=0)


def test_sampled_backward_equals_full_backward():
    s, T, r, k = 1, 32, 4, 2
    N, G, D, scale = oracle.total_len(s, T, r), 2, 8, 0.45
    q, kk, v, dout = rnd((N, G, D), 40), rnd((N, D), 41), rnd((N, D), 42), rnd((N, G, D), 43)
    dq, dk, dv = oracle.attn_bwd_slice(s, T, r, k, scale, q, kk, v, dout)
    rows, keys = [0, 7, 19, N - 1], [2, 9, 10, N - 2]
    dq_s, dk_s, dv_s = oracle.attn_bwd_sample(s, T, r, k, scale, q, kk, v, dout, rows, keys)
    assert np.array_equal(dq_s, dq[rows]) and np.array_equal(dk_s, dk[keys]) and np.array_equal(dv_s, dv[keys])
