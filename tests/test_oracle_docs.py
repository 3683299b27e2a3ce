"""Pins of the oracle's cross-document masking (Section 5.1): a packed sample is a set of independent
sequences.  The dense docs_* functions are checked against the single-sequence oracle (a separate
implementation, in C), against brute-force counting, and for independence between documents."""
import numpy as np

from oracle import oracle


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _bases(s, doc_T, r):
    b, out = 0, []
    for T in doc_T:
        out.append(b)
        b += oracle.total_len(s, T, r)
    return out, b


def test_mask_is_block_diagonal_of_eq3_masks():
    s, r, k, doc_T = 1, 2, 1, [4, 2, 6]
    m = oracle.docs_mask(s, doc_T, r, k)
    bases, n_tot = _bases(s, doc_T, r)
    assert m.shape == (n_tot, n_tot)
    cover = np.zeros_like(m)
    for b, T in zip(bases, doc_T):
        n = oracle.total_len(s, T, r)
        assert (m[b:b + n, b:b + n] == oracle.mask(s, T, r, k)).all()
        cover[b:b + n, b:b + n] = True
    assert not m[~cover].any()  # nothing crosses a boundary
    assert m.sum() == sum(oracle.count_pairs(s, T, r, k) for T in doc_T)


def test_forward_equals_each_document_alone():
    s, r, k, doc_T, Hq, Hkv, D = 2, 4, 2, [8, 16, 4], 4, 2, 8
    bases, n_tot = _bases(s, doc_T, r)
    q, kk, v = _rand((n_tot, Hq, D), 1), _rand((n_tot, Hkv, D), 2), _rand((n_tot, Hkv, D), 3)
    o, lse = oracle.docs_attn_fwd(s, doc_T, r, k, 0.3, q, kk, v)
    for b, T in zip(bases, doc_T):
        n = oracle.total_len(s, T, r)
        o1, l1 = oracle.attn_fwd(s, T, r, k, 0.3, q[None, b:b + n], kk[None, b:b + n], v[None, b:b + n])
        assert np.allclose(o[b:b + n], o1[0], atol=1e-12)
        assert np.allclose(lse[:, b:b + n], l1[0], atol=1e-12)


def test_backward_equals_each_document_alone_and_finite_differences():
    s, r, k, doc_T, Hq, Hkv, D = 1, 2, 1, [4, 6], 2, 1, 4
    bases, n_tot = _bases(s, doc_T, r)
    q, kk, v = _rand((n_tot, Hq, D), 4), _rand((n_tot, Hkv, D), 5), _rand((n_tot, Hkv, D), 6)
    do = _rand((n_tot, Hq, D), 7)
    dq, dk, dv = oracle.docs_attn_bwd(s, doc_T, r, k, 0.5, q, kk, v, do)
    for b, T in zip(bases, doc_T):
        n = oracle.total_len(s, T, r)
        a, c, d = oracle.attn_bwd(s, T, r, k, 0.5, q[None, b:b + n], kk[None, b:b + n], v[None, b:b + n],
                                  do[None, b:b + n])
        assert np.allclose(dq[b:b + n], a[0], atol=1e-11)
        assert np.allclose(dk[b:b + n], c[0], atol=1e-11)
        assert np.allclose(dv[b:b + n], d[0], atol=1e-11)

    def loss(q_, k_, v_):
        return (oracle.docs_attn_fwd(s, doc_T, r, k, 0.5, q_, k_, v_)[0] * do).sum()

    eps = 1e-6
    rng = np.random.default_rng(8)
    for arr, grad, which in ((q, dq, 0), (kk, dk, 1), (v, dv, 2)):
        for _ in range(4):
            idx = tuple(rng.integers(0, n) for n in arr.shape)
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps
            lo[idx] -= eps
            args_hi = [q, kk, v]
            args_lo = [q, kk, v]
            args_hi[which], args_lo[which] = hi, lo
            fd = (loss(*args_hi) - loss(*args_lo)) / (2 * eps)
            assert abs(fd - grad[idx]) < 1e-6 * max(1.0, abs(fd))


def test_documents_do_not_influence_each_other():
    s, r, k, doc_T, H, D = 0, 2, 1, [4, 4], 1, 4
    bases, n_tot = _bases(s, doc_T, r)
    q, kk, v = _rand((n_tot, H, D), 9), _rand((n_tot, H, D), 10), _rand((n_tot, H, D), 11)
    o0, _ = oracle.docs_attn_fwd(s, doc_T, r, k, 1.0, q, kk, v)
    kk2, v2 = kk.copy(), v.copy()
    kk2[:bases[1]] += 3.0  # disturb the first document's keys and values
    v2[:bases[1]] -= 2.0
    o1, _ = oracle.docs_attn_fwd(s, doc_T, r, k, 1.0, q, kk2, v2)
    assert np.array_equal(o0[bases[1]:], o1[bases[1]:])
    assert not np.allclose(o0[:bases[1]], o1[:bases[1]])


def test_one_document_is_the_plain_problem():
    s, T, r, k, H, D = 1, 8, 4, 1, 2, 4
    n = oracle.total_len(s, T, r)
    q, kk, v = _rand((n, H, D), 12), _rand((n, H, D), 13), _rand((n, H, D), 14)
    o, lse = oracle.docs_attn_fwd(s, [T], r, k, 0.7, q, kk, v)
    o1, l1 = oracle.attn_fwd(s, T, r, k, 0.7, q[None], kk[None], v[None])
    assert np.allclose(o, o1[0], atol=1e-12) and np.allclose(lse, l1[0], atol=1e-12)
