"""Pins of the oracle's rotary embedding with aligned position ids (Section 4.1, step 3)."""
import numpy as np

from oracle import oracle


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_rope_is_complex_multiplication():
    # (x_j + i x_{j+D/2}) * exp(i pos theta_j): the same rotation written with complex numbers
    s, T, r, D, H = 2, 12, 3, 8, 2
    _, _, pos = oracle.layout(s, T, r)
    x = _rand((oracle.total_len(s, T, r), H, D), 1)
    y = oracle.rope(x, pos, 10000.0)
    z = x[..., : D // 2] + 1j * x[..., D // 2:]
    freq = 10000.0 ** (-np.arange(D // 2) * 2.0 / D)
    w = z * np.exp(1j * pos[:, None, None] * freq[None, None, :])
    assert np.allclose(y[..., : D // 2], w.real, atol=1e-12)
    assert np.allclose(y[..., D // 2:], w.imag, atol=1e-12)


def test_rope_closed_form_two_features():
    # D = 2: one pair, frequency 1: a plane rotation by pos radians
    x = np.array([[[1.0, 0.0]], [[0.0, 2.0]], [[3.0, 4.0]]])
    pos = np.array([0, 1, 2])
    y = oracle.rope(x, pos, 10000.0)
    assert np.allclose(y[0, 0], [1.0, 0.0])
    assert np.allclose(y[1, 0], [-2.0 * np.sin(1.0), 2.0 * np.cos(1.0)])
    assert np.allclose(y[2, 0], [3 * np.cos(2.0) - 4 * np.sin(2.0), 4 * np.cos(2.0) + 3 * np.sin(2.0)])


def test_rope_keeps_norms_and_relative_distance():
    s, T, r, D, H = 1, 16, 4, 16, 1
    N = oracle.total_len(s, T, r)
    _, _, pos = oracle.layout(s, T, r)
    q, k = _rand((N, H, D), 2), _rand((N, H, D), 3)
    qr, kr = oracle.rope(q, pos, 500000.0), oracle.rope(k, pos, 500000.0)
    assert np.allclose(np.linalg.norm(qr, axis=-1), np.linalg.norm(q, axis=-1))
    # the score of a (query, key) pair depends on the difference of their ids only
    q1 = np.repeat(q[:1], N, 0)
    k1 = np.repeat(k[:1], N, 0)
    a = oracle.rope(q1, pos, 500000.0)
    b = oracle.rope(k1, pos, 500000.0)
    t0, j0, t1, j1 = 7, 3, 12, 8  # raw tokens: pos differences are both 4 (ids skip no gist)
    sp, up, _ = oracle.layout(s, T, r)
    raw = sp[s:s + T]  # interleaved index of each raw token
    d0 = np.dot(a[raw[t0], 0], b[raw[j0], 0])
    d1 = np.dot(a[raw[t1], 0], b[raw[j1], 0])
    assert np.isclose(d0, d1)


def test_gist_shares_the_angle_of_the_next_raw_token():
    s, T, r, D = 0, 8, 2, 4
    N = oracle.total_len(s, T, r)
    _, _, pos = oracle.layout(s, T, r)
    x = np.ones((N, 1, D))
    y = oracle.rope(x, pos, 100.0)
    # interleaved index of gist u is u (r + 1) + r; the raw token after it sits at the next index
    for u in range(T // r - 1):
        g = u * (r + 1) + r
        assert np.allclose(y[g], y[g + 1])
    assert np.allclose(y[0], x[0])  # id 0: no rotation


def test_negated_ids_undo_the_rotation():
    # the rotation is orthogonal: rotating by the negated ids is its transpose and its inverse
    s, T, r, D, H = 2, 12, 4, 8, 2
    _, _, pos = oracle.layout(s, T, r)
    x, dy = _rand((oracle.total_len(s, T, r), H, D), 5), _rand((oracle.total_len(s, T, r), H, D), 6)
    y = oracle.rope(x, pos, 10000.0)
    assert np.allclose(oracle.rope(y, -pos.astype(np.int64), 10000.0), x, atol=1e-12)
    assert np.isclose((y * dy).sum(), (x * oracle.rope(dy, -pos.astype(np.int64), 10000.0)).sum())
