"""Pins for the oracle's mask, layout and compaction rules (CPU only).

Each check compares the oracle with something that is not the oracle: hand-written
fixtures, a literal set construction of Eq. 3 in Python, closed forms, or brute force.
"""
from pathlib import Path

import numpy as np
import pytest

from oracle import oracle

GOLDEN = Path(__file__).parent / "golden"

CASES = [(0, 6, 2, 1), (1, 6, 2, 1), (0, 56, 7, 2), (5, 64, 4, 3), (3, 48, 8, 10),
         (0, 12, 1, 2), (2, 12, 12, 0), (0, 30, 5, 0), (4, 24, 3, 100)]


def literal_visible_sets(s, T, r, k):
    """Eq. 3 built as Python sets: A(z_t) = (S | G | W_t) & {j <= t}."""
    n = T // r
    seq = [("S", i) for i in range(s)]
    units = []
    for u in range(n):
        members = []
        for p in range(r):
            members.append(len(seq))
            seq.append(("x", u * r + p))
        members.append(len(seq))
        seq.append(("g", u))
        units.append(members)
    S = {i for i, (kd, _) in enumerate(seq) if kd == "S"}
    G = {i for i, (kd, _) in enumerate(seq) if kd == "g"}
    unit_of = {}
    for u, members in enumerate(units):
        for i in members:
            unit_of[i] = u
    out = []
    for t in range(len(seq)):
        W = set()
        if t in unit_of:  # current unit + previous k units
            for u in range(max(0, unit_of[t] - k), unit_of[t] + 1):
                W |= set(units[u])
        out.append((S | G | W) & set(range(t + 1)))
    return seq, out


def test_mask_matches_handwritten_fixture():
    rows = [l.strip() for l in (GOLDEN / "eq3_mask_s1_T6_r2_k1.txt").read_text().splitlines()
            if l.strip() and not l.startswith("#")]
    want = np.array([[int(c) for c in row] for row in rows], dtype=np.uint8)
    got = oracle.mask(1, 6, 2, 1)
    assert got.shape == want.shape
    assert (got == want).all()


@pytest.mark.parametrize("s,T,r,k", CASES)
def test_mask_matches_literal_sets(s, T, r, k):
    _, sets = literal_visible_sets(s, T, r, k)
    m = oracle.mask(s, T, r, k)
    N = oracle.total_len(s, T, r)
    assert m.shape == (N, N)
    for t in range(N):
        assert set(np.nonzero(m[t])[0].tolist()) == sets[t], t


def closed_form_row_count(s, T, r, k, seq, t):
    kd, num = seq[t]
    if kd == "S":
        return num + 1
    if kd == "x":
        u, p = divmod(num, r)
        return s + min(u, k) * r + p + 1 + u
    return s + (min(num, k) + 1) * r + num + 1


def closed_form_pairs(s, T, r, k):
    n = T // r
    tot = s * (s + 1) // 2 + s * (T + n)
    for u in range(n):
        tot += r * r * min(u, k) + r * (r + 1) // 2 + r * u
        tot += (min(u, k) + 1) * r + u + 1
    return tot


@pytest.mark.parametrize("s,T,r,k", CASES)
def test_row_and_pair_counts_closed_form(s, T, r, k):
    seq, _ = literal_visible_sets(s, T, r, k)
    m = oracle.mask(s, T, r, k)
    for t in range(len(seq)):
        assert int(m[t].sum()) == closed_form_row_count(s, T, r, k, seq, t)
    assert oracle.count_pairs(s, T, r, k) == int(m.sum()) == closed_form_pairs(s, T, r, k)


def test_every_row_sees_itself_and_nothing_later():
    m = oracle.mask(3, 40, 4, 2)
    assert (np.diag(m) == 1).all()
    assert (np.triu(m, 1) == 0).all()


def test_full_window_is_plain_causal():
    m = oracle.mask(2, 24, 3, 8)  # k >= n
    assert (m == np.tril(np.ones_like(m))).all()


def test_speedup_bound_approaches_ratio():
    """Section 5 (efficiency): the gain over full causal attention grows with length and
    approaches the compression ratio.  Pair counts stand in for time."""
    r, W, s = 4, 128, 128
    prev = 0.0
    for T in (16384, 32768, 65536, 131072):
        ratio = (T * (T + 1) // 2) / closed_form_pairs(s, T, r, W // r)
        assert prev < ratio < r
        prev = ratio
    assert prev > 0.75 * r  # 3.15 at 128K; the paper's table gives 3.18x measured


def test_layout_matches_handwritten_fixture():
    rows = [l for l in (GOLDEN / "eq2_layout_s2_T6_r3.txt").read_text().splitlines()
            if l.strip() and not l.startswith("#")]
    want = [np.array(l.split(), dtype=np.int32) for l in rows]
    sp, up, pos = oracle.layout(2, 6, 3)
    assert (sp == want[0]).all() and (up == want[1]).all() and (pos == want[2]).all()


@pytest.mark.parametrize("s,T,r", [(0, 448, 7), (5, 64, 4), (0, 16, 16), (3, 9, 1), (128, 1024, 8)])
def test_layout_is_stable_partition(s, T, r):
    sp, up, pos = oracle.layout(s, T, r)
    n, N = T // r, s + T + T // r
    assert sorted(sp.tolist()) == list(range(N))
    assert (up[sp] == np.arange(N)).all() and (sp[up] == np.arange(N)).all()
    seq, _ = literal_visible_sets(s, T, r, 0)
    kinds = [seq[i][0] for i in sp]
    assert kinds == ["S"] * s + ["x"] * T + ["g"] * n
    for a, b in ((0, s), (s, s + T), (s + T, N)):  # order kept inside each kind
        assert (np.diff(sp[a:b]) > 0).all()
    # closed forms
    i = np.arange(T)
    assert (sp[s:s + T] == s + i + i // r).all()
    u = np.arange(n)
    assert (sp[s + T:] == s + u * (r + 1) + r).all()
    # raw-token distances are unchanged by the inserted gists
    raw_pos = pos[sp[s:s + T]]
    assert (np.diff(raw_pos) == 1).all()
    if n > 1:
        nxt = sp[s + T:-1] + 1  # raw token right after each gist but the last
        assert (pos[sp[s + T:-1]] == pos[nxt]).all()


@pytest.mark.parametrize("s,T,r,k", CASES)
def test_kept_set_is_future_visible_set(s, T, r, k):
    """Section 4.3: raw tokens outside the local window are never attended to by future
    tokens and can be dropped.  Brute force over a literally extended sequence."""
    n = T // r
    ext_units = k + 3
    _, sets = literal_visible_sets(s, T + ext_units * r, r, k)
    N = oracle.total_len(s, T, r)
    future = set()
    for t in range(N, len(sets)):
        future |= {j for j in sets[t] if j < N}
    kept = oracle.kept_set(s, T, r, k)
    assert set(kept.tolist()) == future
    kk = min(k, n)
    assert len(kept) == s + n + kk * r
    seq, _ = literal_visible_sets(s, T, r, k)
    kinds = [seq[i][0] for i in kept]
    assert kinds == ["S"] * s + ["g"] * n + ["x"] * (kk * r)
    raw_numbers = [seq[i][1] for i in kept[s + n:]]
    assert raw_numbers == list(range(T - kk * r, T))
