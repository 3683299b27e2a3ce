"""ctypes front end of the fp64 CPU oracle -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It imports nothing from the CUDA package and the CUDA package
imports nothing from here.

Arrays are numpy float64 in the INTERLEAVED token order of Eq. 2, laid out
``[B, N, H, D]`` like the tensors the library takes; the helpers below cut them
into (batch, KV-head) slices for the C routines (grouped-query attention:
query head ``h`` uses KV head ``h // G``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "unigist_oracle.c"
_LIB = _HERE / "libunigist_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
             "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        i64, i32, f64 = ctypes.c_int64, ctypes.c_int32, ctypes.c_double
        p = ctypes.c_void_p
        L.ug_oracle_visible.argtypes = [i64] * 5
        L.ug_oracle_visible.restype = i32
        L.ug_oracle_mask.argtypes = [i64] * 6 + [p]
        L.ug_oracle_mask.restype = i32
        L.ug_oracle_count_pairs.argtypes = [i64] * 4
        L.ug_oracle_count_pairs.restype = i64
        L.ug_oracle_layout.argtypes = [i64] * 3 + [p] * 3
        L.ug_oracle_layout.restype = i32
        L.ug_oracle_attn_fwd.argtypes = [i64] * 4 + [i32, i32, f64, p, p, p, i64, i64, p, p]
        L.ug_oracle_attn_fwd.restype = i32
        L.ug_oracle_attn_bwd.argtypes = [i64] * 4 + [i32, i32, f64] + [p] * 7
        L.ug_oracle_attn_bwd.restype = i32
        L.ug_oracle_attn_bwd_sample.argtypes = [i64] * 4 + [i32, i32, f64] + [p] * 4 + [i64, p, i64, p, p, p, p]
        L.ug_oracle_attn_bwd_sample.restype = i32
        L.ug_oracle_kept_set.argtypes = [i64] * 4 + [p]
        L.ug_oracle_kept_set.restype = i64
        L.ug_oracle_decode.argtypes = [i64, i32, i32, f64] + [p] * 5
        L.ug_oracle_decode.restype = i32
        L.ug_oracle_num_threads.restype = i32
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(lib().ug_oracle_num_threads())


def total_len(s: int, T: int, r: int) -> int:
    """Eq. 2: T' = s + T + T/r."""
    assert T % r == 0
    return s + T + T // r


def window_units(W: int, r: int) -> int:
    """Local window of W raw tokens -> k previous gist units, rounded up."""
    return -(-W // r)


def visible(t, j, s, r, k) -> bool:
    return bool(lib().ug_oracle_visible(t, j, s, r, k))


def mask(s, T, r, k, row_begin=0, row_end=None) -> np.ndarray:
    N = total_len(s, T, r)
    row_end = N if row_end is None else row_end
    m = np.empty((row_end - row_begin, N), dtype=np.uint8)
    assert lib().ug_oracle_mask(s, T, r, k, row_begin, row_end, _ptr(m)) == 0
    return m


def count_pairs(s, T, r, k) -> int:
    return int(lib().ug_oracle_count_pairs(s, T, r, k))


def layout(s, T, r):
    """-> (shift_perm, unshift_perm, pos_ids), int32 arrays of length N."""
    N = total_len(s, T, r)
    sp = np.empty(N, np.int32)
    up = np.empty(N, np.int32)
    pos = np.empty(N, np.int32)
    assert lib().ug_oracle_layout(s, T, r, _ptr(sp), _ptr(up), _ptr(pos)) == 0
    return sp, up, pos


def attn_fwd_slice(s, T, r, k, scale, q, kk, v, row_begin=0, row_end=None):
    """One (batch, KV head): q [N,G,D], kk/v [N,D] -> o [rows,G,D], lse [rows,G]."""
    q, kk, v = _c64(q), _c64(kk), _c64(v)
    N, G, D = q.shape
    assert N == total_len(s, T, r) and kk.shape == (N, D) and v.shape == (N, D)
    row_end = N if row_end is None else row_end
    o = np.empty((row_end - row_begin, G, D))
    lse = np.empty((row_end - row_begin, G))
    rc = lib().ug_oracle_attn_fwd(s, T, r, k, G, D, float(scale), _ptr(q), _ptr(kk),
                                  _ptr(v), row_begin, row_end, _ptr(o), _ptr(lse))
    assert rc == 0, rc
    return o, lse


def attn_bwd_slice(s, T, r, k, scale, q, kk, v, dout):
    """One (batch, KV head): -> dq [N,G,D], dk [N,D], dv [N,D]."""
    q, kk, v, dout = _c64(q), _c64(kk), _c64(v), _c64(dout)
    N, G, D = q.shape
    assert N == total_len(s, T, r) and dout.shape == q.shape
    dq = np.empty_like(q)
    dk = np.empty_like(kk)
    dv = np.empty_like(v)
    rc = lib().ug_oracle_attn_bwd(s, T, r, k, G, D, float(scale), _ptr(q), _ptr(kk),
                                  _ptr(v), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv))
    assert rc == 0, rc
    return dq, dk, dv


def attn_bwd_sample(s, T, r, k, scale, q, kk, v, dout, rows, keys):
    """One (batch, KV head), sampled outputs: dq of `rows` [R,G,D]; dk, dv of `keys` [K,D]."""
    q, kk, v, dout = _c64(q), _c64(kk), _c64(v), _c64(dout)
    N, G, D = q.shape
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    keys = np.ascontiguousarray(keys, dtype=np.int64)
    dq = np.empty((len(rows), G, D))
    dk = np.empty((len(keys), D))
    dv = np.empty((len(keys), D))
    rc = lib().ug_oracle_attn_bwd_sample(s, T, r, k, G, D, float(scale), _ptr(q), _ptr(kk), _ptr(v),
                                         _ptr(dout), len(rows), _ptr(rows), len(keys), _ptr(keys),
                                         _ptr(dq), _ptr(dk), _ptr(dv))
    assert rc == 0, rc
    return dq, dk, dv


def attn_fwd(s, T, r, k, scale, q, kk, v):
    """Whole problem: q [B,N,Hq,D], kk/v [B,N,Hkv,D] -> o [B,N,Hq,D], lse [B,Hq,N]."""
    B, N, Hq, D = q.shape
    Hkv = kk.shape[2]
    G = Hq // Hkv
    o = np.empty((B, N, Hq, D))
    lse = np.empty((B, Hq, N))
    for b in range(B):
        for h in range(Hkv):
            os_, ls = attn_fwd_slice(s, T, r, k, scale, q[b, :, h * G:(h + 1) * G],
                                     kk[b, :, h], v[b, :, h])
            o[b, :, h * G:(h + 1) * G] = os_
            lse[b, h * G:(h + 1) * G] = ls.T
    return o, lse


def attn_bwd(s, T, r, k, scale, q, kk, v, dout):
    """Whole problem -> dq [B,N,Hq,D], dk, dv [B,N,Hkv,D]."""
    B, N, Hq, D = q.shape
    Hkv = kk.shape[2]
    G = Hq // Hkv
    dq = np.empty((B, N, Hq, D))
    dk = np.empty((B, N, Hkv, D))
    dv = np.empty((B, N, Hkv, D))
    for b in range(B):
        for h in range(Hkv):
            a, c, d = attn_bwd_slice(s, T, r, k, scale, q[b, :, h * G:(h + 1) * G],
                                     kk[b, :, h], v[b, :, h], dout[b, :, h * G:(h + 1) * G])
            dq[b, :, h * G:(h + 1) * G] = a
            dk[b, :, h] = c
            dv[b, :, h] = d
    return dq, dk, dv


def kept_set(s, T, r, k) -> np.ndarray:
    """Interleaved indices that survive compaction, in cache order."""
    N = total_len(s, T, r)
    buf = np.empty(N, np.int32)
    c = lib().ug_oracle_kept_set(s, T, r, k, _ptr(buf))
    assert c >= 0
    return buf[:c].copy()


def decode_slice(scale, qd, kc, vc):
    """qd [G,D], kc/vc [L,D] -> o [G,D], lse [G]."""
    qd, kc, vc = _c64(qd), _c64(kc), _c64(vc)
    G, D = qd.shape
    L = kc.shape[0]
    o = np.empty((G, D))
    lse = np.empty(G)
    rc = lib().ug_oracle_decode(L, G, D, float(scale), _ptr(qd), _ptr(kc), _ptr(vc),
                                _ptr(o), _ptr(lse))
    assert rc == 0, rc
    return o, lse


def decode(scale, q, k_list, v_list):
    """q [S,Hq,D]; k_list[s], v_list[s] = [L_s,Hkv,D] -> o [S,Hq,D], lse [S,Hq]."""
    S, Hq, D = q.shape
    o = np.empty((S, Hq, D))
    lse = np.empty((S, Hq))
    for i in range(S):
        Hkv = k_list[i].shape[1]
        G = Hq // Hkv
        for h in range(Hkv):
            a, b = decode_slice(scale, q[i, h * G:(h + 1) * G], k_list[i][:, h], v_list[i][:, h])
            o[i, h * G:(h + 1) * G] = a
            lse[i, h * G:(h + 1) * G] = b
    return o, lse


def rope(x, pos_ids, theta_base):
    """Rotary position embedding with the aligned position ids (Section 4.1, step 3).

    x [N, H, D] in interleaved order, pos_ids [N] (from layout()).  The paper fixes the ids, not
    the rotary convention; this is the one of the Llama models it trains: feature j < D/2 pairs
    with feature j + D/2, and the pair of token t is rotated by the angle
    pos_ids[t] * theta_base^(-2 j / D):
        y[j]       = x[j] cos - x[j + D/2] sin
        y[j + D/2] = x[j + D/2] cos + x[j] sin
    """
    x = np.asarray(x, np.float64)
    N, H, D = x.shape
    half = D // 2
    y = np.empty_like(x)
    for t in range(N):
        for j in range(half):
            ang = float(pos_ids[t]) * float(theta_base) ** (-2.0 * j / D)
            c, s_ = np.cos(ang), np.sin(ang)
            y[t, :, j] = x[t, :, j] * c - x[t, :, j + half] * s_
            y[t, :, j + half] = x[t, :, j + half] * c + x[t, :, j] * s_
    return y


def docs_mask(s, doc_T, r, k) -> np.ndarray:
    """Mask of a packed sample under cross-document masking (Section 5.1; documents padded to a
    multiple of r, appendix on training data): token i of document a sees token j of document b
    iff a == b and Eq. 3 holds inside that document (each document restarts its sinks, units and
    window).  Interleaved order, documents one after another.  [N_total, N_total] bool."""
    doc_of, local = [], []
    for d, T in enumerate(doc_T):
        n = total_len(s, T, r)
        doc_of += [d] * n
        local += list(range(n))
    n_tot = len(doc_of)
    m = np.zeros((n_tot, n_tot), bool)
    for i in range(n_tot):
        for j in range(n_tot):
            m[i, j] = doc_of[i] == doc_of[j] and visible(local[i], local[j], s, r, k)
    return m


def docs_attn_fwd(s, doc_T, r, k, scale, q, kk, v):
    """Dense softmax attention under docs_mask: q [N,Hq,D], kk/v [N,Hkv,D] (interleaved, packed)
    -> o [N,Hq,D], lse [Hq,N].  The plain definition, O(N^2): small cases only."""
    q, kk, v = _c64(q), _c64(kk), _c64(v)
    N, Hq, D = q.shape
    G = Hq // kk.shape[1]
    m = docs_mask(s, doc_T, r, k)
    o = np.empty((N, Hq, D))
    lse = np.empty((Hq, N))
    for h in range(Hq):
        sc = scale * (q[:, h] @ kk[:, h // G].T)
        sc = np.where(m, sc, -np.inf)
        mx = sc.max(axis=1, keepdims=True)
        e = np.exp(sc - mx)
        l = e.sum(axis=1, keepdims=True)
        o[:, h] = (e / l) @ v[:, h // G]
        lse[h] = (mx + np.log(l))[:, 0]
    return o, lse


def docs_attn_bwd(s, doc_T, r, k, scale, q, kk, v, dout):
    """Gradients of docs_attn_fwd's o with respect to q, kk, v for the cotangent dout (dense)."""
    q, kk, v, dout = _c64(q), _c64(kk), _c64(v), _c64(dout)
    N, Hq, D = q.shape
    G = Hq // kk.shape[1]
    m = docs_mask(s, doc_T, r, k)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(kk), np.zeros_like(v)
    for h in range(Hq):
        g = h // G
        sc = np.where(m, scale * (q[:, h] @ kk[:, g].T), -np.inf)
        p = np.exp(sc - sc.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        dv[:, g] += p.T @ dout[:, h]
        dp = dout[:, h] @ v[:, g].T
        ds = p * (dp - (p * dp).sum(axis=1, keepdims=True))
        dq[:, h] = scale * (ds @ kk[:, g])
        dk[:, g] += scale * (ds.T @ q[:, h])
    return dq, dk, dv
