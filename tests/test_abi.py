"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
malformed arguments without launching anything (no GPU needed)."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2509_15763_b200 as ug
from paper_2509_15763_b200 import binding, build
from oracle import oracle

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def test_every_declared_symbol_is_exported():
    header = (ROOT / "include" / "unigist.h").read_text()
    declared = set(re.findall(r"\b(unigist_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(str(binding.LIB_PATH))
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.SYMBOLS)


@pytest.mark.parametrize("s,T,r,W", [(0, 448, 7, 64), (5, 64, 4, 12), (3, 48, 8, 80), (0, 56, 7, 14)])
def test_host_geometry_matches_oracle(s, T, r, W):
    p = ug.Problem(1, T, r, W, 1, 1, 64, num_sinks=s)
    k = oracle.window_units(W, r)
    assert ug.unigist_total_len(p) == oracle.total_len(s, T, r)
    assert ug.unigist_window_units(p) == k
    assert ug.unigist_visible_pairs(p) == oracle.count_pairs(s, T, r, k)
    assert ug.unigist_compact_len(p) == len(oracle.kept_set(s, T, r, k))


@pytest.mark.parametrize("s,T,r", [(0, 448, 7), (5, 64, 4), (128, 1024, 8), (0, 16, 16), (3, 9, 1), (2, 6, 3)])
def test_host_layout_matches_oracle(s, T, r):
    """on_device = 0: the index arrays are computed on the host (closed form) and must equal the oracle's,
    which walks Eq. 2 token by token."""
    import numpy as np
    import torch

    p = ug.Problem(1, T, r, 64, 1, 1, 64, num_sinks=s)
    N = ug.unigist_total_len(p)
    sp, up, pos = (torch.full((N,), -1, dtype=torch.int32) for _ in range(3))
    ug.unigist_layout(p, sp, up, pos)
    a, b, c = oracle.layout(s, T, r)
    assert np.array_equal(sp.numpy(), a) and np.array_equal(up.numpy(), b) and np.array_equal(pos.numpy(), c)


def test_interleaved_flag_is_validated_on_the_host():
    lib = binding.lib()
    buf = ctypes.create_string_buffer(1 << 16)
    a = ctypes.addressof(buf)
    a += (-a) % 16
    for prob in (ug.Problem(1, 448, 7, 64, 2, 1, 128, flags=ug.FLAG_INTERLEAVED),     # 7 does not divide 128
                 ug.Problem(1, 64, 8, 64, 2, 1, 64, flags=ug.FLAG_INTERLEAVED)):       # head_dim 64
        p = prob.c()
        before = ug.unigist_launch_count()
        rc = lib.unigist_attn_fwd(ctypes.byref(p), a, a, a, a, ctypes.cast(a, ctypes.POINTER(ctypes.c_float)), None, 0,
                                  None)
        assert rc == 5 and ug.unigist_launch_count() == before   # UNIGIST_ERR_UNSUPPORTED, nothing launched


def test_malformed_problems_are_rejected():
    bad = [ug.Problem(1, 10, 3, 4, 1, 1, 64), ug.Problem(1, 16, 4, 4, 3, 2, 64),
           ug.Problem(1, 16, 4, 4, 1, 1, 96), ug.Problem(0, 16, 4, 4, 1, 1, 64),
           ug.Problem(1, 16, 4, -1, 1, 1, 64),
           # batch entries and heads are grid dimensions of the kernels (at most 65535)
           ug.Problem(65536, 16, 4, 4, 1, 1, 64), ug.Problem(1, 16, 4, 4, 65536, 1, 64)]
    assert ug.unigist_total_len(ug.Problem(65535, 16, 4, 4, 1, 1, 64)) == 20
    for p in bad:
        assert ug.unigist_total_len(p) < 0
        assert ug.unigist_last_error_string()
        assert ug.unigist_workspace_bytes(p, ug.OP_BWD) == 0


def test_null_and_misaligned_pointers_are_rejected_before_any_launch():
    lib = binding.lib()
    p = ug.Problem(1, 16, 4, 4, 1, 1, 64).c()
    before = ug.unigist_launch_count()
    rc = lib.unigist_attn_fwd(ctypes.byref(p), None, None, None, None, None, None, 0, None)
    assert rc == 1
    buf = ctypes.create_string_buffer(4096)
    a = ctypes.addressof(buf)
    a += (-a) % 16
    rc = lib.unigist_gist_shift(ctypes.byref(p), a + 2, a + 1024, 1, 2, None)
    assert rc == 3
    rc = lib.unigist_gist_shift(ctypes.byref(p), a, a + 16, 1, 2, None)  # overlap
    assert rc == 1
    rc = lib.unigist_attn_bwd(ctypes.byref(p), *([a] * 9), a, 0, None)  # workspace too small
    assert rc == 4
    rc = lib.unigist_decode(1, 6, 4, 128, 0.0, a, a, a, 1, a, 1, a, a, None, a, 1 << 20, None)
    assert rc == 2
    assert ug.unigist_launch_count() == before


def test_backward_workspace_sizes_hold_every_part():
    """Host arithmetic only: the backward's scratch is Delta + (a bf16 copy of an fp32 dO) + (head_dim 128: the fp32
    dQ accumulator) + (the partial dK / dV of walks that are cut, only where one KV head's sweep exceeds the L2)."""
    def need(B, T, r, W, Hq, Hkv, D, flags=0, s=0):
        return ug.unigist_workspace_bytes(ug.Problem(B, T, r, W, Hq, Hkv, D, num_sinks=s, flags=flags), ug.OP_BWD)

    al = lambda x: -(-x // 256) * 256
    N = 16384 + 2048
    base = al(32 * N * 4) + al(N * 32 * 128 * 4)
    assert need(1, 16384, 8, 1024, 32, 8, 128) == base                      # 75 MB per KV head: no cut walks
    assert need(1, 16384, 8, 1024, 32, 8, 128, ug.FLAG_DOUT_FP32) == base + al(N * 32 * 128 * 2)
    assert need(1, 16384, 8, 1024, 32, 8, 64) == al(32 * N * 4)              # head_dim 64: Delta only
    # a fixed dQ order takes the two-kernel backward: no accumulator, no partial dK / dV
    assert need(1, 16384, 8, 1024, 32, 8, 128, ug.FLAG_DETERMINISTIC_DQ) == al(32 * N * 4)
    assert need(4, 32768, 4, 2048, 32, 8, 128, ug.FLAG_DETERMINISTIC_DQ) == al(4 * 32 * (32768 + 8192) * 4)
    # the training workload: 168 MB per KV head > 3/4 of the L2 -> 4 chunks over 64 gist key tiles per KV head
    Nt = 32768 + 8192
    got = need(4, 32768, 4, 2048, 32, 8, 128)
    assert got == al(4 * 32 * Nt * 4) + al(4 * Nt * 32 * 128 * 4) + 4 * 8 * 64 * 4 * 2 * 128 * 128 * 4
    # a packed sample: one scratch over all tokens; short documents cut nothing
    p = ug.Problem(1, 64, 4, 8, 4, 2, 128)
    docs = [256, 64, 64, 132]
    n_tot = ug.unigist_docs_total_len(p, docs)
    assert n_tot == sum(t + t // 4 for t in docs)
    assert ug.unigist_docs_workspace_bytes(p, ug.OP_BWD, docs) == al(4 * n_tot * 4) + al(n_tot * 4 * 128 * 4)
    assert ug.unigist_docs_workspace_bytes(p, ug.OP_FWD, docs) == 0
