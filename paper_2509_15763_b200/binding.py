"""Thin ctypes binding of ``libunigist.so``: argument marshalling only.

Every function has the name of the C entry point it calls (``include/unigist.h``).  torch is
used for device memory and streams; all arithmetic of the path runs in the library's kernels.
A missing library is an error: there is no Python or CPU fallback.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libunigist.so"

OP_FWD, OP_BWD, OP_COMPACT = 0, 1, 2
FLAG_DOUT_FP32 = 1
FLAG_DETERMINISTIC_DQ = 4
FLAG_INTERLEAVED = 2
PAGE_TOKENS = 64

SYMBOLS = [
    "unigist_total_len", "unigist_window_units", "unigist_compact_len", "unigist_visible_pairs",
    "unigist_workspace_bytes", "unigist_layout", "unigist_gist_shift", "unigist_gist_unshift",
    "unigist_attn_fwd", "unigist_attn_bwd", "unigist_kv_compact", "unigist_decode_workspace_bytes",
    "unigist_decode", "unigist_launch_count", "unigist_last_error_string",
    "unigist_kernel_timing", "unigist_kernel_timing_count", "unigist_kernel_timing_get",
    "unigist_device_status", "unigist_decode_static", "unigist_prefill_workspace_bytes", "unigist_prefill_chunk",
    "unigist_cache_state_bytes", "unigist_cache_state_init", "unigist_cache_append", "unigist_decode_step",
    "unigist_rope", "unigist_docs_total_len", "unigist_docs_workspace_bytes", "unigist_attn_fwd_docs",
    "unigist_attn_bwd_docs", "unigist_selftest_wait_timeout",
]


class UnigistError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"unigist status {code}: {msg}")
        self.code = code


class CProblem(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("raw_len", ctypes.c_int32), ("num_sinks", ctypes.c_int32),
                ("ratio", ctypes.c_int32), ("window", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
                ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("flags", ctypes.c_uint32)]


@dataclass(frozen=True)
class Problem:
    batch: int
    raw_len: int
    ratio: int
    window: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    num_sinks: int = 0
    softmax_scale: float = 0.0
    flags: int = 0

    def c(self) -> CProblem:
        return CProblem(self.batch, self.raw_len, self.num_sinks, self.ratio, self.window,
                        self.num_q_heads, self.num_kv_heads, self.head_dim, self.softmax_scale,
                        self.flags)


_lib = None


def lib() -> ctypes.CDLL:
    """Load the shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: run `python -m paper_2509_15763_b200.build` (needs nvcc)")
        L = ctypes.CDLL(str(LIB_PATH))
        P = ctypes.POINTER(CProblem)
        vp, i32, i64, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t, ctypes.c_float
        sig = {
            "unigist_total_len": (i32, [P]),
            "unigist_window_units": (i32, [P]),
            "unigist_compact_len": (i32, [P]),
            "unigist_visible_pairs": (i64, [P]),
            "unigist_workspace_bytes": (sz, [P, i32]),
            "unigist_layout": (i32, [P, vp, vp, vp, i32, vp]),
            "unigist_gist_shift": (i32, [P, vp, vp, i32, i32, vp]),
            "unigist_gist_unshift": (i32, [P, vp, vp, i32, i32, vp]),
            "unigist_rope": (i32, [P, vp, vp, i32, f32, ctypes.c_uint32, vp]),
            "unigist_docs_total_len": (i64, [P, i32, vp]),
            "unigist_docs_workspace_bytes": (sz, [P, i32, i32, vp]),
            "unigist_attn_fwd_docs": (i32, [P, i32, vp] + [vp] * 6 + [sz, vp]),
            "unigist_attn_bwd_docs": (i32, [P, i32, vp] + [vp] * 10 + [sz, vp]),
            "unigist_attn_fwd": (i32, [P, vp, vp, vp, vp, vp, vp, sz, vp]),
            "unigist_attn_bwd": (i32, [P] + [vp] * 10 + [sz, vp]),
            "unigist_kv_compact": (i32, [P, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, sz, vp]),
            "unigist_decode_workspace_bytes": (sz, [i32] * 5),
            "unigist_prefill_workspace_bytes": (sz, [P, i32, i32]),
            "unigist_cache_state_bytes": (sz, [P]),
            "unigist_cache_state_init": (i32, [P, i32, vp, vp]),
            "unigist_cache_append": (i32, [P, vp, vp, i32, vp, vp, i32, vp, i32, vp, vp, vp]),
            "unigist_decode_step": (i32, [P, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, vp, sz, vp]),
            "unigist_prefill_chunk": (i32, [P, i32, i32, vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, sz, vp]),
            "unigist_decode": (i32, [i32, i32, i32, i32, f32, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, sz, vp]),
            "unigist_kernel_timing": (i32, [i32]),
            "unigist_kernel_timing_count": (i32, []),
            "unigist_kernel_timing_get": (i32, [i32, ctypes.c_char_p, i32, ctypes.POINTER(ctypes.c_float)]),
            "unigist_device_status": (i32, []),
            "unigist_selftest_wait_timeout": (i32, [vp]),
            "unigist_decode_static": (i32, [i32, i32, i32, i32, f32, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp]),
            "unigist_launch_count": (i64, []),
            "unigist_last_error_string": (ctypes.c_char_p, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise UnigistError(rc, lib().unigist_last_error_string().decode())


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def unigist_total_len(p: Problem) -> int:
    return lib().unigist_total_len(ctypes.byref(p.c()))


def unigist_window_units(p: Problem) -> int:
    return lib().unigist_window_units(ctypes.byref(p.c()))


def unigist_compact_len(p: Problem) -> int:
    return lib().unigist_compact_len(ctypes.byref(p.c()))


def unigist_visible_pairs(p: Problem) -> int:
    return lib().unigist_visible_pairs(ctypes.byref(p.c()))


def unigist_workspace_bytes(p: Problem, op: int) -> int:
    return lib().unigist_workspace_bytes(ctypes.byref(p.c()), op)


def unigist_launch_count() -> int:
    return lib().unigist_launch_count()


def unigist_kernel_timing(enable: bool) -> None:
    _check(lib().unigist_kernel_timing(int(enable)))


def unigist_kernel_timing_count() -> int:
    return lib().unigist_kernel_timing_count()


def unigist_kernel_timing_get(index: int):
    """-> (kernel name, milliseconds) of recorded launch `index` (waits for it to finish)."""
    name = ctypes.create_string_buffer(128)
    ms = ctypes.c_float()
    _check(lib().unigist_kernel_timing_get(index, name, 128, ctypes.byref(ms)))
    return name.value.decode(), ms.value


DECODE_STATIC_SCRATCH_BYTES = 8 << 20


def unigist_decode_static(q, k_cache, v_cache, block_table, seq_lens, o, lse=None,
                          softmax_scale: float = 0.0, stream=None):
    """unigist_decode without a workspace argument: scratch is the library's built-in array, so
    nothing is allocated.  Calls on one device must not overlap; see include/unigist.h."""
    _dev(q, k_cache, v_cache, block_table, seq_lens, o, lse)
    S, Hq, D = q.shape
    _check(lib().unigist_decode_static(S, Hq, k_cache.shape[1], D, softmax_scale, _ptr(q), _ptr(k_cache),
                                       _ptr(v_cache), k_cache.shape[0], _ptr(block_table),
                                       block_table.shape[1], _ptr(seq_lens), _ptr(o), _ptr(lse),
                                       _stream(stream)))


def unigist_device_status() -> None:
    """Synchronise the device; raise UnigistError if a kernel gave up on a bounded wait."""
    _check(lib().unigist_device_status())


def unigist_selftest_wait_timeout(stream=None) -> None:
    """Enqueue the self-check block whose bounded wait runs out (see unigist_device_status)."""
    _check(lib().unigist_selftest_wait_timeout(_stream(stream)))


def unigist_last_error_string() -> str:
    return lib().unigist_last_error_string().decode()


def unigist_layout(p: Problem, shift_perm=None, unshift_perm=None, pos_ids=None, stream=None):
    """Fill int32 tensors of length N; all on the CPU or all on the GPU."""
    ts = [t for t in (shift_perm, unshift_perm, pos_ids) if t is not None]
    on_device = int(bool(ts) and ts[0].is_cuda)
    for t in ts:
        if t.dtype != torch.int32 or not t.is_contiguous() or t.is_cuda != bool(on_device):
            raise ValueError("layout arrays must be contiguous int32 on one device")
    st = _stream(stream) if on_device else None
    _check(lib().unigist_layout(ctypes.byref(p.c()), _ptr(shift_perm), _ptr(unshift_perm),
                                _ptr(pos_ids), on_device, st))


def unigist_gist_shift(p: Problem, src, dst, stream=None):
    _dev(src, dst)
    _check(lib().unigist_gist_shift(ctypes.byref(p.c()), _ptr(src), _ptr(dst), src.shape[2],
                                    src.element_size(), _stream(stream)))


def unigist_gist_unshift(p: Problem, src, dst, stream=None):
    _dev(src, dst)
    _check(lib().unigist_gist_unshift(ctypes.byref(p.c()), _ptr(src), _ptr(dst), src.shape[2],
                                      src.element_size(), _stream(stream)))


def _doc_array(doc_raw_len):
    return (ctypes.c_int32 * len(doc_raw_len))(*[int(t) for t in doc_raw_len])


def unigist_docs_total_len(p: Problem, doc_raw_len) -> int:
    return int(lib().unigist_docs_total_len(ctypes.byref(p.c()), len(doc_raw_len), _doc_array(doc_raw_len)))


def unigist_docs_workspace_bytes(p: Problem, op: int, doc_raw_len) -> int:
    return int(lib().unigist_docs_workspace_bytes(ctypes.byref(p.c()), op, len(doc_raw_len), _doc_array(doc_raw_len)))


def unigist_attn_fwd_docs(p: Problem, doc_raw_len, q, k, v, o, lse, workspace=None, stream=None):
    _dev(q, k, v, o, lse, workspace)
    _check(lib().unigist_attn_fwd_docs(ctypes.byref(p.c()), len(doc_raw_len), _doc_array(doc_raw_len), _ptr(q), _ptr(k),
                                       _ptr(v), _ptr(o), _ptr(lse), _ptr(workspace),
                                       0 if workspace is None else workspace.numel() * workspace.element_size(),
                                       _stream(stream)))


def unigist_attn_bwd_docs(p: Problem, doc_raw_len, q, k, v, o, lse, d_o, dq, dk, dv, workspace, stream=None):
    _dev(q, k, v, o, lse, d_o, dq, dk, dv, workspace)
    _check(lib().unigist_attn_bwd_docs(ctypes.byref(p.c()), len(doc_raw_len), _doc_array(doc_raw_len), _ptr(q), _ptr(k),
                                       _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv),
                                       _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


ROPE_TO_SHIFTED, ROPE_FROM_SHIFTED, ROPE_INVERSE = 1, 2, 4


def unigist_rope(p: Problem, src, dst, theta_base: float, flags: int = 0, stream=None):
    _dev(src, dst)
    _check(lib().unigist_rope(ctypes.byref(p.c()), _ptr(src), _ptr(dst), src.shape[2], float(theta_base), flags,
                              _stream(stream)))


def unigist_attn_fwd(p: Problem, q, k, v, o, lse, workspace=None, stream=None):
    _dev(q, k, v, o, lse, workspace)
    _check(lib().unigist_attn_fwd(ctypes.byref(p.c()), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                  _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
                                  _stream(stream)))


def unigist_attn_bwd(p: Problem, q, k, v, o, lse, d_o, dq, dk, dv, workspace, stream=None):
    _dev(q, k, v, o, lse, d_o, dq, dk, dv, workspace)
    _check(lib().unigist_attn_bwd(ctypes.byref(p.c()), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse),
                                  _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace),
                                  0 if workspace is None else workspace.numel() * workspace.element_size(),
                                  _stream(stream)))


def unigist_kv_compact(p: Problem, k, v, k_cache, v_cache, block_table, seq_lens, kept_idx=None,
                       workspace=None, stream=None):
    _dev(k, v, k_cache, v_cache, block_table, seq_lens, kept_idx, workspace)
    _check(lib().unigist_kv_compact(ctypes.byref(p.c()), _ptr(k), _ptr(v), _ptr(k_cache), _ptr(v_cache),
                                    k_cache.shape[0], _ptr(block_table), block_table.shape[1],
                                    _ptr(seq_lens), _ptr(kept_idx), _ptr(workspace),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream(stream)))


def unigist_prefill_workspace_bytes(p: Problem, unit_begin: int, unit_count: int) -> int:
    return lib().unigist_prefill_workspace_bytes(ctypes.byref(p.c()), unit_begin, unit_count)


def unigist_prefill_chunk(p: Problem, unit_begin: int, unit_count: int, q, k, v, k_cache, v_cache, block_table,
                          seq_lens, o, lse, workspace, stream=None):
    _dev(q, k, v, k_cache, v_cache, block_table, seq_lens, o, lse, workspace)
    _check(lib().unigist_prefill_chunk(ctypes.byref(p.c()), unit_begin, unit_count, _ptr(q), _ptr(k), _ptr(v),
                                       _ptr(k_cache), _ptr(v_cache), k_cache.shape[0], _ptr(block_table),
                                       block_table.shape[1], _ptr(seq_lens), _ptr(o), _ptr(lse), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream)))


def unigist_cache_state_bytes(p: Problem) -> int:
    return lib().unigist_cache_state_bytes(ctypes.byref(p.c()))


def unigist_cache_state_init(p: Problem, units_done: int, state, stream=None):
    _dev(state)
    _check(lib().unigist_cache_state_init(ctypes.byref(p.c()), units_done, _ptr(state), _stream(stream)))


def unigist_cache_append(p: Problem, k_new, v_new, is_gist: bool, k_cache, v_cache, block_table, seq_lens, state,
                         stream=None):
    _dev(k_new, v_new, k_cache, v_cache, block_table, seq_lens, state)
    _check(lib().unigist_cache_append(ctypes.byref(p.c()), _ptr(k_new), _ptr(v_new), int(bool(is_gist)),
                                      _ptr(k_cache), _ptr(v_cache), k_cache.shape[0], _ptr(block_table),
                                      block_table.shape[1], _ptr(seq_lens), _ptr(state), _stream(stream)))


def unigist_decode_step(p: Problem, q, k_cache, v_cache, block_table, seq_lens, state, o, lse=None, workspace=None,
                        stream=None):
    _dev(q, k_cache, v_cache, block_table, seq_lens, state, o, lse, workspace)
    _check(lib().unigist_decode_step(ctypes.byref(p.c()), _ptr(q), _ptr(k_cache), _ptr(v_cache), k_cache.shape[0],
                                     _ptr(block_table), block_table.shape[1], _ptr(seq_lens), _ptr(state), _ptr(o),
                                     _ptr(lse), _ptr(workspace),
                                     0 if workspace is None else workspace.numel() * workspace.element_size(),
                                     _stream(stream)))


def unigist_decode_workspace_bytes(num_seqs, num_q_heads, num_kv_heads, head_dim, max_blocks_per_seq) -> int:
    return lib().unigist_decode_workspace_bytes(num_seqs, num_q_heads, num_kv_heads, head_dim,
                                                max_blocks_per_seq)


def unigist_decode(q, k_cache, v_cache, block_table, seq_lens, o, lse=None, workspace=None,
                   softmax_scale: float = 0.0, stream=None):
    _dev(q, k_cache, v_cache, block_table, seq_lens, o, lse, workspace)
    S, Hq, D = q.shape
    _check(lib().unigist_decode(S, Hq, k_cache.shape[1], D, softmax_scale, _ptr(q), _ptr(k_cache),
                                _ptr(v_cache), k_cache.shape[0], _ptr(block_table), block_table.shape[1],
                                _ptr(seq_lens), _ptr(o), _ptr(lse), _ptr(workspace),
                                0 if workspace is None else workspace.numel() * workspace.element_size(),
                                _stream(stream)))
