"""UniGist gist-masked attention for B200 (sm_100a): Python binding of the C-ABI library."""
from .binding import (DECODE_STATIC_SCRATCH_BYTES, FLAG_DETERMINISTIC_DQ, FLAG_DOUT_FP32, FLAG_INTERLEAVED, ROPE_FROM_SHIFTED, ROPE_INVERSE, ROPE_TO_SHIFTED, unigist_rope, unigist_attn_bwd_docs, unigist_attn_fwd_docs, unigist_docs_total_len,
                      unigist_docs_workspace_bytes, OP_BWD, OP_COMPACT, OP_FWD, PAGE_TOKENS, Problem, UnigistError,  # noqa: F401
                      unigist_attn_bwd, unigist_attn_fwd, unigist_cache_append, unigist_cache_state_bytes,
                      unigist_cache_state_init, unigist_compact_len, unigist_decode,
                      unigist_decode_static, unigist_decode_step, unigist_decode_workspace_bytes, unigist_device_status, unigist_selftest_wait_timeout, unigist_gist_shift, unigist_gist_unshift,
                      unigist_kernel_timing, unigist_kernel_timing_count,
                      unigist_kernel_timing_get, unigist_kv_compact, unigist_last_error_string, unigist_launch_count,
                      unigist_layout, unigist_prefill_chunk, unigist_prefill_workspace_bytes, unigist_total_len, unigist_visible_pairs, unigist_window_units,
                      unigist_workspace_bytes)
