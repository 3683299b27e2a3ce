/*
 * unigist.h -- C ABI of the UniGist gist-masked attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the attention operator of "UniGist: Towards General and
 * Hardware-aligned Sequence-level Long Context Compression" (arXiv 2509.15763):
 * one gist token is inserted after every r raw tokens (Eq. 2), every token attends to all
 * sinks, all earlier gists and the raw tokens of its own gist unit plus the k units before
 * it (Eq. 3), gists are moved to the right end of the sequence so the mask becomes
 * tile-aligned (Section 4.2, "gist shift trick"), and at inference raw tokens outside the
 * window are physically dropped from the KV cache (Section 4.3).
 *
 * Conventions that hold for every call
 *  - Indices are 0-based.  s = sinks, T = raw tokens, r = ratio, n = T / r gists,
 *    N = s + T + n.  The window is given as W raw tokens and means k = ceil(W / r)
 *    previous gist units.
 *  - "Interleaved" order is Eq. 2's Z.  "Shifted" order is [sinks | raw | gists], each kind
 *    in its original order.  Attention calls take SHIFTED tensors.
 *  - Dense tensors are [batch, N, heads, head_dim], head_dim contiguous, bf16 unless stated,
 *    base pointers 16-byte aligned (the fp32 lse arrays: 4-byte).  Query head h uses KV head h / (Hq / Hkv).
 *  - Every pointer named "device" is memory of the current CUDA device; the CALLER owns every
 *    buffer, the library never allocates or frees device memory.  Scratch comes in through
 *    `workspace` (size from unigist_workspace_bytes / unigist_decode_workspace_bytes).
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls only enqueue
 *    work; they do not synchronise.
 *  - Return value: UNIGIST_OK or an error code; nothing is launched when arguments are
 *    rejected.  unigist_last_error_string() describes the last failure of the calling thread.
 *  - There is no CPU fallback: without a CUDA device the compute entry points return
 *    UNIGIST_ERR_CUDA.
 */
#ifndef UNIGIST_H_
#define UNIGIST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  UNIGIST_OK = 0,
  UNIGIST_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad enum */
  UNIGIST_ERR_SHAPE = 2,       /* T % r != 0, Hq % Hkv != 0, unsupported head_dim ... */
  UNIGIST_ERR_ALIGNMENT = 3,   /* pointer or row size not 16-byte aligned */
  UNIGIST_ERR_WORKSPACE = 4,   /* workspace missing or too small */
  UNIGIST_ERR_UNSUPPORTED = 5,
  UNIGIST_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed */
  UNIGIST_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up */
} unigist_status;

/* dO passed to unigist_attn_bwd is fp32 (rounded to bf16 when it is read). */
#define UNIGIST_FLAG_DOUT_FP32 1u

/*
 * q, k, v, o, d_o, dq, dk, dv of unigist_attn_fwd / unigist_attn_bwd are in INTERLEAVED order (Eq. 2)
 * instead of shifted order: the gist shift of Section 4.2 then happens inside the tile addressing of
 * the loads (a raw tile is r rows of each of 128 / r consecutive gist units, a gist tile is one row per
 * unit) and outputs are stored at their interleaved row, so no separate shift / unshift pass is needed.
 * lse stays in shifted order (it is the tensor the backward reads back).  Supported when ratio divides
 * 128 and head_dim is 128; otherwise the calls return UNIGIST_ERR_UNSUPPORTED and the caller uses
 * unigist_gist_shift / unigist_gist_unshift.
 */
#define UNIGIST_FLAG_INTERLEAVED 2u

/*
 * unigist_attn_bwd / unigist_attn_bwd_docs with head_dim 128: dq, too, is the same bit for bit from run to run.
 * dQ of a query tile is then summed in tensor memory by ONE thread block that walks the tile's keys (a second
 * kernel that recomputes S and dP: seven matrix products per tile pair instead of five, 1.5 to 2 times the time)
 * instead of being reduced into memory in the order in which key tiles' blocks arrive.  No effect for head_dim 64,
 * whose backward always works this way.  The workspace then holds no fp32 accumulator (the size queries follow the
 * flag).  Not together with UNIGIST_FLAG_INTERLEAVED (UNIGIST_ERR_UNSUPPORTED).
 */
#define UNIGIST_FLAG_DETERMINISTIC_DQ 4u

enum { UNIGIST_PAGE_TOKENS = 64 }; /* tokens per KV-cache block */

typedef enum {
  UNIGIST_OP_FWD = 0,
  UNIGIST_OP_BWD = 1,
  UNIGIST_OP_COMPACT = 2
} unigist_op;

/* Problem statement of Section 4.1: (s, T, r, window) plus the attention shape. */
typedef struct {
  int32_t batch;        /* B >= 1; B and Hq at most 65535 */
  int32_t raw_len;      /* T, multiple of ratio */
  int32_t num_sinks;    /* s >= 0 */
  int32_t ratio;        /* r >= 1 */
  int32_t window;       /* W >= 0 raw tokens; k = ceil(W / r) */
  int32_t num_q_heads;  /* Hq */
  int32_t num_kv_heads; /* Hkv, divides Hq */
  int32_t head_dim;     /* D: 64 or 128 */
  float softmax_scale;  /* 0 => 1 / sqrt(D) */
  uint32_t flags;       /* UNIGIST_FLAG_* */
} unigist_problem;

/* Eq. 2: N = s + T + T / r.  Negative on a malformed problem. */
int32_t unigist_total_len(const unigist_problem* p);
/* Text after Eq. 3: number k of previous gist units in the local window, ceil(W / r). */
int32_t unigist_window_units(const unigist_problem* p);
/* Tokens left in the cache after compaction: s + n + min(k, n) * r (Section 4.3). */
int32_t unigist_compact_len(const unigist_problem* p);
/* Number of visible (query, key) pairs per head under Eq. 3; what "unmasked FLOPs" counts. */
int64_t unigist_visible_pairs(const unigist_problem* p);
/* Bytes of device scratch the given op needs for this problem (0 on a malformed problem). */
size_t unigist_workspace_bytes(const unigist_problem* p, int32_t op);

/*
 * Gist shift index arrays (Section 4.2; the "original token indexes" the kernel design
 * passes along).  shift_perm[sigma] = interleaved index of the token at shifted position
 * sigma; unshift_perm = inverse; pos_ids[t] (interleaved order) = position id with each gist
 * taking the id of the raw token right after it (Section 4.1, step 3).
 * Each array has N int32 entries and may be NULL.  on_device = 0: host pointers, computed on
 * the host, stream ignored.  on_device = 1: device pointers, filled by a kernel on `stream`.
 */
int32_t unigist_layout(const unigist_problem* p, int32_t* shift_perm, int32_t* unshift_perm,
                       int32_t* pos_ids, int32_t on_device, void* stream);

/*
 * Gist shift / unshift of a [B, N, heads, D] device tensor with elements of elem_bytes
 * (2 or 4) bytes (Section 4.2): dst[b, sigma] = src[b, shift_perm[sigma]] (shift) and
 * dst[b, t] = src[b, unshift_perm[t]] (unshift).  src and dst must not overlap;
 * heads * D * elem_bytes must be a multiple of 16.
 */
int32_t unigist_gist_shift(const unigist_problem* p, const void* src, void* dst, int32_t heads,
                           int32_t elem_bytes, void* stream);
int32_t unigist_gist_unshift(const unigist_problem* p, const void* src, void* dst, int32_t heads,
                             int32_t elem_bytes, void* stream);

/*
 * Position-encoding alignment (Section 4.1, step 3) applied as a rotary embedding to a bf16
 * [B, N, heads, D] device tensor (INTERLEAVED order unless a flag says otherwise): token t is rotated by its aligned position id
 * (sinks and raw tokens count 0, 1, 2, ...; a gist takes the id of the raw token right after it, the
 * last gist the id one past the last raw token), so distances between raw tokens are those of the
 * sequence without gists.  The paper fixes the ids, not the rotary convention; this is the one of the
 * Llama models it trains: feature j < D / 2 pairs with feature j + D / 2 and the pair turns by
 * id * theta_base^(-2 j / D).  Angles are formed in fp64, the rotation in fp32, one rounding to bf16.
 * flags (a combination):
 *   UNIGIST_ROPE_TO_SHIFTED    dst is written in SHIFTED order (Section 4.2): the rotation fused with
 *                              unigist_gist_shift;
 *   UNIGIST_ROPE_FROM_SHIFTED  src is in SHIFTED order (with both flags the tensor stays shifted; with this one
 *                              alone the rotation is fused with unigist_gist_unshift);
 *   UNIGIST_ROPE_INVERSE       rotate by the negative angle: the transpose of the rotation, which is what the
 *                              backward pass applies to the gradient of a rotated tensor.
 * Where src and dst have the same order, dst == src (in place) is allowed; otherwise they must not overlap.
 * Errors: INVALID_ARG (NULL, heads < 1, theta_base <= 1, unknown flag, overlap), ALIGNMENT, CUDA.
 */
#define UNIGIST_ROPE_TO_SHIFTED 1u
#define UNIGIST_ROPE_FROM_SHIFTED 2u
#define UNIGIST_ROPE_INVERSE 4u
int32_t unigist_rope(const unigist_problem* p, const void* src, void* dst, int32_t heads, float theta_base,
                     uint32_t flags, void* stream);

/*
 * Forward (Section 4.2 kernel; Eq. 3 mask): for each (b, head, row t)
 *   S_tj = scale * q_t . k_j over visible j,  LSE_t = log sum_j exp(S_tj),  O_t = softmax(S_t) V.
 * q [B,N,Hq,D], k, v [B,N,Hkv,D], o [B,N,Hq,D]: device bf16, SHIFTED order.
 * lse [B,Hq,N]: device fp32, natural log, shifted order.  Masked-out tiles are never read.
 * The forward needs no scratch: workspace may be NULL with ws_bytes 0 (unigist_workspace_bytes(p, UNIGIST_OP_FWD) is 0).
 */
int32_t unigist_attn_fwd(const unigist_problem* p, const void* q, const void* k, const void* v,
                         void* o, float* lse, void* workspace, size_t ws_bytes, void* stream);

/*
 * Backward of the forward above (the paper's backward kernel, Appendix speed-up table):
 *   Delta = rowsum(dO o O), P = exp(S - LSE), dV = P^T dO, dP = dO V^T, dS = P o (dP - Delta),
 *   dQ = scale dS K, dK = scale dS^T Q;  dK, dV summed over the query heads of a KV head.
 * q, k, v, o, lse as in the forward; d_o [B,N,Hq,D] device bf16 (fp32 with
 * UNIGIST_FLAG_DOUT_FP32); dq [B,N,Hq,D], dk, dv [B,N,Hkv,D] device bf16, all shifted.
 * dK/dV are accumulated without atomics: a key tile is owned by one thread block, or, where very many queries see
 * it (sink and gist keys of a long sequence), by one block per chunk of those queries whose fp32 partial sums a
 * small kernel adds in chunk order; either way they are the same bit for bit from run to run.  For head_dim 128
 * dQ is the sum, over the key tiles that see a query tile, of fp32 partial tiles reduced into the workspace in
 * whatever order the blocks arrive: its last bit may differ between runs (UNIGIST_FLAG_DETERMINISTIC_DQ trades
 * speed for a fixed order).  workspace:
 * unigist_workspace_bytes(p, UNIGIST_OP_BWD) bytes (Delta, a bf16 copy of an fp32 dO, and for head_dim 128 the
 * fp32 dQ accumulator and the chunks' partial dK / dV), 16-byte aligned.
 */
int32_t unigist_attn_bwd(const unigist_problem* p, const void* q, const void* k, const void* v,
                         const void* o, const float* lse, const void* d_o, void* dq, void* dk,
                         void* dv, void* workspace, size_t ws_bytes, void* stream);

/*
 * Cross-document masking (the training set-up of Section 5.1; every document of a packed sample is padded to a
 * multiple of the ratio, Appendix "Training Data Processing"): attention is blocked across document
 * boundaries and every document restarts its sinks, gist units and window, so a packed sample is a list of
 * independent sequences.  doc_raw_len (HOST pointer, num_docs entries) gives each document's raw length T_d, a
 * multiple of ratio; p->batch must be 1 and p->raw_len is ignored.  Tensors are [N_total, heads, D] device
 * tensors with N_total = sum_d (s + T_d + T_d / r) rows: document d owns the rows from the sum of the earlier
 * documents' lengths on, in shifted order inside its block (interleaved with UNIGIST_FLAG_INTERLEAVED).
 * lse holds one [Hq, N_d] block per document (shifted order), document d's block starting at float
 * Hq * (first row of d).  Consecutive documents of equal length form one launch unit (a batch); up to twelve
 * units, of equal or different lengths, share ONE launch of each kernel (every thread block finds its document
 * from its block index; the units' tensor maps travel as kernel parameters), a sample with more units takes one
 * launch per twelve.  Everything is enqueued on `stream`.  For head_dim 64 the backward runs its two kernels once
 * per unit.  workspace (backward only): unigist_docs_workspace_bytes bytes.
 * Errors as for unigist_attn_fwd / unigist_attn_bwd, raised before the first launch where the list is malformed.
 */
int64_t unigist_docs_total_len(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len);
size_t unigist_docs_workspace_bytes(const unigist_problem* p, int32_t op, int32_t num_docs, const int32_t* doc_raw_len);
int32_t unigist_attn_fwd_docs(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len, const void* q,
                              const void* k, const void* v, void* o, float* lse, void* workspace, size_t ws_bytes,
                              void* stream);
int32_t unigist_attn_bwd_docs(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len, const void* q,
                              const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
                              void* dk, void* dv, void* workspace, size_t ws_bytes, void* stream);

/*
 * KV compaction (Section 4.3): after the last gist of a T-token prefix, keep the sinks, all n
 * gists and the raw tokens of the last min(k, n) units; every other raw token is dropped.
 * Cache order is [sinks | gists | window raw]; L = unigist_compact_len().
 * The cache is paged: k_cache, v_cache [num_blocks, Hkv, 64, D] device bf16;
 * block_table [B, max_blocks_per_seq] device int32 maps logical block -> physical block.
 *
 *  k, v != NULL: gather from the shifted tensors k, v [B,N,Hkv,D] (interleaved tensors with
 *      UNIGIST_FLAG_INTERLEAVED, for any s and r) into the pages named by the first ceil(L / 64)
 *      entries of each block_table row (read only).
 *  k == v == NULL: compact IN PLACE a paged cache that holds the whole shifted sequence
 *      (logical position = shifted position; the first ceil(N / 64) entries of each row are
 *      valid and distinct).  The row is rewritten: entries [0, ceil(L/64)) are the compacted
 *      cache, entries [ceil(L/64), ceil(N/64)) list the freed physical blocks.  When
 *      s, T, n and T - min(k,n)*r are multiples of 64 this is a block-table edit and no token
 *      moves; otherwise kept tokens are staged through `workspace`
 *      (unigist_workspace_bytes(p, UNIGIST_OP_COMPACT)).
 * seq_lens [B] device int32 receives L.  kept_idx (nullable) [B, L] device int32 receives the
 * SHIFTED position each cache entry came from.
 */
int32_t unigist_kv_compact(const unigist_problem* p, const void* k, const void* v, void* k_cache,
                           void* v_cache, int32_t num_blocks, int32_t* block_table,
                           int32_t max_blocks_per_seq, int32_t* seq_lens, int32_t* kept_idx,
                           void* workspace, size_t ws_bytes, void* stream);

/*
 * Chunk-wise prefill (Section 4.3: "re-adopt the chunk-wise scheme and encode each chunk with our kernel").
 * The prompt of p->raw_len raw tokens is fed in chunks of whole gist units; the chunk of unit_count units
 * that starts at unit unit_begin attends to what the paged cache holds -- the sinks, the gists of units
 * [0, unit_begin) and the raw tokens of the last min(k, unit_begin) units, in the cache order of
 * unigist_kv_compact -- and to itself under Eq. 3; its outputs equal the corresponding rows of the one-pass
 * forward over the whole prompt.  Afterwards the cache holds the state after unit_begin + unit_count units
 * (seq_lens updated), ready for the next chunk or for unigist_decode.
 *
 * q [B, Nc, Hq, D], k, v [B, Nc, Hkv, D], o [B, Nc, Hq, D] device bf16, lse [B, Hq, Nc] device fp32: the
 * chunk's own tokens in shifted CHUNK order [sinks (only when unit_begin == 0) | unit_count * r raw |
 * unit_count gists], Nc = that many rows.  k_cache, v_cache, block_table, seq_lens as in unigist_kv_compact;
 * for unit_begin > 0 the cache must be in the state a previous chunk (or unigist_kv_compact of the first
 * unit_begin units) left it in.  block_table needs entries for the cache after the chunk.
 * workspace: unigist_prefill_workspace_bytes() bytes (a dense copy of the keys and values the chunk sees).
 */
size_t unigist_prefill_workspace_bytes(const unigist_problem* p, int32_t unit_begin, int32_t unit_count);
int32_t unigist_prefill_chunk(const unigist_problem* p, int32_t unit_begin, int32_t unit_count, const void* q,
                              const void* k, const void* v, void* k_cache, void* v_cache, int32_t num_blocks,
                              int32_t* block_table, int32_t max_blocks_per_seq, int32_t* seq_lens, void* o, float* lse,
                              void* workspace, size_t ws_bytes, void* stream);

/*
 * Cache maintenance while decoding (Section 4.3: raw tokens outside the local window "can be safely discarded
 * at each compression point").  The sequence grows token by token: r raw tokens, then their gist, and so on.
 * unigist_cache_append writes one new token's K / V rows (k_new, v_new [B, Hkv, D] device bf16) into every
 * sequence's cache.  A gist (is_gist = 1, after exactly r raw tokens) still attends to the k + 1 units of the
 * window; the first raw token after it (is_gist = 0) opens a new unit, at which point the oldest unit's r
 * raw tokens are seen by no one any more: their slots are freed and reused by the new unit's raw tokens.
 * No entry ever moves; the cache occupies slots [0, seq_lens[b]) in an order that becomes arbitrary (attention
 * does not care), grows by one slot per gist unit, and after every append its live slots hold exactly the
 * tokens the new token sees.  p->raw_len is not used as a bound here.
 *
 * state: unigist_cache_state_bytes(p) bytes of device memory owned by the caller; unigist_cache_state_init
 * sets it up for caches in the order unigist_kv_compact / unigist_prefill_chunk leave them in after
 * units_done whole units (0 with an empty or sinks-only cache).  Misuse (a gist before its unit is
 * complete, a raw token after it, a block table that is too short) sets state[b * ints + 4] != 0 and
 * leaves the cache, seq_lens and the rest of the state unchanged.
 *
 * Between the first raw token of a unit and its last, up to r - 1 freed slots inside [0, seq_lens[b]) still
 * hold the evicted tokens; unigist_decode_step is unigist_decode (one query per sequence, p->batch sequences,
 * shapes and scale from p) that leaves those slots, listed in `state`, out of the attention.  Use it for
 * every query of a loop that maintains its cache with unigist_cache_append.
 */
size_t unigist_cache_state_bytes(const unigist_problem* p);
int32_t unigist_cache_state_init(const unigist_problem* p, int32_t units_done, int32_t* state, void* stream);
int32_t unigist_cache_append(const unigist_problem* p, const void* k_new, const void* v_new, int32_t is_gist,
                             void* k_cache, void* v_cache, int32_t num_blocks, const int32_t* block_table,
                             int32_t max_blocks_per_seq, int32_t* seq_lens, int32_t* state, void* stream);
int32_t unigist_decode_step(const unigist_problem* p, const void* q, const void* k_cache, const void* v_cache,
                            int32_t num_blocks, const int32_t* block_table, int32_t max_blocks_per_seq,
                            const int32_t* seq_lens, const int32_t* state, void* o, float* lse, void* workspace,
                            size_t ws_bytes, void* stream);

/* Scratch for unigist_decode (split-KV partial results). */
size_t unigist_decode_workspace_bytes(int32_t num_seqs, int32_t num_q_heads, int32_t num_kv_heads,
                                      int32_t head_dim, int32_t max_blocks_per_seq);

/*
 * Decode over the compressed cache (Section 4.3; FlashDecoding-style split over keys): one
 * query per sequence attends to ALL seq_lens[i] cache entries (what is left in a compacted
 * cache is visible by construction; the caller appends the new token's K/V first).
 * q, o [num_seqs, Hq, D] device bf16; k_cache, v_cache [num_blocks, Hkv, 64, D] device bf16;
 * block_table [num_seqs, max_blocks_per_seq], seq_lens [num_seqs] device int32 (>= 0);
 * lse [num_seqs, Hq] device fp32, nullable.  head_dim must be 128, Hq / Hkv at most 8, num_seqs at most 65535.
 * A sequence with nothing to attend to (length 0: a padding slot of the batch) gets O = 0 and LSE = -inf.
 */
int32_t unigist_decode(int32_t num_seqs, int32_t num_q_heads, int32_t num_kv_heads,
                       int32_t head_dim, float softmax_scale, const void* q, const void* k_cache,
                       const void* v_cache, int32_t num_blocks, const int32_t* block_table,
                       int32_t max_blocks_per_seq, const int32_t* seq_lens, void* o, float* lse,
                       void* workspace, size_t ws_bytes, void* stream);

/*
 * Measurement aid (no counterpart in the paper): per-kernel device times.
 * unigist_kernel_timing(1) clears the record list and makes every later kernel launch of the
 * library record a CUDA event before and after itself on its stream (at most 4096 launches are
 * kept); unigist_kernel_timing(0) stops recording.  unigist_kernel_timing_count() returns the
 * number of recorded launches; unigist_kernel_timing_get(i, name, cap, &ms) waits for launch i
 * to finish and returns its kernel name (copied into name[cap]) and duration in milliseconds.
 * Not thread safe; meant for benchmarks.
 */
int32_t unigist_kernel_timing(int32_t enable);
int32_t unigist_kernel_timing_count(void);
int32_t unigist_kernel_timing_get(int32_t index, char* name, int32_t cap, float* ms);

/*
 * unigist_decode for callers that have no device memory to hand over as scratch and may not
 * allocate any.  (The paper has no counterpart; this exists for deployment.)  Typical cases: a
 * plugin called from inside an inference server that has already claimed the whole GPU for its
 * own memory pool, so a cudaMalloc from the plugin would fail or stall the device; or a decode
 * loop with a hard latency limit, where an allocation's implicit device-wide synchronisation is
 * not acceptable.
 *
 * Same arguments, same accepted shapes and bit-identical results as unigist_decode, minus workspace /
 * ws_bytes.  The split-KV
 * partial results are kept in a fixed array of UNIGIST_DECODE_STATIC_SCRATCH_BYTES bytes that is
 * part of the library image: every GPU that loads the library holds that much global memory
 * until the process exits.  The call allocates and frees nothing.
 *  - A problem whose unigist_decode_workspace_bytes() exceeds the array is rejected with
 *    UNIGIST_ERR_WORKSPACE before anything is launched (use unigist_decode, or fewer sequences).
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array.  Nothing in it has to start at zero (each call
 *    overwrites every slot it later reads), so back-to-back calls on one stream are fine, but two
 *    calls that may overlap on the GPU (different streams, different host threads) race on it
 *    and must be serialised by the caller.
 */
#define UNIGIST_DECODE_STATIC_SCRATCH_BYTES (8u << 20)
int32_t unigist_decode_static(int32_t num_seqs, int32_t num_q_heads, int32_t num_kv_heads,
                              int32_t head_dim, float softmax_scale, const void* q,
                              const void* k_cache, const void* v_cache, int32_t num_blocks,
                              const int32_t* block_table, int32_t max_blocks_per_seq,
                              const int32_t* seq_lens, void* o, float* lse, void* stream);

/*
 * Device-side waits in the tensor-core kernels (on TMA and MMA completion barriers) are bounded:
 * a wait that does not end within about a second of SM clock makes its thread block leave early
 * and raises a flag instead of hanging the GPU.  This call synchronises the current device, then
 * returns UNIGIST_ERR_TIMEOUT (and clears the flag) if any kernel gave up since the last call,
 * UNIGIST_OK otherwise.  No counterpart in the paper.
 */
int32_t unigist_device_status(void);

/*
 * Self-check of that mechanism (no counterpart in the paper): enqueues one small thread block that waits on a
 * barrier nothing ever completes.  Its wait runs out after about a second, the block leaves the way the
 * attention kernels leave after a wait that gave up (tensor memory freed, flag raised), and the next
 * unigist_device_status() returns UNIGIST_ERR_TIMEOUT once; the device stays usable.  Nothing faults or hangs.
 */
int32_t unigist_selftest_wait_timeout(void* stream);

/* Number of kernels the library has launched in this process (all threads). */
int64_t unigist_launch_count(void);

/* Message for the last non-OK status returned to the calling thread ("" if none). */
const char* unigist_last_error_string(void);

#ifdef __cplusplus
}
#endif
#endif /* UNIGIST_H_ */
