// Shared declarations of the UniGist CUDA library: problem geometry in shifted coordinates,
// error reporting and launch bookkeeping.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "unigist.h"

namespace ug {

// Geometry of one sequence.  Shifted order = [sinks | raw | gists] (Section 4.2).
struct Geom {
  int s, T, r, k, n, N;  // k is clamped to n
  // Gist number of raw unit 0.  0 for a whole sequence.  In chunk-wise prefill (Section 4.3) the raw
  // segment holds only the units still in the cache plus the new chunk, while the gist segment holds
  // every gist so far: raw unit u then belongs to gist number u + uoff, and n = T / r + uoff.
  int uoff;
};

// Columns a query row may see, per segment, numbered inside the segment and inclusive
// (Eq. 3 rewritten for the shifted order).  hi < lo means "none".
struct RowIv {
  int hi_sink;  // sink columns [0, hi_sink]
  int lo_raw;   // raw columns [lo_raw, hi_raw]
  int hi_raw;
  int hi_gist;  // gist columns [0, hi_gist]
};

// Division of a non-negative int (< 2^31) by a divisor fixed on the host: n / d = (n * mul) >> sh with
// sh = 31 + ceil(log2 d) and mul = ceil(2^sh / d), exact for every such n.  A runtime integer division costs a
// few hundred clocks at the start of a block; this is one wide multiply and a shift.
struct FastDiv {
  uint32_t mul, sh;
};
inline FastDiv make_fastdiv(int d) {
  int s = 0;
  while ((1ll << s) < d) ++s;
  FastDiv f;
  f.sh = 31 + s;
  f.mul = (uint32_t)(((1ull << f.sh) + (unsigned long long)d - 1) / (unsigned long long)d);
  return f;
}
__host__ __device__ inline int fdiv(const FastDiv& f, int n) {
  return (int)(((unsigned long long)(unsigned)n * f.mul) >> f.sh);
}

// div_r(x) = x / g.r for x >= 0.
template <typename DivR>
__host__ __device__ inline RowIv row_intervals_with(const Geom& g, int sigma, DivR div_r) {
  RowIv v;
  if (sigma < g.s) {  // sink query: earlier sinks only
    v.hi_sink = sigma;
    v.lo_raw = 0;
    v.hi_raw = -1;
    v.hi_gist = -1;
  } else if (sigma < g.s + g.T) {  // raw query i of unit u
    const int i = sigma - g.s;
    const int u = div_r(i);
    const int u0 = u > g.k ? u - g.k : 0;
    v.hi_sink = g.s - 1;
    v.lo_raw = u0 * g.r;
    v.hi_raw = i;
    v.hi_gist = u + g.uoff - 1;
  } else {  // gist query: its own unit's raw tokens and itself
    const int ug = sigma - g.s - g.T;  // gist number
    const int u = ug - g.uoff;         // its raw unit inside the raw segment (>= 0 for every gist that is a query)
    const int u0 = u > g.k ? u - g.k : 0;
    v.hi_sink = g.s - 1;
    v.lo_raw = u0 * g.r;
    v.hi_raw = (u + 1) * g.r - 1;
    v.hi_gist = ug;
  }
  return v;
}
__host__ __device__ inline RowIv row_intervals(const Geom& g, int sigma) {
  return row_intervals_with(g, sigma, [&](int x) { return x / g.r; });
}

__host__ __device__ inline bool visible(const Geom& g, const RowIv& v, int col_sigma) {
  if (col_sigma < g.s) return col_sigma <= v.hi_sink;
  if (col_sigma < g.s + g.T) {
    const int j = col_sigma - g.s;
    return j >= v.lo_raw && j <= v.hi_raw;
  }
  return col_sigma - g.s - g.T <= v.hi_gist;
}

// Interleaved index of the token at shifted position sigma, and the inverse.
__host__ __device__ inline int shift_perm(const Geom& g, int sigma) {
  if (sigma < g.s) return sigma;
  if (sigma < g.s + g.T) {
    const int i = sigma - g.s;
    return g.s + i + i / g.r;
  }
  const int u = sigma - g.s - g.T;
  return g.s + u * (g.r + 1) + g.r;
}
__host__ __device__ inline int unshift_perm(const Geom& g, int t) {
  if (t < g.s) return t;
  const int q = t - g.s;
  const int u = q / (g.r + 1), p = q % (g.r + 1);
  return p == g.r ? g.s + g.T + u : g.s + u * g.r + p;
}

// Row of a [B, N, H, D] tensor that holds row `row` of a segment: in shifted order, or in
// interleaved order (Eq. 2) when the caller's tensors were never shifted.
// The three segments of the shifted order.
enum { kSegSink = 0, kSegRaw = 1, kSegGist = 2 };
__host__ __device__ inline int seg_len(const Geom& g, int seg) { return seg == kSegRaw ? g.T : (seg == kSegGist ? g.n : g.s); }
__host__ __device__ inline int seg_base(const Geom& g, int seg) {  // shifted position of the segment's row 0
  return seg == kSegRaw ? g.s : (seg == kSegGist ? g.s + g.T : 0);
}
__host__ __device__ inline int seg_row_to_token(const Geom& g, bool interleaved, int seg, int row) {
  if (!interleaved || seg == kSegSink) return seg_base(g, seg) + row;
  return seg == kSegRaw ? g.s + row + row / g.r : g.s + row * (g.r + 1) + g.r;
}

// Host side helpers (api.cu).
int32_t fail(int32_t code, const char* fmt, ...);
int32_t check_problem(const unigist_problem* p, Geom* g, float* scale);
int32_t check_launch(const char* what);
int32_t check_interleaved(const unigist_problem* p, const Geom& g);
void count_launch(int n = 1);
// Streaming multiprocessors of the current device (asked once per device); 148, the B200's count, when no
// device can be asked (a size query on a machine without a GPU).
int sm_count();
// Bytes of L2 cache of the current device (asked once per device); 126 MB, the B200's, when no device can be asked.
size_t l2_bytes();
// Records a CUDA event before and after the kernels launched in its scope when per-kernel
// timing is switched on; also counts the launch.
struct KernelScope {
  KernelScope(const char* name, cudaStream_t st);
  ~KernelScope();
  int slot;
  cudaStream_t st;
};
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Kernel launchers (one per .cu file).
int32_t launch_layout(const Geom& g, int32_t* sp, int32_t* up, int32_t* pos, cudaStream_t st);
int32_t launch_rope(const Geom& g, int B, int heads, int D, float theta_base, bool to_shifted, bool from_shifted,
                    bool inverse, const void* src, void* dst, cudaStream_t st);
int32_t launch_shift(const Geom& g, int B, const void* src, void* dst, size_t row_bytes,
                     bool inverse, cudaStream_t st);
// Where the query rows of a forward call sit.  A whole-sequence call has queries for every row
// (off = 0, out_base = the segments' shifted positions, n_out = N); a prefill chunk has queries only for
// the tail of each segment: query row j of segment sg is row off[sg] + j of that segment, and its
// output goes to token out_base[sg] + j of an [B, n_out, Hq, D] tensor.
struct QueryRows {
  int off[3], out_base[3], n_out;
};
int32_t launch_fwd_sm100(const Geom& g, const unigist_problem& p, float scale, const void* q,
                         const void* k, const void* v, void* o, float* lse, cudaStream_t st,
                         const QueryRows* chunk = nullptr);
// A run of `batch` consecutive sequences of one geometry inside packed [N_total, heads, D] tensors (a packed
// sample under cross-document masking), starting at packed row first_row.  The *_runs launchers take the
// tensors' base pointers and put up to twelve runs into one launch.
struct SeqRun {
  Geom g;
  int batch;
  long long first_row;
};
int32_t launch_fwd_sm100_runs(const SeqRun* runs, int n_runs, const unigist_problem& p, float scale, const void* q,
                              const void* k, const void* v, void* o, float* lse, cudaStream_t st);
int32_t fwd_sm100_take_timeout(bool* timed_out);
int32_t launch_bwd_sm100(const Geom& g, const unigist_problem& p, float scale, const void* q,
                         const void* k, const void* v, const void* o, const float* lse,
                         const void* d_o, void* dq, void* dk, void* dv, void* workspace,
                         cudaStream_t st);
// The same over a packed sample (head_dim 128; `runs` in token order, `tokens` = rows of the packed tensors).
int32_t launch_bwd_sm100_runs(const SeqRun* runs, int n_runs, long long tokens, const unigist_problem& p, float scale,
                              const void* q, const void* k, const void* v, const void* o, const float* lse,
                              const void* d_o, void* dq, void* dk, void* dv, void* workspace, cudaStream_t st);
// The fused backward serves head_dim 128 unless a fixed dQ summation order is asked for; otherwise two kernels.
inline bool bwd_is_fused(int D, uint32_t flags) { return D == 128 && !(flags & UNIGIST_FLAG_DETERMINISTIC_DQ); }
// Bytes of backward scratch for `tokens` packed tokens: Delta, the bf16 copy of an fp32 dO, and for the fused
// backward the fp32 dQ accumulator.
size_t bwd_scratch_bytes(long long tokens, int Hq, int D, bool dout_fp32, bool fused);
// Bytes behind that scratch for the fp32 partial dK / dV of the sink and gist key tiles whose walk over the
// queries is cut into chunks (0 where nothing is cut, or the backward is not the fused one), for `batch` sequences
// of geometry g.
size_t bwd_partial_bytes(const Geom& g, int batch, int Hq, int Hkv, bool fused);
int32_t bwd_sm100_take_timeout(bool* timed_out);
int32_t launch_compact_gather(const Geom& g, const unigist_problem& p, const void* k,
                              const void* v, void* kc, void* vc, int num_blocks,
                              const int32_t* table, int max_blocks, int32_t* seq_lens,
                              int32_t* kept_idx, cudaStream_t st);
int32_t launch_compact_inplace(const Geom& g, const unigist_problem& p, void* kc, void* vc,
                               int num_blocks, int32_t* table, int max_blocks, int32_t* seq_lens,
                               int32_t* kept_idx, void* ws, cudaStream_t st);
int32_t launch_decode(int S, int Hq, int Hkv, int D, float scale, const void* q, const void* kc,
                      const void* vc, int num_blocks, const int32_t* table, int max_blocks,
                      const int32_t* seq_lens, void* o, float* lse, void* ws, cudaStream_t st,
                      const int32_t* holes = nullptr, int holes_stride = 0, int holes_off = 0);
int32_t launch_prefill_chunk(const unigist_problem& p, const Geom& g_full, float scale, int u0, int c, const void* q,
                             const void* k, const void* v, void* kc, void* vc, int num_blocks, int32_t* table,
                             int max_blocks, int32_t* seq_lens, void* o, float* lse, void* workspace, cudaStream_t st);
size_t cache_state_bytes(int B, int r, int k);
void cache_state_layout(int r, int k, int* stride_ints, int* free_list_off);
int32_t launch_cache_state_init(const Geom& g, int B, int units_done, int32_t* state, cudaStream_t st);
int32_t launch_cache_append(const Geom& g, const unigist_problem& p, int is_gist, const void* k_new, const void* v_new,
                            void* kc, void* vc, int num_blocks, const int32_t* table, int max_blocks,
                            int32_t* seq_lens, int32_t* state, cudaStream_t st);
int decode_num_splits(int S, int Hkv, int max_blocks);
int32_t decode_take_timeout(bool* timed_out);
int32_t launch_selftest_wait(cudaStream_t st);
int32_t selftest_take_timeout(bool* timed_out);

}  // namespace ug
