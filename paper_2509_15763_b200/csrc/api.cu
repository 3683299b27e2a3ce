// C-ABI entry points: argument validation, error reporting, dispatch to the kernel launchers.
#include <algorithm>
#include <vector>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "ug_common.cuh"

namespace ug {

static thread_local char g_err[512] = "";
static std::atomic<int64_t> g_launches{0};

int32_t fail(int32_t code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int sm_count() {
  constexpr int kMaxDevices = 64, kB200 = 148;
  static std::atomic<int> cached[kMaxDevices];  // 0 = not asked yet
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();  // a size query on a machine without a GPU is not an error of the caller's
    return kB200;
  }
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
    cudaGetLastError();
    return kB200;
  }
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

size_t l2_bytes() {
  constexpr int kMaxDevices = 64;
  constexpr size_t kB200 = 126u << 20;
  static std::atomic<size_t> cached[kMaxDevices];  // 0 = not asked yet
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return kB200;
  }
  size_t n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  int v = 0;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, dev) != cudaSuccess || v < 1) {
    cudaGetLastError();
    return kB200;
  }
  cached[dev].store((size_t)v, std::memory_order_relaxed);
  return (size_t)v;
}

namespace {
struct TimingRecord {
  const char* name;
  cudaEvent_t e0, e1;
};
constexpr int kMaxRecords = 4096;
bool g_timing = false;
int g_num_records = 0;
TimingRecord g_records[kMaxRecords];
}  // namespace

KernelScope::KernelScope(const char* name, cudaStream_t stream) : slot(-1), st(stream) {
  count_launch();
  if (!g_timing || g_num_records >= kMaxRecords) return;
  TimingRecord& r = g_records[g_num_records];
  if (cudaEventCreate(&r.e0) != cudaSuccess) return;
  if (cudaEventCreate(&r.e1) != cudaSuccess) {
    cudaEventDestroy(r.e0);
    return;
  }
  r.name = name;
  slot = g_num_records++;
  cudaEventRecord(r.e0, st);
}

KernelScope::~KernelScope() {
  if (slot >= 0) cudaEventRecord(g_records[slot].e1, st);
}

int32_t check_launch(const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return UNIGIST_OK;
}

constexpr int kMaxGridYZ = 65535;

int32_t check_problem(const unigist_problem* p, Geom* g, float* scale) {
  if (!p) return fail(UNIGIST_ERR_INVALID_ARG, "problem is NULL");
  if (p->batch < 1 || p->raw_len < 1 || p->num_sinks < 0 || p->ratio < 1 || p->window < 0 ||
      p->num_q_heads < 1 || p->num_kv_heads < 1)
    return fail(UNIGIST_ERR_INVALID_ARG, "problem has a non-positive size");
  if (p->raw_len % p->ratio != 0)
    return fail(UNIGIST_ERR_SHAPE, "raw_len %d is not a multiple of ratio %d", p->raw_len,
                p->ratio);
  if (p->num_q_heads % p->num_kv_heads != 0)
    return fail(UNIGIST_ERR_SHAPE, "num_q_heads %d is not a multiple of num_kv_heads %d",
                p->num_q_heads, p->num_kv_heads);
  if (p->head_dim != 64 && p->head_dim != 128)
    return fail(UNIGIST_ERR_SHAPE, "head_dim %d is not 64 or 128", p->head_dim);
  // batch entries and heads are grid dimensions y / z of the kernels
  if (p->batch > kMaxGridYZ || p->num_q_heads > kMaxGridYZ)
    return fail(UNIGIST_ERR_SHAPE, "batch %d or num_q_heads %d exceeds %d", p->batch, p->num_q_heads, kMaxGridYZ);
  const int64_t n = p->raw_len / p->ratio;
  const int64_t N = (int64_t)p->num_sinks + p->raw_len + n;
  if (N > (int64_t)1 << 30) return fail(UNIGIST_ERR_SHAPE, "sequence too long");
  if (!(p->softmax_scale >= 0.f) || std::isinf(p->softmax_scale))
    return fail(UNIGIST_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0");
  if (g) {
    g->s = p->num_sinks;
    g->T = p->raw_len;
    g->r = p->ratio;
    g->n = (int)n;
    g->N = (int)N;
    const int64_t k = ((int64_t)p->window + p->ratio - 1) / p->ratio;
    g->k = (int)(k < n ? k : n);
    g->uoff = 0;
  }
  if (scale) *scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  return UNIGIST_OK;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// UNIGIST_FLAG_INTERLEAVED needs the tile addressing of the tensor-core kernels for head_dim 128.
int32_t check_interleaved(const unigist_problem* p, const Geom& g) {
  if (!(p->flags & UNIGIST_FLAG_INTERLEAVED)) return UNIGIST_OK;
  if (p->flags & UNIGIST_FLAG_DETERMINISTIC_DQ)
    return fail(UNIGIST_ERR_UNSUPPORTED,
                "UNIGIST_FLAG_DETERMINISTIC_DQ takes shifted tensors: its kernels do not address interleaved ones");
  if (p->head_dim != 128 || 128 % g.r != 0)
    return fail(UNIGIST_ERR_UNSUPPORTED,
                "interleaved tensors need head_dim 128 and a ratio that divides 128 (got D = %d, r = %d): "
                "shift the tensors with unigist_gist_shift instead",
                p->head_dim, g.r);
  return UNIGIST_OK;
}

}  // namespace ug

using namespace ug;

extern "C" {

int32_t unigist_total_len(const unigist_problem* p) {
  Geom g;
  if (check_problem(p, &g, nullptr) != UNIGIST_OK) return -1;
  return g.N;
}

int32_t unigist_window_units(const unigist_problem* p) {
  if (check_problem(p, nullptr, nullptr) != UNIGIST_OK) return -1;
  return (int32_t)(((int64_t)p->window + p->ratio - 1) / p->ratio);
}

int32_t unigist_compact_len(const unigist_problem* p) {
  Geom g;
  if (check_problem(p, &g, nullptr) != UNIGIST_OK) return -1;
  return g.s + g.n + g.k * g.r;
}

int64_t unigist_visible_pairs(const unigist_problem* p) {
  Geom g;
  if (check_problem(p, &g, nullptr) != UNIGIST_OK) return -1;
  // Row counts of Eq. 3 summed over sink, raw and gist queries.
  int64_t tot = (int64_t)g.s * (g.s + 1) / 2 + (int64_t)g.s * ((int64_t)g.T + g.n);
  const int64_t r = g.r;
  for (int64_t u = 0; u < g.n; ++u) {
    const int64_t w = u < g.k ? u : g.k;
    tot += r * r * w + r * (r + 1) / 2 + r * u;  // raw queries of unit u
    tot += (w + 1) * r + u + 1;                  // gist query u
  }
  return tot;
}

size_t unigist_workspace_bytes(const unigist_problem* p, int32_t op) {
  Geom g;
  if (check_problem(p, &g, nullptr) != UNIGIST_OK) return 0;
  switch (op) {
    case UNIGIST_OP_FWD:
      return 0;
    case UNIGIST_OP_BWD:
      // Delta [B,Hq,N] fp32, a bf16 copy of dO when it arrives as fp32, and for the fused tensor-core backward
      // the fp32 dQ accumulator and the chunks' partial dK / dV
      return bwd_scratch_bytes((long long)p->batch * g.N, p->num_q_heads, p->head_dim,
                               (p->flags & UNIGIST_FLAG_DOUT_FP32) != 0, bwd_is_fused(p->head_dim, p->flags)) +
             bwd_partial_bytes(g, p->batch, p->num_q_heads, p->num_kv_heads, bwd_is_fused(p->head_dim, p->flags));
    case UNIGIST_OP_COMPACT: {
      const size_t L = (size_t)g.s + g.n + (size_t)g.k * g.r;
      return align_up(2 * (size_t)p->batch * L * p->num_kv_heads * p->head_dim * 2, 256);
    }
    default:
      return 0;
  }
}

int32_t unigist_layout(const unigist_problem* p, int32_t* sp, int32_t* up, int32_t* pos,
                       int32_t on_device, void* stream) {
  Geom g;
  if (int32_t rc = check_problem(p, &g, nullptr)) return rc;
  if (!on_device) {
    for (int i = 0; i < g.N; ++i) {
      if (sp) sp[i] = shift_perm(g, i);
      if (up) up[i] = unshift_perm(g, i);
      if (pos) {  // i is an interleaved index here
        const int sig = unshift_perm(g, i);
        pos[i] = sig < g.s + g.T ? sig : g.s + (sig - g.s - g.T + 1) * g.r;
      }
    }
    return UNIGIST_OK;
  }
  return launch_layout(g, sp, up, pos, (cudaStream_t)stream);
}

static int32_t shift_common(const unigist_problem* p, const void* src, void* dst, int32_t heads,
                            int32_t elem_bytes, void* stream, bool inverse) {
  Geom g;
  if (int32_t rc = check_problem(p, &g, nullptr)) return rc;
  if (!src || !dst) return fail(UNIGIST_ERR_INVALID_ARG, "src/dst is NULL");
  if (heads < 1 || (elem_bytes != 2 && elem_bytes != 4))
    return fail(UNIGIST_ERR_INVALID_ARG, "heads must be >= 1 and elem_bytes 2 or 4");
  const size_t row = (size_t)heads * p->head_dim * elem_bytes;
  if (row % 16 || !aligned16(src) || !aligned16(dst))
    return fail(UNIGIST_ERR_ALIGNMENT, "rows and pointers must be 16-byte aligned");
  const char* a = (const char*)src;
  const char* b = (const char*)dst;
  const size_t tot = row * g.N * p->batch;
  if (a < b + tot && b < a + tot) return fail(UNIGIST_ERR_INVALID_ARG, "src and dst overlap");
  return launch_shift(g, p->batch, src, dst, row, inverse, (cudaStream_t)stream);
}

int32_t unigist_gist_shift(const unigist_problem* p, const void* src, void* dst, int32_t heads,
                           int32_t elem_bytes, void* stream) {
  return shift_common(p, src, dst, heads, elem_bytes, stream, false);
}
int32_t unigist_gist_unshift(const unigist_problem* p, const void* src, void* dst, int32_t heads,
                             int32_t elem_bytes, void* stream) {
  return shift_common(p, src, dst, heads, elem_bytes, stream, true);
}

int32_t unigist_rope(const unigist_problem* p, const void* src, void* dst, int32_t heads, float theta_base,
                     uint32_t flags, void* stream) {
  Geom g;
  if (int32_t rc = check_problem(p, &g, nullptr)) return rc;
  if (!src || !dst) return fail(UNIGIST_ERR_INVALID_ARG, "src/dst is NULL");
  if (heads < 1 || !(theta_base > 1.f) || (flags & ~(UNIGIST_ROPE_TO_SHIFTED | UNIGIST_ROPE_FROM_SHIFTED | UNIGIST_ROPE_INVERSE)))
    return fail(UNIGIST_ERR_INVALID_ARG, "heads must be >= 1, theta_base > 1, flags a combination of UNIGIST_ROPE_*");
  if (!aligned16(src) || !aligned16(dst)) return fail(UNIGIST_ERR_ALIGNMENT, "pointers must be 16-byte aligned");
  const bool to_shifted = (flags & UNIGIST_ROPE_TO_SHIFTED) != 0, from_shifted = (flags & UNIGIST_ROPE_FROM_SHIFTED) != 0;
  const bool same_order = to_shifted == from_shifted;  // a row is read and written at the same place
  const char* a = (const char*)src;
  const char* b = (const char*)dst;
  const size_t tot = (size_t)heads * p->head_dim * 2 * g.N * p->batch;
  if ((!same_order || a != b) && a < b + tot && b < a + tot)
    return fail(UNIGIST_ERR_INVALID_ARG, "src and dst overlap (in place is allowed only where the order does not change)");
  return launch_rope(g, p->batch, heads, p->head_dim, theta_base, to_shifted, from_shifted,
                     (flags & UNIGIST_ROPE_INVERSE) != 0, src, dst, (cudaStream_t)stream);
}

int32_t unigist_attn_fwd(const unigist_problem* p, const void* q, const void* k, const void* v,
                         void* o, float* lse, void* workspace, size_t ws_bytes, void* stream) {
  Geom g;
  float scale;
  if (int32_t rc = check_problem(p, &g, &scale)) return rc;
  (void)workspace;
  (void)ws_bytes;
  if (!q || !k || !v || !o || !lse) return fail(UNIGIST_ERR_INVALID_ARG, "a tensor is NULL");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || (reinterpret_cast<uintptr_t>(lse) & 3))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned (lse: 4-byte)");
  if (int32_t rc = check_interleaved(p, g)) return rc;
  return launch_fwd_sm100(g, *p, scale, q, k, v, o, lse, (cudaStream_t)stream);
}

int32_t unigist_device_status(void) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaDeviceSynchronize: %s", cudaGetErrorString(e));
  bool timed_out = false;
  bool bwd_timed_out = false;
  if (int32_t rc = fwd_sm100_take_timeout(&timed_out)) return rc;
  if (int32_t rc = bwd_sm100_take_timeout(&bwd_timed_out)) return rc;
  bool dec_timed_out = false;
  if (int32_t rc = decode_take_timeout(&dec_timed_out)) return rc;
  bool self_timed_out = false;
  if (int32_t rc = selftest_take_timeout(&self_timed_out)) return rc;
  if (timed_out || bwd_timed_out || dec_timed_out || self_timed_out) return fail(UNIGIST_ERR_TIMEOUT, "a kernel gave up on a bounded wait; its outputs are invalid");
  return UNIGIST_OK;
}

int32_t unigist_attn_bwd(const unigist_problem* p, const void* q, const void* k, const void* v,
                         const void* o, const float* lse, const void* d_o, void* dq, void* dk,
                         void* dv, void* workspace, size_t ws_bytes, void* stream) {
  Geom g;
  float scale;
  if (int32_t rc = check_problem(p, &g, &scale)) return rc;
  if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv)
    return fail(UNIGIST_ERR_INVALID_ARG, "a tensor is NULL");
  const void* ptrs[] = {q, k, v, o, d_o, dq, dk, dv, workspace};
  for (const void* x : ptrs)
    if (!aligned16(x)) return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(lse) & 3) return fail(UNIGIST_ERR_ALIGNMENT, "lse must be 4-byte aligned");
  if (int32_t rc = check_interleaved(p, g)) return rc;
  const size_t need = unigist_workspace_bytes(p, UNIGIST_OP_BWD);
  if (!workspace || ws_bytes < need)
    return fail(UNIGIST_ERR_WORKSPACE, "backward needs %zu bytes of workspace, got %zu", need,
                ws_bytes);
  // the fused kernel for head_dim 128, the two-kernel path for head_dim 64; both on the tensor cores
  return launch_bwd_sm100(g, *p, scale, q, k, v, o, lse, d_o, dq, dk, dv, workspace, (cudaStream_t)stream);
}

// ---- cross-document masking: a packed sample is a list of independent sequences -------------------------------

extern "C++" {
namespace {

// Checks the document list; fills the problem of a run of `count` equal documents starting at doc `first`.
int32_t check_docs(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len) {
  if (!p || !doc_raw_len || num_docs < 1) return fail(UNIGIST_ERR_INVALID_ARG, "document list is NULL or empty");
  if (p->batch != 1) return fail(UNIGIST_ERR_INVALID_ARG, "a packed sample has batch 1 (append the documents of more samples to the list)");
  for (int32_t d = 0; d < num_docs; ++d) {
    unigist_problem one = *p;
    one.raw_len = doc_raw_len[d];
    if (int32_t rc = check_problem(&one, nullptr, nullptr)) return rc;
  }
  return UNIGIST_OK;
}

// Calls fn(problem of the run, first token row of the run, index of the run) for every run of consecutive
// documents of equal length.
template <typename Fn>
int32_t for_each_doc_run(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len, Fn fn) {
  int64_t base = 0;
  int32_t index = 0;
  for (int32_t d = 0; d < num_docs; ++index) {
    int32_t e = d + 1;
    while (e < num_docs && doc_raw_len[e] == doc_raw_len[d]) ++e;
    unigist_problem run = *p;
    run.raw_len = doc_raw_len[d];
    run.batch = e - d;
    const int64_t n_doc = (int64_t)run.num_sinks + run.raw_len + run.raw_len / run.ratio;
    if (int32_t rc = fn(run, base, index)) return rc;
    base += n_doc * run.batch;
    d = e;
  }
  return UNIGIST_OK;
}

// The runs of a packed sample as launch units, in token order.
int32_t doc_runs(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len, std::vector<SeqRun>* out,
                 int64_t* tokens) {
  out->clear();
  int64_t end = 0;
  int32_t rc = for_each_doc_run(p, num_docs, doc_raw_len, [&](const unigist_problem& run, int64_t base, int32_t) {
    SeqRun r;
    if (int32_t e = check_problem(&run, &r.g, nullptr)) return e;
    r.batch = run.batch;
    r.first_row = base;
    out->push_back(r);
    end = base + (int64_t)r.g.N * r.batch;
    return (int32_t)UNIGIST_OK;
  });
  *tokens = end;
  return rc;
}

}  // namespace
}  // extern "C++"

int64_t unigist_docs_total_len(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len) {
  if (check_docs(p, num_docs, doc_raw_len) != UNIGIST_OK) return -1;
  int64_t tot = 0;
  for (int32_t d = 0; d < num_docs; ++d) tot += (int64_t)p->num_sinks + doc_raw_len[d] + doc_raw_len[d] / p->ratio;
  return tot;
}

size_t unigist_docs_workspace_bytes(const unigist_problem* p, int32_t op, int32_t num_docs, const int32_t* doc_raw_len) {
  if (check_docs(p, num_docs, doc_raw_len) != UNIGIST_OK) return 0;
  if (op != UNIGIST_OP_BWD) return 0;
  if (bwd_is_fused(p->head_dim, p->flags)) {  // one scratch layout over all packed tokens, then the runs' partial dK / dV
    size_t need = bwd_scratch_bytes(unigist_docs_total_len(p, num_docs, doc_raw_len), p->num_q_heads, p->head_dim,
                                    (p->flags & UNIGIST_FLAG_DOUT_FP32) != 0, true);
    for_each_doc_run(p, num_docs, doc_raw_len, [&](const unigist_problem& run, int64_t, int32_t) {
      Geom g;
      if (check_problem(&run, &g, nullptr) == UNIGIST_OK)
        need += bwd_partial_bytes(g, run.batch, run.num_q_heads, run.num_kv_heads, true);
      return (int32_t)UNIGIST_OK;
    });
    return need;
  }
  size_t need = 0;  // head_dim 64: one launch set per run, each with its own slice
  for_each_doc_run(p, num_docs, doc_raw_len, [&](const unigist_problem& run, int64_t, int32_t) {
    need += align_up(unigist_workspace_bytes(&run, op), 256);
    return (int32_t)UNIGIST_OK;
  });
  return need;
}

int32_t unigist_attn_fwd_docs(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len, const void* q,
                              const void* k, const void* v, void* o, float* lse, void* workspace, size_t ws_bytes,
                              void* stream) {
  (void)workspace;
  (void)ws_bytes;
  if (int32_t rc = check_docs(p, num_docs, doc_raw_len)) return rc;
  if (!q || !k || !v || !o || !lse) return fail(UNIGIST_ERR_INVALID_ARG, "a tensor is NULL");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || (reinterpret_cast<uintptr_t>(lse) & 3))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned (lse: 4-byte)");
  std::vector<SeqRun> runs;
  int64_t tokens = 0;
  if (int32_t rc = doc_runs(p, num_docs, doc_raw_len, &runs, &tokens)) return rc;
  if (int32_t rc = check_interleaved(p, runs[0].g)) return rc;
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  return launch_fwd_sm100_runs(runs.data(), (int)runs.size(), *p, scale, q, k, v, o, lse, (cudaStream_t)stream);
}

int32_t unigist_attn_bwd_docs(const unigist_problem* p, int32_t num_docs, const int32_t* doc_raw_len, const void* q,
                              const void* k, const void* v, const void* o, const float* lse, const void* d_o, void* dq,
                              void* dk, void* dv, void* workspace, size_t ws_bytes, void* stream) {
  if (int32_t rc = check_docs(p, num_docs, doc_raw_len)) return rc;
  if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv) return fail(UNIGIST_ERR_INVALID_ARG, "a tensor is NULL");
  const void* ptrs[] = {q, k, v, o, d_o, dq, dk, dv, workspace};
  for (const void* x : ptrs)
    if (!aligned16(x)) return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(lse) & 3) return fail(UNIGIST_ERR_ALIGNMENT, "lse must be 4-byte aligned");
  const size_t need = unigist_docs_workspace_bytes(p, UNIGIST_OP_BWD, num_docs, doc_raw_len);
  if (!workspace || ws_bytes < need)
    return fail(UNIGIST_ERR_WORKSPACE, "backward over documents needs %zu bytes of 16-byte aligned workspace, got %zu", need,
                ws_bytes);
  std::vector<SeqRun> runs;
  int64_t tokens = 0;
  if (int32_t rc = doc_runs(p, num_docs, doc_raw_len, &runs, &tokens)) return rc;
  if (int32_t rc = check_interleaved(p, runs[0].g)) return rc;
  const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
  if (bwd_is_fused(p->head_dim, p->flags))
    return launch_bwd_sm100_runs(runs.data(), (int)runs.size(), tokens, *p, scale, q, k, v, o, lse, d_o, dq, dk, dv,
                                 workspace, (cudaStream_t)stream);
  // the two-kernel backward (head_dim 64, or a fixed summation order asked for): the runs one after the other on the caller's stream
  const size_t rq = (size_t)p->num_q_heads * p->head_dim * 2, rk = (size_t)p->num_kv_heads * p->head_dim * 2;
  const size_t rdo = (p->flags & UNIGIST_FLAG_DOUT_FP32) ? 2 * rq : rq;
  size_t ws_off = 0;
  return for_each_doc_run(p, num_docs, doc_raw_len, [&](const unigist_problem& run, int64_t base, int32_t) {
    const size_t mine = align_up(unigist_workspace_bytes(&run, UNIGIST_OP_BWD), 256);
    char* ws = (char*)workspace + ws_off;
    ws_off += mine;
    return unigist_attn_bwd(&run, (const char*)q + base * rq, (const char*)k + base * rk, (const char*)v + base * rk,
                            (const char*)o + base * rq, lse + base * p->num_q_heads, (const char*)d_o + base * rdo,
                            (char*)dq + base * rq, (char*)dk + base * rk, (char*)dv + base * rk, ws, mine, stream);
  });
}

int32_t unigist_kv_compact(const unigist_problem* p, const void* k, const void* v, void* kc,
                           void* vc, int32_t num_blocks, int32_t* table, int32_t max_blocks,
                           int32_t* seq_lens, int32_t* kept_idx, void* workspace, size_t ws_bytes,
                           void* stream) {
  Geom g;
  if (int32_t rc = check_problem(p, &g, nullptr)) return rc;
  if (!kc || !vc || !table || !seq_lens) return fail(UNIGIST_ERR_INVALID_ARG, "a pointer is NULL");
  if ((k == nullptr) != (v == nullptr))
    return fail(UNIGIST_ERR_INVALID_ARG, "k and v must both be given or both be NULL");
  if (!aligned16(k) || !aligned16(v) || !aligned16(kc) || !aligned16(vc) || !aligned16(workspace))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  const int L = g.s + g.n + g.k * g.r;
  const int need_blocks = ((k ? L : g.N) + UNIGIST_PAGE_TOKENS - 1) / UNIGIST_PAGE_TOKENS;
  if (num_blocks < 1 || max_blocks < need_blocks)
    return fail(UNIGIST_ERR_SHAPE, "block table has %d entries per sequence, %d needed", max_blocks,
                need_blocks);
  if (k) {
    return launch_compact_gather(g, *p, k, v, kc, vc, num_blocks, table, max_blocks, seq_lens,
                                 kept_idx, (cudaStream_t)stream);
  }
  const bool edit_only = g.s % 64 == 0 && g.T % 64 == 0 && g.n % 64 == 0 && (g.k * g.r) % 64 == 0;
  if (!edit_only) {
    const size_t need = unigist_workspace_bytes(p, UNIGIST_OP_COMPACT);
    if (!workspace || ws_bytes < need)
      return fail(UNIGIST_ERR_WORKSPACE, "in-place compaction needs %zu bytes of workspace, got %zu",
                  need, ws_bytes);
  }
  return launch_compact_inplace(g, *p, kc, vc, num_blocks, table, max_blocks, seq_lens, kept_idx,
                                edit_only ? nullptr : workspace, (cudaStream_t)stream);
}

static int32_t check_chunk(const unigist_problem* p, const Geom& g, int32_t u0, int32_t c) {
  if (u0 < 0 || c < 1 || (int64_t)u0 + c > g.n)
    return fail(UNIGIST_ERR_INVALID_ARG, "chunk of %d units from unit %d does not fit the %d units of the prompt", c, u0,
                g.n);
  (void)p;
  return UNIGIST_OK;
}

size_t unigist_prefill_workspace_bytes(const unigist_problem* p, int32_t unit_begin, int32_t unit_count) {
  Geom g;
  if (check_problem(p, &g, nullptr) != UNIGIST_OK || check_chunk(p, g, unit_begin, unit_count) != UNIGIST_OK) return 0;
  const int64_t w_units = unit_begin < g.k ? unit_begin : g.k;
  const int64_t n_ctx = (int64_t)g.s + (w_units + unit_count) * g.r + unit_begin + unit_count;
  return align_up(2 * (size_t)p->batch * n_ctx * p->num_kv_heads * p->head_dim * 2, 256);
}

int32_t unigist_prefill_chunk(const unigist_problem* p, int32_t unit_begin, int32_t unit_count, const void* q,
                              const void* k, const void* v, void* kc, void* vc, int32_t num_blocks, int32_t* table,
                              int32_t max_blocks, int32_t* seq_lens, void* o, float* lse, void* workspace,
                              size_t ws_bytes, void* stream) {
  Geom g;
  float scale;
  if (int32_t rc = check_problem(p, &g, &scale)) return rc;
  if (int32_t rc = check_chunk(p, g, unit_begin, unit_count)) return rc;
  if (!q || !k || !v || !kc || !vc || !table || !seq_lens || !o || !lse)
    return fail(UNIGIST_ERR_INVALID_ARG, "a pointer is NULL");
  const void* ptrs[] = {q, k, v, kc, vc, o, lse, workspace};
  for (const void* x : ptrs)
    if (!aligned16(x)) return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  const size_t need = unigist_prefill_workspace_bytes(p, unit_begin, unit_count);
  if (!workspace || ws_bytes < need)
    return fail(UNIGIST_ERR_WORKSPACE, "this chunk needs %zu bytes of workspace, got %zu", need, ws_bytes);
  const int64_t kept = (int64_t)g.s + unit_begin + unit_count +
                       (int64_t)(g.k < unit_begin + unit_count ? g.k : unit_begin + unit_count) * g.r;
  if (num_blocks < 1 || (int64_t)max_blocks * UNIGIST_PAGE_TOKENS < kept)
    return fail(UNIGIST_ERR_SHAPE, "block table has %d entries per sequence, the cache after this chunk needs %lld tokens",
                max_blocks, (long long)kept);
  return launch_prefill_chunk(*p, g, scale, unit_begin, unit_count, q, k, v, kc, vc, num_blocks, table, max_blocks,
                              seq_lens, o, lse, workspace, (cudaStream_t)stream);
}

size_t unigist_cache_state_bytes(const unigist_problem* p) {
  Geom g;
  if (check_problem(p, &g, nullptr) != UNIGIST_OK) return 0;
  return align_up(cache_state_bytes(p->batch, g.r, unigist_window_units(p)), 256);
}

// The window of a growing sequence is k = ceil(W / r) units, not clamped by the prompt's length.
static Geom decode_geom(const unigist_problem* p, const Geom& g) {
  Geom d = g;
  d.k = (int)(((int64_t)p->window + p->ratio - 1) / p->ratio);
  return d;
}

int32_t unigist_cache_state_init(const unigist_problem* p, int32_t units_done, int32_t* state, void* stream) {
  Geom g;
  if (int32_t rc = check_problem(p, &g, nullptr)) return rc;
  if (!state || units_done < 0) return fail(UNIGIST_ERR_INVALID_ARG, "state is NULL or units_done < 0");
  return launch_cache_state_init(decode_geom(p, g), p->batch, units_done, state, (cudaStream_t)stream);
}

int32_t unigist_cache_append(const unigist_problem* p, const void* k_new, const void* v_new, int32_t is_gist, void* kc,
                             void* vc, int32_t num_blocks, const int32_t* table, int32_t max_blocks, int32_t* seq_lens,
                             int32_t* state, void* stream) {
  Geom g;
  if (int32_t rc = check_problem(p, &g, nullptr)) return rc;
  if (!k_new || !v_new || !kc || !vc || !table || !seq_lens || !state)
    return fail(UNIGIST_ERR_INVALID_ARG, "a pointer is NULL");
  if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(kc) || !aligned16(vc))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (num_blocks < 1 || max_blocks < 1) return fail(UNIGIST_ERR_INVALID_ARG, "the cache has no blocks");
  return launch_cache_append(decode_geom(p, g), *p, is_gist != 0, k_new, v_new, kc, vc, num_blocks, table, max_blocks,
                             seq_lens, state, (cudaStream_t)stream);
}

size_t unigist_decode_workspace_bytes(int32_t S, int32_t Hq, int32_t Hkv, int32_t D,
                                      int32_t max_blocks) {
  if (S < 1 || Hq < 1 || Hkv < 1 || D < 1 || max_blocks < 1) return 0;
  const int splits = decode_num_splits(S, Hkv, max_blocks);
  // per (seq, q head, split): D fp32 partial outputs + running max + running sum
  return align_up((size_t)S * Hq * splits * (D + 2) * sizeof(float), 256);
}

int32_t unigist_decode(int32_t S, int32_t Hq, int32_t Hkv, int32_t D, float softmax_scale,
                       const void* q, const void* kc, const void* vc, int32_t num_blocks,
                       const int32_t* table, int32_t max_blocks, const int32_t* seq_lens, void* o,
                       float* lse, void* workspace, size_t ws_bytes, void* stream) {
  if (S < 1 || Hq < 1 || Hkv < 1 || max_blocks < 1 || num_blocks < 1)
    return fail(UNIGIST_ERR_INVALID_ARG, "decode has a non-positive size");
  if (S > kMaxGridYZ || Hkv > kMaxGridYZ)
    return fail(UNIGIST_ERR_SHAPE, "num_seqs %d or num_kv_heads %d exceeds %d", S, Hkv, kMaxGridYZ);
  if (Hq % Hkv) return fail(UNIGIST_ERR_SHAPE, "num_q_heads %d is not a multiple of num_kv_heads %d", Hq, Hkv);
  if (D != 128) return fail(UNIGIST_ERR_SHAPE, "decode supports head_dim 128, got %d", D);
  if (Hq / Hkv > 8) return fail(UNIGIST_ERR_UNSUPPORTED, "decode supports at most 8 query heads per KV head");
  if (!q || !kc || !vc || !table || !seq_lens || !o) return fail(UNIGIST_ERR_INVALID_ARG, "a pointer is NULL");
  if (!aligned16(q) || !aligned16(kc) || !aligned16(vc) || !aligned16(o) || !aligned16(workspace))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (!(softmax_scale >= 0.f) || std::isinf(softmax_scale))
    return fail(UNIGIST_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0");
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
  const size_t need = unigist_decode_workspace_bytes(S, Hq, Hkv, D, max_blocks);
  if (!workspace || ws_bytes < need)
    return fail(UNIGIST_ERR_WORKSPACE, "decode needs %zu bytes of workspace, got %zu", need, ws_bytes);
  return launch_decode(S, Hq, Hkv, D, scale, q, kc, vc, num_blocks, table, max_blocks, seq_lens, o,
                       lse, workspace, (cudaStream_t)stream);
}

int32_t unigist_decode_step(const unigist_problem* p, const void* q, const void* kc, const void* vc, int32_t num_blocks,
                            const int32_t* table, int32_t max_blocks, const int32_t* seq_lens, const int32_t* state,
                            void* o, float* lse, void* workspace, size_t ws_bytes, void* stream) {
  Geom g;
  float scale;
  if (int32_t rc = check_problem(p, &g, &scale)) return rc;
  const int S = p->batch, Hq = p->num_q_heads, Hkv = p->num_kv_heads, D = p->head_dim;
  if (max_blocks < 1 || num_blocks < 1) return fail(UNIGIST_ERR_INVALID_ARG, "the cache has no blocks");
  if (D != 128) return fail(UNIGIST_ERR_SHAPE, "decode supports head_dim 128, got %d", D);
  if (Hq / Hkv > 8) return fail(UNIGIST_ERR_UNSUPPORTED, "decode supports at most 8 query heads per KV head");
  if (!q || !kc || !vc || !table || !seq_lens || !state || !o) return fail(UNIGIST_ERR_INVALID_ARG, "a pointer is NULL");
  if (!aligned16(q) || !aligned16(kc) || !aligned16(vc) || !aligned16(o) || !aligned16(workspace))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  const size_t need = unigist_decode_workspace_bytes(S, Hq, Hkv, D, max_blocks);
  if (!workspace || ws_bytes < need)
    return fail(UNIGIST_ERR_WORKSPACE, "decode needs %zu bytes of workspace, got %zu", need, ws_bytes);
  int stride = 0, free_off = 0;
  cache_state_layout(g.r, decode_geom(p, g).k, &stride, &free_off);
  return launch_decode(S, Hq, Hkv, D, scale, q, kc, vc, num_blocks, table, max_blocks, seq_lens, o, lse, workspace,
                       (cudaStream_t)stream, state, stride, free_off);
}

int32_t unigist_selftest_wait_timeout(void* stream) { return launch_selftest_wait((cudaStream_t)stream); }

int32_t unigist_kernel_timing(int32_t enable) {
  for (int i = 0; i < g_num_records; ++i) {
    cudaEventDestroy(g_records[i].e0);
    cudaEventDestroy(g_records[i].e1);
  }
  g_num_records = 0;
  g_timing = enable != 0;
  return UNIGIST_OK;
}

int32_t unigist_kernel_timing_count(void) { return g_num_records; }

int32_t unigist_kernel_timing_get(int32_t index, char* name, int32_t cap, float* ms) {
  if (index < 0 || index >= g_num_records || !ms) return fail(UNIGIST_ERR_INVALID_ARG, "no such timing record");
  TimingRecord& r = g_records[index];
  cudaError_t e = cudaEventSynchronize(r.e1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(ms, r.e0, r.e1);
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "kernel timing: %s", cudaGetErrorString(e));
  if (name && cap > 0) {
    strncpy(name, r.name, (size_t)cap - 1);
    name[cap - 1] = 0;
  }
  return UNIGIST_OK;
}

int64_t unigist_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* unigist_last_error_string(void) { return g_err; }

}  // extern "C"
