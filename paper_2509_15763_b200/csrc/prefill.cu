// Chunk-wise prefill over the compressed cache (Section 4.3): a chunk of gist units is encoded against
// what the cache still holds -- the sinks, every earlier gist and the raw tokens of the last k units --
// and the cache is then advanced to the state after the chunk.  The chunk's outputs are, by
// construction of the mask, the rows of the one-pass forward over the whole prompt.
//
// Three launches: (1) gather the cache and the chunk's K / V into a dense context
// [sinks | window raw + chunk raw | all gists] (HBM-bound, small next to the attention), (2) the
// forward kernel with queries for the chunk rows only, (3) the compaction gather from the context back
// into the pages.
#include "ug_common.cuh"

namespace ug {
namespace {

constexpr int PG = UNIGIST_PAGE_TOKENS;

// ctx[b, sigma, hk, :] for sigma in the context's shifted order; vecs = D / 8 16-byte vectors per head row.
// Cache order is [sinks | gists | window raw]; chunk order is [sinks (first chunk only) | raw | gists].
__global__ void __launch_bounds__(256)
prefill_gather_kernel(int B, int Hkv, int vecs, int s, int u0, int w0, int c_raw, int c_gists,
                      const uint4* __restrict__ kc, const uint4* __restrict__ vc, int num_blocks,
                      const int32_t* __restrict__ table, int max_blocks, const uint4* __restrict__ k_chunk,
                      const uint4* __restrict__ v_chunk, uint4* __restrict__ k_ctx, uint4* __restrict__ v_ctx) {
  const int Tc = w0 + c_raw, n_ctx = s + Tc + u0 + c_gists;
  const int sq = u0 == 0 ? s : 0, n_chunk = sq + c_raw + c_gists;
  const long long per_tok = (long long)Hkv * vecs;
  const long long total = (long long)B * n_ctx * per_tok;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long tok = e / per_tok;
    const int rem = (int)(e - tok * per_tok);
    const int hk = rem / vecs, vec = rem - hk * vecs;
    const int b = (int)(tok / n_ctx), sigma = (int)(tok - (long long)b * n_ctx);
    int cache_pos = -1, chunk_row = -1;
    if (sigma < s) {
      if (u0 == 0) chunk_row = sigma; else cache_pos = sigma;
    } else if (sigma < s + Tc) {
      const int i = sigma - s;
      if (i < w0) cache_pos = s + u0 + i; else chunk_row = sq + (i - w0);
    } else {
      const int ug = sigma - s - Tc;
      if (ug < u0) cache_pos = s + ug; else chunk_row = sq + c_raw + (ug - u0);
    }
    uint4 kk, vv;
    if (chunk_row >= 0) {
      const long long so = (((long long)b * n_chunk + chunk_row) * Hkv + hk) * vecs + vec;
      kk = __ldg(k_chunk + so);
      vv = __ldg(v_chunk + so);
    } else {
      int blk = table[(long long)b * max_blocks + cache_pos / PG];
      blk = min(max(blk, 0), num_blocks - 1);  // never read outside the cache
      const long long so = (((long long)blk * Hkv + hk) * PG + cache_pos % PG) * vecs + vec;
      kk = __ldg(kc + so);
      vv = __ldg(vc + so);
    }
    k_ctx[e] = kk;
    v_ctx[e] = vv;
  }
}

}  // namespace

int32_t launch_prefill_chunk(const unigist_problem& p, const Geom& g_full, float scale, int u0, int c, const void* q,
                             const void* k, const void* v, void* kc, void* vc, int num_blocks, int32_t* table,
                             int max_blocks, int32_t* seq_lens, void* o, float* lse, void* workspace, cudaStream_t st) {
  const int r = g_full.r, s = g_full.s, kw = g_full.k;  // kw: window units, clamped to the whole prompt's units
  const int w_units = u0 < kw ? u0 : kw;                 // raw units still in the cache
  const int w0 = w_units * r, c_raw = c * r;
  // geometry of the dense context [sinks | window raw + chunk raw | every gist so far]
  Geom gc;
  gc.s = s;
  gc.T = w0 + c_raw;
  gc.r = r;
  gc.n = u0 + c;
  gc.N = gc.s + gc.T + gc.n;
  gc.uoff = u0 - w_units;
  gc.k = kw < gc.T / r ? kw : gc.T / r;
  const int B = p.batch, Hkv = p.num_kv_heads, vecs = p.head_dim / 8;
  uint4* k_ctx = static_cast<uint4*>(workspace);
  uint4* v_ctx = k_ctx + (size_t)B * gc.N * Hkv * vecs;
  {
    const long long total = (long long)B * gc.N * Hkv * vecs;
    const long long want = (total + 255) / 256;
    const long long cap = (long long)sm_count() * 16;
    const int blocks = (int)(want < cap ? want : cap);
    KernelScope ks("prefill_gather_kernel", st);
    prefill_gather_kernel<<<blocks, 256, 0, st>>>(B, Hkv, vecs, s, u0, w0, c_raw, c, (const uint4*)kc, (const uint4*)vc,
                                                  num_blocks, table, max_blocks, (const uint4*)k, (const uint4*)v, k_ctx,
                                                  v_ctx);
  }
  if (int32_t rc = check_launch("prefill gather kernel")) return rc;
  // queries: the chunk's rows only, i.e. the tail of each segment of the context
  QueryRows qr;
  const int sq = u0 == 0 ? s : 0;
  qr.off[kSegSink] = s - sq;
  qr.off[kSegRaw] = w0;
  qr.off[kSegGist] = u0;
  qr.out_base[kSegSink] = 0;
  qr.out_base[kSegRaw] = sq;
  qr.out_base[kSegGist] = sq + c_raw;
  qr.n_out = sq + c_raw + c;
  unigist_problem pc = p;
  pc.flags = 0;
  if (int32_t rc = launch_fwd_sm100(gc, pc, scale, q, k_ctx, v_ctx, o, lse, st, &qr)) return rc;
  // the cache after the chunk: sinks, every gist, the raw tokens of the last min(k, u0 + c) units
  Geom gk = gc;
  gk.k = kw < u0 + c ? kw : u0 + c;
  return launch_compact_gather(gk, pc, k_ctx, v_ctx, kc, vc, num_blocks, table, max_blocks, seq_lens, nullptr, st);
}

}  // namespace ug
