// KV compaction (Section 4.3): keep sinks, all gists and the raw tokens of the last k gist
// units; cache order [sinks | gists | window raw] in 64-token pages.
#include "ug_common.cuh"

namespace ug {
namespace {

constexpr int PG = UNIGIST_PAGE_TOKENS;

// Shifted position of the token that lands at cache position c.
__host__ __device__ inline int kept_source(const Geom& g, int c) {
  if (c < g.s) return c;
  if (c < g.s + g.n) return g.s + g.T + (c - g.s);
  return g.s + (g.T - g.k * g.r) + (c - g.s - g.n);
}

// src: shifted (or interleaved) [B,N,Hkv,D] (vecs = D/8 16-byte vectors per head row) -> pages.
__global__ void __launch_bounds__(256)
compact_gather_kernel(Geom g, int B, int Hkv, int vecs, int L, const uint4* __restrict__ k,
                      const uint4* __restrict__ v, uint4* __restrict__ kc, uint4* __restrict__ vc,
                      int num_blocks, const int32_t* __restrict__ table, int max_blocks,
                      int32_t* __restrict__ seq_lens, int32_t* __restrict__ kept_idx, int interleaved) {
  const long long per_tok = (long long)Hkv * vecs;
  const long long total = (long long)B * L * per_tok;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long tok = e / per_tok;
    const int rem = (int)(e - tok * per_tok);
    const int hk = rem / vecs, vec = rem - hk * vecs;
    const int b = (int)(tok / L), c = (int)(tok - (long long)b * L);
    const int src = kept_source(g, c);
    if (rem == 0) {
      if (kept_idx) kept_idx[(long long)b * L + c] = src;
      if (c == 0) seq_lens[b] = L;
    }
    const int blk = table[(long long)b * max_blocks + c / PG];
    if (blk < 0 || blk >= num_blocks) continue;  // never write outside the cache
    const int src_row = interleaved ? shift_perm(g, src) : src;  // k, v given in interleaved order
    const long long so = (((long long)b * g.N + src_row) * Hkv + hk) * vecs + vec;
    const long long d = (((long long)blk * Hkv + hk) * PG + c % PG) * vecs + vec;
    kc[d] = __ldg(k + so);
    vc[d] = __ldg(v + so);
  }
}

// In place, aligned segments: only the block table changes.
__global__ void compact_edit_table_kernel(Geom g, int L, int32_t* __restrict__ table, int max_blocks,
                                          int32_t* __restrict__ seq_lens, int32_t* __restrict__ kept_idx) {
  extern __shared__ int32_t old_row[];
  const int b = blockIdx.x;
  const int nbN = g.N / PG, nbL = L / PG;
  int32_t* row = table + (long long)b * max_blocks;
  for (int i = threadIdx.x; i < nbN; i += blockDim.x) old_row[i] = row[i];
  __syncthreads();
  const int sb = g.s / PG, gb = g.n / PG, wb = (g.k * g.r) / PG, tb = g.T / PG;
  for (int i = threadIdx.x; i < nbN; i += blockDim.x) {
    int src;
    if (i < sb) src = i;                               // sinks stay
    else if (i < sb + gb) src = sb + tb + (i - sb);    // gist pages
    else if (i < nbL) src = sb + (tb - wb) + (i - sb - gb);  // window pages
    else src = sb + (i - nbL);                         // freed raw pages
    row[i] = old_row[src];
  }
  if (threadIdx.x == 0) seq_lens[b] = L;
  if (kept_idx)
    for (int c = threadIdx.x; c < L; c += blockDim.x) kept_idx[(long long)b * L + c] = kept_source(g, c);
}

// In place, ragged segments, step 1: kept tokens -> staging [2][B][L][Hkv][D].
// step 2 (kToCache): staging -> logical positions [0, L) through the same table.
template <bool kToCache>
__global__ void __launch_bounds__(256)
compact_stage_kernel(Geom g, int B, int Hkv, int vecs, int L, uint4* __restrict__ kc,
                     uint4* __restrict__ vc, int num_blocks, const int32_t* __restrict__ table,
                     int max_blocks, uint4* __restrict__ stage, int32_t* __restrict__ seq_lens,
                     int32_t* __restrict__ kept_idx) {
  const long long per_tok = (long long)Hkv * vecs;
  const long long total = (long long)B * L * per_tok;
  uint4* stage_v = stage + total;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long tok = e / per_tok;
    const int rem = (int)(e - tok * per_tok);
    const int hk = rem / vecs, vec = rem - hk * vecs;
    const int b = (int)(tok / L), c = (int)(tok - (long long)b * L);
    const int pos = kToCache ? c : kept_source(g, c);  // logical cache position
    if (kToCache && rem == 0) {
      if (kept_idx) kept_idx[(long long)b * L + c] = kept_source(g, c);
      if (c == 0) seq_lens[b] = L;
    }
    const int blk = table[(long long)b * max_blocks + pos / PG];
    if (blk < 0 || blk >= num_blocks) continue;
    const long long d = (((long long)blk * Hkv + hk) * PG + pos % PG) * vecs + vec;
    if (kToCache) {
      kc[d] = stage[e];
      vc[d] = stage_v[e];
    } else {
      stage[e] = kc[d];
      stage_v[e] = vc[d];
    }
  }
}

int grid_for(long long total) {
  long long want = (total + 255) / 256;
  const long long cap = (long long)sm_count() * 16;
  return (int)(want < cap ? (want < 1 ? 1 : want) : cap);
}

}  // namespace

int32_t launch_compact_gather(const Geom& g, const unigist_problem& p, const void* k, const void* v,
                              void* kc, void* vc, int num_blocks, const int32_t* table,
                              int max_blocks, int32_t* seq_lens, int32_t* kept_idx,
                              cudaStream_t st) {
  const int L = g.s + g.n + g.k * g.r, vecs = p.head_dim / 8;
  const long long total = (long long)p.batch * L * p.num_kv_heads * vecs;
  {
    KernelScope ks("compact_gather_kernel", st);
    compact_gather_kernel<<<grid_for(total), 256, 0, st>>>(
        g, p.batch, p.num_kv_heads, vecs, L, (const uint4*)k, (const uint4*)v, (uint4*)kc, (uint4*)vc,
        num_blocks, table, max_blocks, seq_lens, kept_idx, (p.flags & UNIGIST_FLAG_INTERLEAVED) ? 1 : 0);
  }
  return check_launch("compaction gather kernel");
}

int32_t launch_compact_inplace(const Geom& g, const unigist_problem& p, void* kc, void* vc,
                               int num_blocks, int32_t* table, int max_blocks, int32_t* seq_lens,
                               int32_t* kept_idx, void* ws, cudaStream_t st) {
  const int L = g.s + g.n + g.k * g.r, vecs = p.head_dim / 8;
  if (!ws) {  // segments are page aligned: edit the table
    const size_t smem = (size_t)(g.N / PG) * sizeof(int32_t);
    if (smem > 200 * 1024) return fail(UNIGIST_ERR_UNSUPPORTED, "sequence too long for the table edit");
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(compact_edit_table_kernel,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    }
    {
      KernelScope ks("compact_edit_table_kernel", st);
      compact_edit_table_kernel<<<p.batch, 256, smem, st>>>(g, L, table, max_blocks, seq_lens, kept_idx);
    }
    return check_launch("compaction table edit kernel");
  }
  const long long total = (long long)p.batch * L * p.num_kv_heads * vecs;
  {
    KernelScope ks("compact_stage_kernel", st);
    compact_stage_kernel<false><<<grid_for(total), 256, 0, st>>>(
        g, p.batch, p.num_kv_heads, vecs, L, (uint4*)kc, (uint4*)vc, num_blocks, table, max_blocks,
        (uint4*)ws, seq_lens, kept_idx);
  }
  if (int32_t rc = check_launch("compaction staging kernel")) return rc;
  {
    KernelScope ks("compact_writeback_kernel", st);
    compact_stage_kernel<true><<<grid_for(total), 256, 0, st>>>(
        g, p.batch, p.num_kv_heads, vecs, L, (uint4*)kc, (uint4*)vc, num_blocks, table, max_blocks,
        (uint4*)ws, seq_lens, kept_idx);
  }
  return check_launch("compaction write-back kernel");
}

}  // namespace ug
