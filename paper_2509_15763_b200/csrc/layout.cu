// Gist shift index arrays and the shift / unshift row permutations (Section 4.2).
// Both are closed forms of (s, T, r); no index table is read by the copy kernels.
#include "ug_common.cuh"

namespace ug {

__global__ void layout_kernel(Geom g, int32_t* __restrict__ sp, int32_t* __restrict__ up,
                              int32_t* __restrict__ pos) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < g.N; i += gridDim.x * blockDim.x) {
    if (sp) sp[i] = shift_perm(g, i);
    const int sig = unshift_perm(g, i);
    if (up) up[i] = sig;
    if (pos) pos[i] = sig < g.s + g.T ? sig : g.s + (sig - g.s - g.T + 1) * g.r;
  }
}

int32_t launch_layout(const Geom& g, int32_t* sp, int32_t* up, int32_t* pos, cudaStream_t st) {
  const int threads = 256;
  int blocks = (g.N + threads - 1) / threads;
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  {
    KernelScope ks("layout_kernel", st);
    layout_kernel<<<blocks, threads, 0, st>>>(g, sp, up, pos);
  }
  return check_launch("layout kernel");
}

// dst[b, i, :] = src[b, perm(i), :] with rows of `vecs` 16-byte vectors.  HBM-bound: every
// vector is read once and written once, coalesced along the row.  One warp per destination row
// (the permutation is evaluated once per row), kRows rows in flight per warp.
template <bool kInverse>
__global__ void __launch_bounds__(256)
shift_rows_kernel(Geom g, const uint4* __restrict__ src, uint4* __restrict__ dst, int vecs,
                  long long rows) {
  constexpr int kRows = 4, kVec = 4;  // up to kRows * kVec loads in flight per lane
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r0 = warp * kRows; r0 < rows; r0 += nwarps * kRows) {
    const uint4* sp[kRows];
    uint4* dp[kRows];
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      const long long row = r0 + u < rows ? r0 + u : rows - 1;  // the tail repeats the last row (same bytes)
      const int b = (int)(row / g.N);
      const int i = (int)(row - (long long)b * g.N);
      const int j = kInverse ? unshift_perm(g, i) : shift_perm(g, i);
      sp[u] = src + ((long long)b * g.N + j) * vecs;
      dp[u] = dst + row * vecs;
    }
    for (int v0 = lane; v0 < vecs; v0 += 32 * kVec) {
      uint4 val[kRows][kVec];
#pragma unroll
      for (int u = 0; u < kRows; ++u)
#pragma unroll
        for (int w = 0; w < kVec; ++w)
          if (v0 + 32 * w < vecs) val[u][w] = __ldcs(sp[u] + v0 + 32 * w);
#pragma unroll
      for (int u = 0; u < kRows; ++u)
#pragma unroll
        for (int w = 0; w < kVec; ++w)
          if (v0 + 32 * w < vecs) __stcs(dp[u] + v0 + 32 * w, val[u][w]);
    }
  }
}

int32_t launch_shift(const Geom& g, int B, const void* src, void* dst, size_t row_bytes,
                     bool inverse, cudaStream_t st) {
  const int vecs = (int)(row_bytes / 16);
  const long long rows = (long long)B * g.N;
  const long long want = (rows + 31) / 32;  // 8 warps x 4 rows per block and pass
  const long long cap = (long long)sm_count() * 8;
  const int blocks = (int)(want < cap ? (want > 0 ? want : 1) : cap);
  {
    KernelScope ks(inverse ? "unshift_rows_kernel" : "shift_rows_kernel", st);
    if (inverse)
      shift_rows_kernel<true><<<blocks, 256, 0, st>>>(g, (const uint4*)src, (uint4*)dst, vecs, rows);
    else
      shift_rows_kernel<false><<<blocks, 256, 0, st>>>(g, (const uint4*)src, (uint4*)dst, vecs, rows);
  }
  return check_launch("gist shift kernel");
}

}  // namespace ug
