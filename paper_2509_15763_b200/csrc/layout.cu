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
  if (blocks > 148 * 8) blocks = 148 * 8;
  {
    KernelScope ks("layout_kernel", st);
    layout_kernel<<<blocks, threads, 0, st>>>(g, sp, up, pos);
  }
  return check_launch("layout kernel");
}

// dst[b, i, :] = src[b, perm(i), :] with rows of `vecs` 16-byte vectors.  HBM-bound: every
// vector is read once and written once, coalesced along the row.
template <bool kInverse>
__global__ void __launch_bounds__(256)
shift_rows_kernel(Geom g, const uint4* __restrict__ src, uint4* __restrict__ dst, int vecs,
                  long long total) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  constexpr int kUnroll = 4;
  for (; idx + (kUnroll - 1) * stride < total; idx += kUnroll * stride) {
    uint4 val[kUnroll];
    long long out[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const long long e = idx + u * stride;
      const long long row = e / vecs;
      const int vec = (int)(e - row * vecs);
      const int b = (int)(row / g.N);
      const int i = (int)(row - (long long)b * g.N);
      const int j = kInverse ? unshift_perm(g, i) : shift_perm(g, i);
      out[u] = e;
      val[u] = __ldg(src + ((long long)b * g.N + j) * vecs + vec);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) dst[out[u]] = val[u];
  }
  for (; idx < total; idx += stride) {
    const long long row = idx / vecs;
    const int vec = (int)(idx - row * vecs);
    const int b = (int)(row / g.N);
    const int i = (int)(row - (long long)b * g.N);
    const int j = kInverse ? unshift_perm(g, i) : shift_perm(g, i);
    dst[idx] = __ldg(src + ((long long)b * g.N + j) * vecs + vec);
  }
}

int32_t launch_shift(const Geom& g, int B, const void* src, void* dst, size_t row_bytes,
                     bool inverse, cudaStream_t st) {
  const int vecs = (int)(row_bytes / 16);
  const long long total = (long long)B * g.N * vecs;
  long long want = (total + 255) / 256;
  const int blocks = (int)(want < 148 * 16 ? want : 148 * 16);
  {
    KernelScope ks(inverse ? "unshift_rows_kernel" : "shift_rows_kernel", st);
    if (inverse)
      shift_rows_kernel<true><<<blocks, 256, 0, st>>>(g, (const uint4*)src, (uint4*)dst, vecs, total);
    else
      shift_rows_kernel<false><<<blocks, 256, 0, st>>>(g, (const uint4*)src, (uint4*)dst, vecs, total);
  }
  return check_launch("gist shift kernel");
}

}  // namespace ug
