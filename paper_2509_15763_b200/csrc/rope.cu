// Rotary position embedding with the aligned position ids of Section 4.1 (step 3: a gist token takes
// the position id of the raw token right after it), optionally fused with the gist shift of Section 4.2.
// HBM-bound: every element is read once and written once.  The position id and the destination row are
// closed forms of the interleaved token index; no index table is read.
#include "ug_common.cuh"

namespace ug {

namespace {

// Position id of interleaved token t: sinks and raw tokens count up, gist u gets s + (u + 1) r.
__device__ __forceinline__ int aligned_pos(const Geom& g, int t) {
  if (t < g.s) return t;
  const int u = (t - g.s) / (g.r + 1), p = (t - g.s) - u * (g.r + 1);
  return g.s + u * g.r + p;  // p = r for the gist of unit u
}

// One warp per token.  A lane owns 4 consecutive rotary frequencies j .. j + 3 of one head row (features
// j and j + D / 2 pair up), D / 8 lanes cover a row and the warp takes 256 / D rows per pass; the
// angles are computed once per token in fp64 (a position times a frequency reaches 1e5 rad) and reused
// for every head.
template <int D>
__global__ void __launch_bounds__(256)
rope_kernel(Geom g, long long tokens, int heads, double log2_theta, int to_shifted, int from_shifted, int inverse,
            const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst) {
  constexpr int kLanesPerRow = D / 8, kRowsPerPass = 32 / kLanesPerRow;
  const int lane = threadIdx.x & 31;
  const int j0 = (lane % kLanesPerRow) * 4, sub = lane / kLanesPerRow;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  double inv_freq[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) inv_freq[e] = exp2(-2.0 * (j0 + e) / D * log2_theta);
  for (long long tk = warp; tk < tokens; tk += nwarps) {  // tk = b * N + t, t interleaved
    const long long b = tk / g.N;
    const int t = (int)(tk - b * g.N);
    const double pos = (double)aligned_pos(g, t);
    float cs[4], sn[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      double a = pos * inv_freq[e];
      a -= 6.283185307179586476925 * rint(a * 0.15915494309189533577);  // into [-pi, pi]
      sincosf((float)a, &sn[e], &cs[e]);
      if (inverse) sn[e] = -sn[e];  // the transpose of the rotation: what the backward pass applies to a gradient
    }
    const int sigma = (to_shifted | from_shifted) ? unshift_perm(g, t) : t;  // the token's shifted position
    const long long out_tk = b * g.N + (to_shifted ? sigma : t);
    const __nv_bfloat16* s_tok = src + (b * g.N + (from_shifted ? sigma : t)) * heads * D;
    __nv_bfloat16* d_tok = dst + out_tk * heads * D;
    for (int h0 = 0; h0 < heads; h0 += 2 * kRowsPerPass) {  // two passes in flight
      uint2 lo[2], hi[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int h = h0 + u * kRowsPerPass + sub;
        if (h < heads) {
          lo[u] = *reinterpret_cast<const uint2*>(s_tok + h * D + j0);
          hi[u] = *reinterpret_cast<const uint2*>(s_tok + h * D + D / 2 + j0);
        }
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int h = h0 + u * kRowsPerPass + sub;
        if (h < heads) {
          // a bf16 is the high half of an fp32
          const float x[4] = {__uint_as_float(lo[u].x << 16), __uint_as_float(lo[u].x & 0xffff0000u),
                              __uint_as_float(lo[u].y << 16), __uint_as_float(lo[u].y & 0xffff0000u)};
          const float y[4] = {__uint_as_float(hi[u].x << 16), __uint_as_float(hi[u].x & 0xffff0000u),
                              __uint_as_float(hi[u].y << 16), __uint_as_float(hi[u].y & 0xffff0000u)};
          float a[4], c[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            a[e] = x[e] * cs[e] - y[e] * sn[e];
            c[e] = y[e] * cs[e] + x[e] * sn[e];
          }
          const __nv_bfloat162 a01 = __floats2bfloat162_rn(a[0], a[1]), a23 = __floats2bfloat162_rn(a[2], a[3]);
          const __nv_bfloat162 c01 = __floats2bfloat162_rn(c[0], c[1]), c23 = __floats2bfloat162_rn(c[2], c[3]);
          uint2 wl, wh;
          wl.x = *reinterpret_cast<const uint32_t*>(&a01);
          wl.y = *reinterpret_cast<const uint32_t*>(&a23);
          wh.x = *reinterpret_cast<const uint32_t*>(&c01);
          wh.y = *reinterpret_cast<const uint32_t*>(&c23);
          *reinterpret_cast<uint2*>(d_tok + h * D + j0) = wl;
          *reinterpret_cast<uint2*>(d_tok + h * D + D / 2 + j0) = wh;
        }
      }
    }
  }
}

}  // namespace

int32_t launch_rope(const Geom& g, int B, int heads, int D, float theta_base, bool to_shifted, bool from_shifted,
                    bool inverse, const void* src, void* dst, cudaStream_t st) {
  const long long tokens = (long long)B * g.N;
  const long long want = (tokens + 7) / 8;  // 8 warps per block
  const long long cap = (long long)sm_count() * 8;
  const int blocks = (int)(want < cap ? (want > 0 ? want : 1) : cap);
  const double log2_theta = log2((double)theta_base);
  {
    KernelScope ks("rope_kernel", st);
    if (D == 128)
      rope_kernel<128><<<blocks, 256, 0, st>>>(g, tokens, heads, log2_theta, to_shifted ? 1 : 0, from_shifted ? 1 : 0, inverse ? 1 : 0,
                                                 (const __nv_bfloat16*)src, (__nv_bfloat16*)dst);
    else
      rope_kernel<64><<<blocks, 256, 0, st>>>(g, tokens, heads, log2_theta, to_shifted ? 1 : 0, from_shifted ? 1 : 0, inverse ? 1 : 0,
                                                (const __nv_bfloat16*)src, (__nv_bfloat16*)dst);
  }
  return check_launch("rope kernel");
}

}  // namespace ug
