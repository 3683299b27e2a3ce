// CUDA-core (no tensor core) backward of the gist-masked attention: dQ and dK/dV kernels on 64x64
// tiles of the SHIFTED sequence.  The general path (any s, T, r, W, head_dim 64 or 128; tiles may
// straddle the sink / raw / gist segments because the mask is evaluated per element from the
// closed-form row intervals; tiles with no visible pair are skipped without being read), used for the
// one case the tensor-core backward does not cover: head_dim 64 with a sink prefix.
#include "ug_common.cuh"

namespace ug {
namespace {

constexpr int TS = 64;        // tile side
constexpr int LDS_ = TS + 4;  // leading dimension of the score tile in shared memory

// Does any row of [a, b] see any column of [c0, c1] (shifted coordinates, inclusive)?
// Inside one segment the per-row intervals are monotone and overlapping, so the union over the
// rows is the interval [lo(first row), hi(last row)].
__device__ bool tile_any_visible(const Geom& g, int a, int b, int c0, int c1) {
  const int seg_lo[3] = {0, g.s, g.s + g.T};
  const int seg_hi[3] = {g.s - 1, g.s + g.T - 1, g.N - 1};
  for (int sr = 0; sr < 3; ++sr) {
    const int ra = max(a, seg_lo[sr]), rb = min(b, seg_hi[sr]);
    if (ra > rb) continue;
    const RowIv va = row_intervals(g, ra), vb = row_intervals(g, rb);
    // sink columns [0, vb.hi_sink]
    if (c0 <= vb.hi_sink && c0 < g.s) return true;
    // raw columns [va.lo_raw, vb.hi_raw]
    {
      const int x0 = max(c0, g.s + va.lo_raw), x1 = min(c1, g.s + vb.hi_raw);
      if (x0 <= x1) return true;
    }
    // gist columns [0, vb.hi_gist]
    {
      const int x0 = max(c0, g.s + g.T), x1 = min(c1, g.s + g.T + vb.hi_gist);
      if (x0 <= x1) return true;
    }
  }
  return false;
}

template <int D>
__device__ void load_tile_bf16(float* dst, const __nv_bfloat16* base, long long row_stride,
                               int row0, int nrows_valid) {
  constexpr int LD = D + 4;
  constexpr int VPR = D / 8;  // 16-byte vectors per row
  for (int e = threadIdx.x; e < TS * VPR; e += blockDim.x) {
    const int rr = e / VPR, vv = e % VPR;
    float f[8];
    if (rr < nrows_valid) {
      const uint4 raw = *reinterpret_cast<const uint4*>(base + (long long)(row0 + rr) * row_stride + vv * 8);
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const float2 t = __bfloat1622float2(h[x]);
        f[2 * x] = t.x;
        f[2 * x + 1] = t.y;
      }
    } else {
#pragma unroll
      for (int x = 0; x < 8; ++x) f[x] = 0.f;
    }
    float4* d4 = reinterpret_cast<float4*>(dst + rr * LD + vv * 8);
    d4[0] = make_float4(f[0], f[1], f[2], f[3]);
    d4[1] = make_float4(f[4], f[5], f[6], f[7]);
  }
}

// fp32 source rounded to bf16 first, so the arithmetic matches a bf16 dO.
template <int D>
__device__ void load_tile_f32(float* dst, const float* base, long long row_stride, int row0,
                              int nrows_valid) {
  constexpr int LD = D + 4;
  constexpr int VPR = D / 4;
  for (int e = threadIdx.x; e < TS * VPR; e += blockDim.x) {
    const int rr = e / VPR, vv = e % VPR;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (rr < nrows_valid) {
      t = *reinterpret_cast<const float4*>(base + (long long)(row0 + rr) * row_stride + vv * 4);
      t.x = __bfloat162float(__float2bfloat16_rn(t.x));
      t.y = __bfloat162float(__float2bfloat16_rn(t.y));
      t.z = __bfloat162float(__float2bfloat16_rn(t.z));
      t.w = __bfloat162float(__float2bfloat16_rn(t.w));
    }
    *reinterpret_cast<float4*>(dst + rr * LD + vv * 4) = t;
  }
}

// acc[i][j] += sum_d A[ty + 16 i][d] * B[tx + 16 j][d]
template <int D>
__device__ __forceinline__ void gemm_nt(const float* A, const float* B, float (&acc)[4][4], int ty,
                                        int tx) {
  constexpr int LD = D + 4;
#pragma unroll 4
  for (int d = 0; d < D; d += 4) {
    float4 a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4*>(A + (ty + 16 * i) * LD + d);
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = *reinterpret_cast<const float4*>(B + (tx + 16 * j) * LD + d);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j)
        acc[i][j] += a[i].x * b[j].x + a[i].y * b[j].y + a[i].z * b[j].z + a[i].w * b[j].w;
  }
}

// acc[i][h] (float4 at columns tx*4 + 64 h) += sum_j P[ty + 16 i][j] * M[j][cols]
template <int D>
__device__ __forceinline__ void gemm_nn(const float* P, const float* M, float4 (&acc)[4][D / 64],
                                        int ty, int tx) {
  constexpr int LD = D + 4;
#pragma unroll 2
  for (int j = 0; j < TS; j += 4) {
    float4 p[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = *reinterpret_cast<const float4*>(P + (ty + 16 * i) * LDS_ + j);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      float4 m[D / 64];
#pragma unroll
      for (int h = 0; h < D / 64; ++h)
        m[h] = *reinterpret_cast<const float4*>(M + (j + jj) * LD + tx * 4 + 64 * h);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float pv = jj == 0 ? p[i].x : jj == 1 ? p[i].y : jj == 2 ? p[i].z : p[i].w;
#pragma unroll
        for (int h = 0; h < D / 64; ++h) {
          acc[i][h].x += pv * m[h].x;
          acc[i][h].y += pv * m[h].y;
          acc[i][h].z += pv * m[h].z;
          acc[i][h].w += pv * m[h].w;
        }
      }
    }
  }
}

__device__ __forceinline__ float group16_max(float x) {
#pragma unroll
  for (int o = 8; o >= 1; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float group16_sum(float x) {
#pragma unroll
  for (int o = 8; o >= 1; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

template <int D>
__device__ __forceinline__ void store_rows_bf16(__nv_bfloat16* base, long long row_stride, int row0,
                                                int nrows_valid, const float4 (&acc)[4][D / 64],
                                                const float (&mul)[4], int ty, int tx) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int rr = ty + 16 * i;
    if (rr >= nrows_valid) continue;
#pragma unroll
    for (int h = 0; h < D / 64; ++h) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(acc[i][h].x * mul[i], acc[i][h].y * mul[i]);
      __nv_bfloat162 hi = __floats2bfloat162_rn(acc[i][h].z * mul[i], acc[i][h].w * mul[i]);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(base + (long long)(row0 + rr) * row_stride + tx * 4 + 64 * h) = pk;
    }
  }
}

// ---------------------------------------------------------------- backward: Delta
// delta[b,h,t] = sum_d dO * O, and an optional bf16 copy of an fp32 dO.
template <bool kF32>
__global__ void bwd_delta_kernel(int N, int Hq, int D, long long rows, const void* __restrict__ d_o,
                                 const __nv_bfloat16* __restrict__ o, float* __restrict__ delta) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long rw = warp; rw < rows; rw += nwarps) {  // rw = (b*N + t)*Hq + h
    float acc = 0.f;
    for (int d = lane; d < D; d += 32) {
      float x;
      if (kF32)
        x = __bfloat162float(__float2bfloat16_rn(reinterpret_cast<const float*>(d_o)[rw * D + d]));
      else
        x = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(d_o)[rw * D + d]);
      acc += x * __bfloat162float(o[rw * D + d]);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) {
      const int h = (int)(rw % Hq);
      const long long bt = rw / Hq;
      const int t = (int)(bt % N);
      const long long b = bt / N;
      delta[(b * Hq + h) * N + t] = acc;
    }
  }
}

// ---------------------------------------------------------------- backward: dQ (query-tile outer)
template <int D>
__global__ void __launch_bounds__(256)
bwd_dq_simt_kernel(Geom g, int Hq, int Hkv, float scale, int dout_f32,
                   const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, const void* __restrict__ d_o,
                   const float* __restrict__ lse, const float* __restrict__ delta,
                   __nv_bfloat16* __restrict__ dq) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* dOs = Qs + TS * LD;
  float* Ks = dOs + TS * LD;
  float* Vs = Ks + TS * LD;
  float* Ss = Vs + TS * LD;
  const int ntiles = (g.N + TS - 1) / TS;
  const int qt = ntiles - 1 - blockIdx.x;
  const int h = blockIdx.y, b = blockIdx.z, hk = h / (Hq / Hkv);
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const int row0 = qt * TS, nrows = min(TS, g.N - row0);
  const long long qs = (long long)Hq * D, ks = (long long)Hkv * D;
  const long long qoff = ((long long)b * g.N * Hq + h) * D;
  load_tile_bf16<D>(Qs, q + qoff, qs, row0, nrows);
  if (dout_f32)
    load_tile_f32<D>(dOs, reinterpret_cast<const float*>(d_o) + qoff, qs, row0, nrows);
  else
    load_tile_bf16<D>(dOs, reinterpret_cast<const __nv_bfloat16*>(d_o) + qoff, qs, row0, nrows);
  const __nv_bfloat16* kb = k + ((long long)b * g.N * Hkv + hk) * D;
  const __nv_bfloat16* vb = v + ((long long)b * g.N * Hkv + hk) * D;

  RowIv iv[4];
  float L[4], dl[4];
  float4 acc[4][D / 64];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = min(row0 + ty + 16 * i, g.N - 1);
    iv[i] = row_intervals(g, row);
    L[i] = lse[((long long)b * Hq + h) * g.N + row];
    dl[i] = delta[((long long)b * Hq + h) * g.N + row];
#pragma unroll
    for (int hh = 0; hh < D / 64; ++hh) acc[i][hh] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int kt = 0; kt < ntiles; ++kt) {
    const int col0 = kt * TS, ncols = min(TS, g.N - col0);
    if (!tile_any_visible(g, row0, row0 + nrows - 1, col0, col0 + ncols - 1)) continue;
    __syncthreads();
    load_tile_bf16<D>(Ks, kb, ks, col0, ncols);
    load_tile_bf16<D>(Vs, vb, ks, col0, ncols);
    __syncthreads();
    float sc[4][4] = {}, dp[4][4] = {};
    gemm_nt<D>(Qs, Ks, sc, ty, tx);
    gemm_nt<D>(dOs, Vs, dp, ty, tx);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = col0 + tx + 16 * j;
        const bool ok = col < g.N && visible(g, iv[i], col);
        const float p = ok ? __expf(sc[i][j] * scale - L[i]) : 0.f;
        Ss[(ty + 16 * i) * LDS_ + tx + 16 * j] = p * (dp[i][j] - dl[i]);
      }
    __syncthreads();
    gemm_nn<D>(Ss, Ks, acc, ty, tx);
  }
  float mul[4] = {scale, scale, scale, scale};
  store_rows_bf16<D>(dq + qoff, qs, row0, nrows, acc, mul, ty, tx);
}

// ---------------------------------------------------------------- backward: dK, dV (key-tile outer)
// One thread block owns a 64-key tile of one KV head and walks every query tile of every query
// head of the group that can see it, so dK and dV are accumulated in registers without atomics.
template <int D>
__global__ void __launch_bounds__(256)
bwd_dkdv_simt_kernel(Geom g, int Hq, int Hkv, float scale, int dout_f32,
                     const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, const void* __restrict__ d_o,
                     const float* __restrict__ lse, const float* __restrict__ delta,
                     __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Ks = smem;
  float* Vs = Ks + TS * LD;
  float* Qs = Vs + TS * LD;
  float* dOs = Qs + TS * LD;
  float* Pt = dOs + TS * LD;      // [key][query]
  float* dSt = Pt + TS * LDS_;    // [key][query]
  float* Ls = dSt + TS * LDS_;    // LSE of the query tile
  float* Dl = Ls + TS;            // Delta of the query tile
  const int ntiles = (g.N + TS - 1) / TS;
  const int kt = blockIdx.x;
  const int hk = blockIdx.y, b = blockIdx.z, G = Hq / Hkv;
  const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
  const int col0 = kt * TS, ncols = min(TS, g.N - col0);
  const long long qs = (long long)Hq * D, ks = (long long)Hkv * D;
  const long long koff = ((long long)b * g.N * Hkv + hk) * D;
  load_tile_bf16<D>(Ks, k + koff, ks, col0, ncols);
  load_tile_bf16<D>(Vs, v + koff, ks, col0, ncols);
  float4 acck[4][D / 64], accv[4][D / 64];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int hh = 0; hh < D / 64; ++hh) acck[i][hh] = accv[i][hh] = make_float4(0.f, 0.f, 0.f, 0.f);

  for (int qt = 0; qt < ntiles; ++qt) {
    const int row0 = qt * TS, nrows = min(TS, g.N - row0);
    if (!tile_any_visible(g, row0, row0 + nrows - 1, col0, col0 + ncols - 1)) continue;
    RowIv iv[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) iv[j] = row_intervals(g, min(row0 + tx + 16 * j, g.N - 1));
    for (int gq = 0; gq < G; ++gq) {
      const int h = hk * G + gq;
      const long long qoff = ((long long)b * g.N * Hq + h) * D;
      __syncthreads();
      load_tile_bf16<D>(Qs, q + qoff, qs, row0, nrows);
      if (dout_f32)
        load_tile_f32<D>(dOs, reinterpret_cast<const float*>(d_o) + qoff, qs, row0, nrows);
      else
        load_tile_bf16<D>(dOs, reinterpret_cast<const __nv_bfloat16*>(d_o) + qoff, qs, row0, nrows);
      if (threadIdx.x < TS) {
        const int row = min(row0 + (int)threadIdx.x, g.N - 1);
        Ls[threadIdx.x] = lse[((long long)b * Hq + h) * g.N + row];
        Dl[threadIdx.x] = delta[((long long)b * Hq + h) * g.N + row];
      }
      __syncthreads();
      float st[4][4] = {}, dpt[4][4] = {};  // [key i][query j]
      gemm_nt<D>(Ks, Qs, st, ty, tx);
      gemm_nt<D>(Vs, dOs, dpt, ty, tx);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int qr = tx + 16 * j, kc = ty + 16 * i;
          const bool ok = qr < nrows && kc < ncols && visible(g, iv[j], col0 + kc);
          const float p = ok ? __expf(st[i][j] * scale - Ls[qr]) : 0.f;
          Pt[kc * LDS_ + qr] = p;
          dSt[kc * LDS_ + qr] = p * (dpt[i][j] - Dl[qr]);
        }
      __syncthreads();
      gemm_nn<D>(Pt, dOs, accv, ty, tx);
      gemm_nn<D>(dSt, Qs, acck, ty, tx);
    }
  }
  float one[4] = {1.f, 1.f, 1.f, 1.f}, sc4[4] = {scale, scale, scale, scale};
  store_rows_bf16<D>(dv + koff, ks, col0, ncols, accv, one, ty, tx);
  store_rows_bf16<D>(dk + koff, ks, col0, ncols, acck, sc4, ty, tx);
}

template <typename K>
int32_t set_smem(K kernel, size_t bytes) {
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  return UNIGIST_OK;
}

}  // namespace

int32_t launch_bwd_simt(const Geom& g, const unigist_problem& p, float scale, const void* q,
                        const void* k, const void* v, const void* o, const float* lse,
                        const void* d_o, void* dq, void* dk, void* dv, float* delta,
                        cudaStream_t st) {
  const int ntiles = (g.N + TS - 1) / TS;
  const int f32 = (p.flags & UNIGIST_FLAG_DOUT_FP32) ? 1 : 0;
  const long long rows = (long long)p.batch * g.N * p.num_q_heads;
  {
    const int blocks = (int)((rows + 7) / 8 < 148 * 16 ? (rows + 7) / 8 : 148 * 16);
    KernelScope ks("bwd_delta_kernel", st);
    if (f32)
      bwd_delta_kernel<true><<<blocks, 256, 0, st>>>(g.N, p.num_q_heads, p.head_dim, rows, d_o,
                                                     (const __nv_bfloat16*)o, delta);
    else
      bwd_delta_kernel<false><<<blocks, 256, 0, st>>>(g.N, p.num_q_heads, p.head_dim, rows, d_o,
                                                      (const __nv_bfloat16*)o, delta);
  }
  if (int32_t rc = check_launch("delta kernel")) return rc;
  auto go = [&](auto kq, auto kkv, int D) -> int32_t {
    const size_t smem_q = (size_t)(4 * TS * (D + 4) + TS * LDS_) * sizeof(float);
    const size_t smem_kv = (size_t)(4 * TS * (D + 4) + 2 * TS * LDS_ + 2 * TS) * sizeof(float);
    if (int32_t rc = set_smem(kq, smem_q)) return rc;
    if (int32_t rc = set_smem(kkv, smem_kv)) return rc;
    {
      KernelScope ks("bwd_dq_simt_kernel", st);
      kq<<<dim3(ntiles, p.num_q_heads, p.batch), 256, smem_q, st>>>(
          g, p.num_q_heads, p.num_kv_heads, scale, f32, (const __nv_bfloat16*)q,
          (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, d_o, lse, delta, (__nv_bfloat16*)dq);
    }
    if (int32_t rc = check_launch("dQ kernel")) return rc;
    {
      KernelScope ks("bwd_dkdv_simt_kernel", st);
      kkv<<<dim3(ntiles, p.num_kv_heads, p.batch), 256, smem_kv, st>>>(
          g, p.num_q_heads, p.num_kv_heads, scale, f32, (const __nv_bfloat16*)q,
          (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, d_o, lse, delta, (__nv_bfloat16*)dk,
          (__nv_bfloat16*)dv);
    }
    return check_launch("dK/dV kernel");
  };
  return p.head_dim == 64 ? go(bwd_dq_simt_kernel<64>, bwd_dkdv_simt_kernel<64>, 64)
                          : go(bwd_dq_simt_kernel<128>, bwd_dkdv_simt_kernel<128>, 128);
}

}  // namespace ug
