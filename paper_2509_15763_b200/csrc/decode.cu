// Decode attention over the compacted, paged KV cache (Section 4.3): one query per sequence,
// every cache entry visible.  Split over keys: each thread block streams a contiguous range of
// 64-token pages of one (sequence, KV head) through shared memory with 16-byte asynchronous
// copies (a page of one KV head is one contiguous 64 * D * 2 byte run), keeps a running
// (max, sum, output) for the G query heads that share the KV head, and a second kernel merges
// the splits.  HBM-bound: K and V are read exactly once.
#include <cmath>

#include "ug_common.cuh"

namespace ug {
namespace {

constexpr int PG = UNIGIST_PAGE_TOKENS;
constexpr int DD = 128;                     // head_dim
constexpr int STAGES = 3;
constexpr int PAGE_BYTES = PG * DD * 2;     // one K (or V) page of one KV head
constexpr int THREADS = 256;
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// Partial results per (seq, q head, split): o[D] unnormalised, then m (log2 domain), l.
template <int G>
__global__ void __launch_bounds__(THREADS, 2)
decode_split_kernel(int Hq, int Hkv, float scale_log2, const __nv_bfloat16* __restrict__ q,
                    const __nv_bfloat16* __restrict__ kc, const __nv_bfloat16* __restrict__ vc,
                    int num_blocks, const int32_t* __restrict__ table, int max_blocks,
                    const int32_t* __restrict__ seq_lens, int splits, int blocks_per_split,
                    float* __restrict__ part) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* stage = smem_raw;                                     // STAGES * 2 * PAGE_BYTES
  float* sc = reinterpret_cast<float*>(smem_raw + STAGES * 2 * PAGE_BYTES);  // [G][PG]
  float* run_m = sc + G * PG;                                         // [G]
  float* run_l = run_m + G;
  float* fac = run_l + G;
  const int split = blockIdx.x, hk = blockIdx.y, seq = blockIdx.z;
  const int tid = threadIdx.x;
  const int len = seq_lens[seq];
  const int nblk = (len + PG - 1) / PG;
  const int b0 = min(split * blocks_per_split, nblk);
  const int b1 = min(b0 + blocks_per_split, min(nblk, max_blocks));
  const int32_t* row = table + (long long)seq * max_blocks;

  // query fragments: thread (c = tid % 8) owns elements [8c, 8c+8) and [64+8c, 64+8c+8)
  const int c8 = tid & 7;
  float qf[G][16];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const __nv_bfloat16* qp = q + ((long long)seq * Hq + hk * G + g) * DD;
    float a[8], b[8];
    unpack8(*reinterpret_cast<const uint4*>(qp + c8 * 8), a);
    unpack8(*reinterpret_cast<const uint4*>(qp + 64 + c8 * 8), b);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      qf[g][e] = a[e] * scale_log2;
      qf[g][8 + e] = b[e] * scale_log2;
    }
  }
  if (tid < G) {
    run_m[tid] = -INFINITY;
    run_l[tid] = 0.f;
  }
  float acc[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[g][e] = 0.f;

  auto issue = [&](int blk_idx, int st) {
    if (blk_idx < b1) {
      int phys = row[blk_idx];
      phys = min(max(phys, 0), num_blocks - 1);  // never read outside the cache
      const char* ksrc = reinterpret_cast<const char*>(kc) + ((long long)phys * Hkv + hk) * PAGE_BYTES;
      const char* vsrc = reinterpret_cast<const char*>(vc) + ((long long)phys * Hkv + hk) * PAGE_BYTES;
      unsigned char* kd = stage + st * 2 * PAGE_BYTES;
      unsigned char* vd = kd + PAGE_BYTES;
#pragma unroll
      for (int i = 0; i < PAGE_BYTES / 16 / THREADS; ++i) {
        const int off = (i * THREADS + tid) * 16;
        cp_async16(kd + off, ksrc + off);
        cp_async16(vd + off, vsrc + off);
      }
    }
    cp_async_commit();  // empty groups keep the wait arithmetic uniform
  };

#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) issue(b0 + s, s);

  for (int blk = b0; blk < b1; ++blk) {
    const int st = (blk - b0) % STAGES;
    cp_async_wait<STAGES - 2>();
    __syncthreads();  // page `blk` has landed; everyone is done with the stage refilled next
    issue(blk + STAGES - 1, (blk - b0 + STAGES - 1) % STAGES);
    const unsigned char* ks = stage + st * 2 * PAGE_BYTES;
    const unsigned char* vs = ks + PAGE_BYTES;
    const int nvalid = min(PG, len - blk * PG);

    // scores: 8 threads per token, 32 tokens per pass
#pragma unroll
    for (int pass = 0; pass < PG / 32; ++pass) {
      const int tok = pass * 32 + (tid >> 3);
      float ka[8], kb[8];
      unpack8(*reinterpret_cast<const uint4*>(ks + tok * (DD * 2) + c8 * 16), ka);
      unpack8(*reinterpret_cast<const uint4*>(ks + tok * (DD * 2) + 128 + c8 * 16), kb);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) d += qf[g][e] * ka[e] + qf[g][8 + e] * kb[e];
        d += __shfl_xor_sync(0xffffffffu, d, 1);
        d += __shfl_xor_sync(0xffffffffu, d, 2);
        d += __shfl_xor_sync(0xffffffffu, d, 4);
        if (c8 == 0) sc[g * PG + tok] = tok < nvalid ? d : -INFINITY;
      }
    }
    __syncthreads();
    // running softmax: warp g owns query head g
    if ((tid >> 5) < G) {
      const int g = tid >> 5, lane = tid & 31;
      const float s0 = sc[g * PG + lane], s1 = sc[g * PG + 32 + lane];
      float mx = fmaxf(s0, s1);
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float mo = run_m[g];
      const float mn = fmaxf(mo, mx);  // finite: token 0 of the page is always valid
      const float p0 = exp2f(s0 - mn), p1 = exp2f(s1 - mn);
      float ps = p0 + p1;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      sc[g * PG + lane] = p0;
      sc[g * PG + 32 + lane] = p1;
      if (lane == 0) {
        const float f = exp2f(mo - mn);
        fac[g] = f;
        run_l[g] = run_l[g] * f + ps;
        run_m[g] = mn;
      }
    }
    __syncthreads();
    // O += P V: thread owns 8 output columns (piece) for 4 tokens of the page
    {
      const int piece = tid & 15, tg = tid >> 4;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float f = fac[g];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[g][e] *= f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = tg * 4 + i;
        if (tok < nvalid) {
          float vf[8];
          unpack8(*reinterpret_cast<const uint4*>(vs + tok * (DD * 2) + piece * 16), vf);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float p = sc[g * PG + tok];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[g][e] += p * vf[e];
          }
        }
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();
  // reduce the 16 token groups through shared memory (the page stages are free now)
  float* red = reinterpret_cast<float*>(stage);  // [16][G][DD]
  {
    const int piece = tid & 15, tg = tid >> 4;
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < 8; ++e) red[(tg * G + g) * DD + piece * 8 + e] = acc[g][e];
  }
  __syncthreads();
  for (int idx = tid; idx < G * DD; idx += THREADS) {
    const int g = idx / DD, d = idx % DD;
    float s = 0.f;
#pragma unroll
    for (int tg = 0; tg < 16; ++tg) s += red[(tg * G + g) * DD + d];
    const long long slot = ((long long)seq * Hq + hk * G + g) * splits + split;
    part[slot * (DD + 2) + d] = s;
    if (d == 0) {
      part[slot * (DD + 2) + DD] = run_m[g];
      part[slot * (DD + 2) + DD + 1] = run_l[g];
    }
  }
}

// One block per (seq, q head): merge the splits.
__global__ void __launch_bounds__(DD)
decode_combine_kernel(int splits, const float* __restrict__ part, __nv_bfloat16* __restrict__ o,
                      float* __restrict__ lse) {
  const long long sh = blockIdx.x;
  const float* base = part + sh * splits * (DD + 2);
  float M = -INFINITY;
  for (int i = 0; i < splits; ++i) M = fmaxf(M, base[i * (DD + 2) + DD]);
  float L = 0.f, acc = 0.f;
  for (int i = 0; i < splits; ++i) {
    const float m = base[i * (DD + 2) + DD];
    const float w = m == -INFINITY ? 0.f : exp2f(m - M);
    L += w * base[i * (DD + 2) + DD + 1];
    acc += w * base[i * (DD + 2) + threadIdx.x];
  }
  o[sh * DD + threadIdx.x] = __float2bfloat16_rn(acc / L);
  if (lse && threadIdx.x == 0) lse[sh] = (M + log2f(L)) * 0.6931471805599453f;
}

size_t split_smem(int G) { return (size_t)STAGES * 2 * PAGE_BYTES + (size_t)(G * PG + 3 * G) * sizeof(float); }

}  // namespace

// Pick the split count that fills whole waves of 2 blocks per SM on 148 SMs.
int decode_num_splits(int S, int Hkv, int max_blocks) {
  const long long slots = 148 * 2;
  const long long base = (long long)S * Hkv;
  int best = 1;
  double best_eff = -1.0;
  for (int sp = 1; sp <= 32; ++sp) {
    const int bps = (max_blocks + sp - 1) / sp;
    if (sp > 1 && bps < 4) break;
    if ((max_blocks + bps - 1) / bps != sp) continue;  // this count leaves an empty split
    const double waves = (double)(base * sp) / (double)slots;
    const double eff = waves / ceil(waves);
    if (eff > best_eff + 1e-9) {
      best_eff = eff;
      best = sp;
    }
  }
  return best;
}

int32_t launch_decode(int S, int Hq, int Hkv, int D, float scale, const void* q, const void* kc,
                      const void* vc, int num_blocks, const int32_t* table, int max_blocks,
                      const int32_t* seq_lens, void* o, float* lse, void* ws, cudaStream_t st) {
  (void)D;
  const int G = Hq / Hkv;
  const int splits = decode_num_splits(S, Hkv, max_blocks);
  const int bps = (max_blocks + splits - 1) / splits;
  dim3 grid(splits, Hkv, S);
  auto go = [&](auto kern, int g) -> int32_t {
    const size_t smem = split_smem(g);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    {
      KernelScope ks("decode_split_kernel", st);
      kern<<<grid, THREADS, smem, st>>>(Hq, Hkv, scale * LOG2E, (const __nv_bfloat16*)q,
                                        (const __nv_bfloat16*)kc, (const __nv_bfloat16*)vc, num_blocks,
                                        table, max_blocks, seq_lens, splits, bps, (float*)ws);
    }
    return check_launch("decode split kernel");
  };
  int32_t rc;
  switch (G) {
    case 1: rc = go(decode_split_kernel<1>, 1); break;
    case 2: rc = go(decode_split_kernel<2>, 2); break;
    case 4: rc = go(decode_split_kernel<4>, 4); break;
    case 8: rc = go(decode_split_kernel<8>, 8); break;
    default: return fail(UNIGIST_ERR_UNSUPPORTED, "decode supports 1, 2, 4 or 8 query heads per KV head, got %d", G);
  }
  if (rc) return rc;
  {
    KernelScope ks("decode_combine_kernel", st);
    decode_combine_kernel<<<S * Hq, DD, 0, st>>>(splits, (const float*)ws, (__nv_bfloat16*)o, lse);
  }
  return check_launch("decode combine kernel");
}

}  // namespace ug

// ------------------------------------------------------------------------------------------------
// Decode without caller-provided scratch.  The split-KV partial results go to a fixed array that
// is part of the library image, so this entry point needs no allocation from anyone.
#include <cmath>
#include <mutex>

namespace {

// Lives in the global memory of every GPU that loads the library, from load until process exit.
static __device__ __align__(256) unsigned char g_decode_static_scratch[UNIGIST_DECODE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_scratch_ptr[kMaxDevices] = {};

// In host code the array's name is only a handle; the device address has to be asked for, once
// per device, with that device current.
int32_t static_scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return ug::fail(UNIGIST_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return ug::fail(UNIGIST_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_scratch_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_decode_static_scratch);
    if (e != cudaSuccess || !ptr)
      return ug::fail(UNIGIST_ERR_CUDA, "cudaGetSymbolAddress(static decode scratch): %s", cudaGetErrorString(e));
    g_static_scratch_ptr[dev] = ptr;
  }
  *out = g_static_scratch_ptr[dev];
  return UNIGIST_OK;
}

}  // namespace

extern "C" int32_t unigist_decode_static(int32_t S, int32_t Hq, int32_t Hkv, int32_t D, float softmax_scale,
                                         const void* q, const void* kc, const void* vc, int32_t num_blocks,
                                         const int32_t* table, int32_t max_blocks, const int32_t* seq_lens,
                                         void* o, float* lse, void* stream) {
  using namespace ug;
  if (S < 1 || Hq < 1 || Hkv < 1 || max_blocks < 1 || num_blocks < 1)
    return fail(UNIGIST_ERR_INVALID_ARG, "decode has a non-positive size");
  if (Hq % Hkv) return fail(UNIGIST_ERR_SHAPE, "num_q_heads %d is not a multiple of num_kv_heads %d", Hq, Hkv);
  if (D != 128) return fail(UNIGIST_ERR_SHAPE, "decode supports head_dim 128, got %d", D);
  const int G = Hq / Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8)
    return fail(UNIGIST_ERR_UNSUPPORTED, "decode supports 1, 2, 4 or 8 query heads per KV head, got %d", G);
  if (!q || !kc || !vc || !table || !seq_lens || !o) return fail(UNIGIST_ERR_INVALID_ARG, "a pointer is NULL");
  if (!aligned16(q) || !aligned16(kc) || !aligned16(vc) || !aligned16(o))
    return fail(UNIGIST_ERR_ALIGNMENT, "tensor pointers must be 16-byte aligned");
  if (!(softmax_scale >= 0.f) || std::isinf(softmax_scale))
    return fail(UNIGIST_ERR_INVALID_ARG, "softmax_scale must be finite and >= 0");
  const size_t need = unigist_decode_workspace_bytes(S, Hq, Hkv, D, max_blocks);
  if (need > (size_t)UNIGIST_DECODE_STATIC_SCRATCH_BYTES)
    return fail(UNIGIST_ERR_WORKSPACE,
                "this decode needs %zu bytes of scratch but the built-in array holds %zu: use unigist_decode "
                "with a caller-provided workspace, or decode fewer sequences per call",
                need, (size_t)UNIGIST_DECODE_STATIC_SCRATCH_BYTES);
  void* scratch = nullptr;
  if (int32_t rc = static_scratch_address(&scratch)) return rc;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
  return launch_decode(S, Hq, Hkv, D, scale, q, kc, vc, num_blocks, table, max_blocks, seq_lens, o, lse, scratch,
                       (cudaStream_t)stream);
}
