// Decode attention over the compacted, paged KV cache (Section 4.3): one query per sequence,
// every cache entry visible.  Split over keys: each thread block streams a contiguous range of
// 64-token pages of one (sequence, KV head) through a ring in shared memory and a second kernel
// merges the splits.  HBM-bound: K and V are read exactly once.
//   producer warp:  per page one K and one V tile (64 tokens x 128 dims, 16 KB each) by TMA, 128-byte
//                   swizzle, into a 3-stage ring guarded by full / empty mbarriers; two thread blocks
//                   per SM keep about 128 KB of loads in flight.
//   consumer warps: three warps, one per ring stage, each takes every third page on its own and keeps a running
//                   (max, sum, output) for the G query heads of the KV head: S = Q K^T and O += P V
//                   with warp-level mma (m16n8k16, query heads padded to 16 rows), fragments
//                   fetched with ldmatrix.  The warps merge once, at the end.
#include <cmath>

#include "sm100_ptx.cuh"
#include "ug_common.cuh"

namespace ug {
namespace {

using namespace sm100;

constexpr int PG = UNIGIST_PAGE_TOKENS;
constexpr int DD = 128;                     // head_dim
constexpr int STAGES = 3;
constexpr int PAGE_BYTES = PG * DD * 2;     // one K (or V) page of one KV head
constexpr int SLAB_BYTES = PAGE_BYTES / 2;  // [64 tokens x 64 dims], rows of 128 bytes
constexpr int STAGE_BYTES = 2 * PAGE_BYTES;
constexpr int kConsumers = STAGES;  // page i lives in stage i % STAGES and belongs to warp i % STAGES: every barrier
                                    // has one waiter, which sees each of its phases in turn
constexpr int THREADS = (kConsumers + 1) * 32;
constexpr float LOG2E = 1.4426950408889634f;

__device__ unsigned int g_decode_timeout = 0;

__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D (16x8 fp32) += A (16x16 bf16, row) * B (16x8 bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct DecSmem {
  static constexpr int kOffBars = STAGES * STAGE_BYTES;
  static constexpr int kOffMerge = kOffBars + 64;                      // [warps][8 heads][128 + 2] fp32
  static constexpr int kBytes = kOffMerge + kConsumers * 8 * (DD + 2) * 4 + 1024 /*align*/;
};

// Partial results per (seq, q head, split): o[D] unnormalised, then m (log2 domain), l.
__global__ void __launch_bounds__(THREADS, 2)
decode_split_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, int Hq,
                    int Hkv, int G, float scale_log2, const __nv_bfloat16* __restrict__ q, int num_blocks,
                    const int32_t* __restrict__ table, int max_blocks, const int32_t* __restrict__ seq_lens,
                    int splits, int blocks_per_split, float* __restrict__ part, const int32_t* __restrict__ holes,
                    int holes_stride, int holes_off) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* gen = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bars = base + DecSmem::kOffBars;  // full[s] at + 8 s, empty[s] at + 8 (STAGES + s)
  float* merge = reinterpret_cast<float*>(gen + DecSmem::kOffMerge);
  const int split = blockIdx.x, hk = blockIdx.y, seq = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int len = seq_lens[seq];
  const int nblk = (len + PG - 1) / PG;
  const int b0 = min(split * blocks_per_split, nblk);
  const int b1 = min(b0 + blocks_per_split, min(nblk, max_blocks));
  const int npages = b1 - b0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bars + 8 * i, 1);
      mbar_init(bars + 8 * (STAGES + i), 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  bool ok = true;

  if (warp == kConsumers) {
    // ------------------------------------------------------------ producer
    const int32_t* row = table + (long long)seq * max_blocks;
    int32_t phys_mine = 0;
    for (int i = 0; i < npages && ok; ++i) {
      if ((i & 31) == 0) {  // the next 32 block-table entries, one per lane
        const int idx = b0 + i + lane;
        phys_mine = idx < b1 ? row[idx] : 0;
        phys_mine = min(max(phys_mine, 0), num_blocks - 1);  // never read outside the cache
      }
      const int phys = __shfl_sync(0xffffffffu, phys_mine, i & 31);
      const int st = i % STAGES, use = i / STAGES;
      if (use > 0) ok = mbar_wait_warp(bars + 8 * (STAGES + st), (use - 1) & 1);
      if (!ok) break;
      if (lane == 0) {
        const uint32_t full = bars + 8 * st, dst = base + st * STAGE_BYTES;
        const int row0 = (phys * Hkv + hk) * PG;
        mbar_arrive_expect_tx(full, STAGE_BYTES);
        tma_load_2d(dst, &tm_k, full, 0, row0);
        tma_load_2d(dst + SLAB_BYTES, &tm_k, full, 64, row0);
        tma_load_2d(dst + PAGE_BYTES, &tm_v, full, 0, row0);
        tma_load_2d(dst + PAGE_BYTES + SLAB_BYTES, &tm_v, full, 64, row0);
      }
      __syncwarp();
    }
    if (!ok && lane == 0) atomicExch(&g_decode_timeout, 1u);
  } else {
    // ------------------------------------------------------------ consumer: pages warp, warp + 3, ...
    const int g = lane >> 2, qc = lane & 3;  // query head (row of the padded 16 x 128 Q), column pair
    // A fragments of Q for the 8 k-steps of 16 dims: rows 8..15 are padding (zero)
    uint32_t qa0[8], qa2[8];
    {
      const __nv_bfloat16* qp = q + ((long long)seq * Hq + hk * G + min(g, G - 1)) * DD;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint32_t lo = *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 2 * qc);
        const uint32_t hi = *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 8 + 2 * qc);
        qa0[ks] = g < G ? lo : 0u;
        qa2[ks] = g < G ? hi : 0u;
      }
    }
    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[i][e] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;  // of row g (the 4 lanes of a quad hold the same values)
    const int lr = lane & 7, lj = lane >> 3;  // ldmatrix: this lane supplies row lr of matrix lj

    for (int i = warp; i < npages && ok; i += kConsumers) {
      const int st = i % STAGES, use = i / STAGES;
      ok = mbar_wait_warp(bars + 8 * st, use & 1);
      if (!ok) break;
      const uint32_t sK = base + st * STAGE_BYTES, sV = sK + PAGE_BYTES;
      const int nvalid = min(PG, len - (b0 + i) * PG);
      // cache slots that were freed and not yet reused (a decoding loop's eviction list) hold stale tokens
      unsigned long long hole_bits = 0ull;
      if (holes) {
        const int32_t* hs = holes + (long long)seq * holes_stride;
        const int nh = hs[2];
        for (int h2 = 0; h2 < nh; ++h2) {
          const int pos = hs[holes_off + h2] - (b0 + i) * PG;
          if (pos >= 0 && pos < PG) hole_bits |= 1ull << pos;
        }
      }
      // S = Q K^T: 8 token tiles of 8, fp32
      float s[8][4];
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
        const int t = 8 * nt + lr;  // token whose row address this lane supplies
#pragma unroll
        for (int kq = 0; kq < 4; ++kq) {  // 32 dims = 4 chunks of 16 bytes per ldmatrix.x4
          const int chunk = (kq & 1) * 4 + lj;
          uint32_t k0, k1, k2, k3;
          ldsm_x4(sK + (kq >> 1) * SLAB_BYTES + t * 128 + ((chunk ^ (t & 7)) << 4), k0, k1, k2, k3);
          mma_bf16(s[nt], qa0[2 * kq], 0u, qa2[2 * kq], 0u, k0, k1);
          mma_bf16(s[nt], qa0[2 * kq + 1], 0u, qa2[2 * kq + 1], 0u, k2, k3);
        }
      }
      // running softmax of row g over the page's 64 tokens (this lane: tokens 8 nt + 2 qc + {0, 1})
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int tok = 8 * nt + 2 * qc;
        s[nt][0] = (tok < nvalid && !((hole_bits >> tok) & 1ull)) ? s[nt][0] * scale_log2 : -INFINITY;
        s[nt][1] = (tok + 1 < nvalid && !((hole_bits >> (tok + 1)) & 1ull)) ? s[nt][1] * scale_log2 : -INFINITY;
        mx = fmaxf(mx, fmaxf(s[nt][0], s[nt][1]));
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);
      // (a page of nothing but freed slots leaves the maximum at -inf: keep the exponent arguments finite)
      const float f = m_new == -INFINITY ? 1.f : ex2(m_run - m_new);
      m_run = m_new;
      float ps = 0.f;
      uint32_t pa[8];  // P as bf16 pairs: pa[nt] = tokens 8 nt + 2 qc + {0, 1} of row g
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const float p0 = m_new == -INFINITY ? 0.f : ex2(s[nt][0] - m_new);
        const float p1 = m_new == -INFINITY ? 0.f : ex2(s[nt][1] - m_new);
        ps += p0 + p1;
        pa[nt] = pack_bf16(p0, p1);
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      l_run = l_run * f + ps;
#pragma unroll
      for (int i2 = 0; i2 < 16; ++i2) {
        o[i2][0] *= f;
        o[i2][1] *= f;
      }
      // O += P V: 4 k-steps of 16 tokens, 16 dim tiles of 8
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        const int t = 16 * ks + (lj & 1) * 8 + lr;
#pragma unroll
        for (int np = 0; np < 8; ++np) {  // dim tiles 2 np, 2 np + 1
          const int chunk = 2 * np + (lj >> 1);  // 16-byte chunk of the 256-byte V row
          uint32_t v0, v1, v2, v3;
          ldsm_x4_trans(sV + (chunk >> 3) * SLAB_BYTES + t * 128 + (((chunk & 7) ^ (t & 7)) << 4), v0, v1, v2, v3);
          mma_bf16(o[2 * np], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, v0, v1);
          mma_bf16(o[2 * np + 1], pa[2 * ks], 0u, pa[2 * ks + 1], 0u, v2, v3);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + 8 * (STAGES + st));  // the stage may be refilled
    }
    if (!ok && lane == 0) atomicExch(&g_decode_timeout, 1u);
    // this warp's partial result for row g -> shared memory
    if (g < G) {
      float* mrow = merge + (warp * 8 + g) * (DD + 2);
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        mrow[8 * nt + 2 * qc] = o[nt][0];
        mrow[8 * nt + 2 * qc + 1] = o[nt][1];
      }
      if (qc == 0) {
        mrow[DD] = m_run;
        mrow[DD + 1] = l_run;
      }
    }
  }
  __syncthreads();
  // merge the consumer warps
  for (int idx = threadIdx.x; idx < G * DD; idx += THREADS) {
    const int g = idx / DD, d = idx % DD;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kConsumers; ++w) M = fmaxf(M, merge[(w * 8 + g) * (DD + 2) + DD]);
    float acc = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumers; ++w) {
      const float* mrow = merge + (w * 8 + g) * (DD + 2);
      const float wgt = mrow[DD] == -INFINITY ? 0.f : ex2(mrow[DD] - M);
      acc += wgt * mrow[d];
      L += wgt * mrow[DD + 1];
    }
    const long long slot = ((long long)seq * Hq + hk * G + g) * splits + split;
    part[slot * (DD + 2) + d] = acc;
    if (d == 0) {
      part[slot * (DD + 2) + DD] = M;
      part[slot * (DD + 2) + DD + 1] = L;
    }
  }
}

constexpr int kMaxSplits = 32;  // one lane of a warp per split in the combine kernel

// One block per (seq, q head): merge the splits.  Lane t of the first warp takes split t's maximum and
// sum, so that all of them are in flight at once, and the warp reduces them; the weighted sum over the splits then
// runs with eight splits' loads in flight instead of one dependent load after the other.
__global__ void __launch_bounds__(DD)
decode_combine_kernel(int splits, const float* __restrict__ part, __nv_bfloat16* __restrict__ o,
                      float* __restrict__ lse) {
  __shared__ float s_w[kMaxSplits];
  __shared__ float s_ml[2];
  const long long sh = blockIdx.x;
  const float* base = part + sh * splits * (DD + 2);
  const int t = threadIdx.x;
  if (t < 32) {
    float m = -INFINITY, l = 0.f;
    if (t < splits) {
      m = base[t * (DD + 2) + DD];
      l = base[t * (DD + 2) + DD + 1];
    }
    float M = m;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    const float w = m == -INFINITY ? 0.f : exp2f(m - M);
    float L = w * l;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) L += __shfl_xor_sync(0xffffffffu, L, off);
    s_w[t] = w;
    if (t == 0) {
      s_ml[0] = M;
      s_ml[1] = L;
    }
  }
  __syncthreads();
  float acc = 0.f;
#pragma unroll 8
  for (int i = 0; i < splits; ++i) acc += s_w[i] * base[i * (DD + 2) + t];
  const float M = s_ml[0], L = s_ml[1];
  // a sequence with nothing to attend to (length 0, or every slot freed): O = 0, LSE = -inf, not 0 / 0
  o[sh * DD + t] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
  if (lse && t == 0) lse[sh] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
}

}  // namespace

// Pick the split count that fills whole waves of 2 blocks per SM.
int decode_num_splits(int S, int Hkv, int max_blocks) {
  const long long slots = (long long)sm_count() * 2;
  const long long base = (long long)S * Hkv;
  int best = 1;
  double best_eff = -1.0;
  for (int sp = 1; sp <= kMaxSplits; ++sp) {
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
                      const int32_t* seq_lens, void* o, float* lse, void* ws, cudaStream_t st, const int32_t* holes,
                      int holes_stride, int holes_off) {
  (void)D;
  const int G = Hq / Hkv;
  if (G < 1 || G > 8) return fail(UNIGIST_ERR_UNSUPPORTED, "decode supports 1 to 8 query heads per KV head, got %d", G);
  const int splits = decode_num_splits(S, Hkv, max_blocks);
  const int bps = (max_blocks + splits - 1) / splits;
  // the caches as 2-D tensors [num_blocks * Hkv * 64 tokens, 128 dims], tiles of 64 tokens x 64 dims
  CUtensorMap mk, mv;
  const long long rows = (long long)num_blocks * Hkv * PG;
  if (int32_t rc = encode_map_2d_bf16(&mk, kc, rows, DD, PG, 64)) return rc;
  if (int32_t rc = encode_map_2d_bf16(&mv, vc, rows, DD, PG, 64)) return rc;
  cudaError_t e = cudaFuncSetAttribute(decode_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       DecSmem::kBytes);
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  {
    KernelScope ks("decode_split_kernel", st);
    decode_split_kernel<<<dim3(splits, Hkv, S), THREADS, DecSmem::kBytes, st>>>(
        mk, mv, Hq, Hkv, G, scale * LOG2E, (const __nv_bfloat16*)q, num_blocks, table, max_blocks, seq_lens, splits, bps,
        (float*)ws, holes, holes_stride, holes_off);
  }
  if (int32_t rc = check_launch("decode split kernel")) return rc;
  {
    KernelScope ks("decode_combine_kernel", st);
    decode_combine_kernel<<<S * Hq, DD, 0, st>>>(splits, (const float*)ws, (__nv_bfloat16*)o, lse);
  }
  return check_launch("decode combine kernel");
}

int32_t decode_take_timeout(bool* timed_out) {
  unsigned int flag = 0, zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&flag, g_decode_timeout, sizeof(flag));
  if (e == cudaSuccess && flag) e = cudaMemcpyToSymbol(g_decode_timeout, &zero, sizeof(zero));
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "reading the device status: %s", cudaGetErrorString(e));
  *timed_out = flag != 0;
  return UNIGIST_OK;
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
  if (Hq / Hkv > 8) return fail(UNIGIST_ERR_UNSUPPORTED, "decode supports at most 8 query heads per KV head");
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
