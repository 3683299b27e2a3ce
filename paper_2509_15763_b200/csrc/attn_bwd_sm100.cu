// Backward gist-masked attention on Blackwell tensor cores (tcgen05 + TMEM + TMA) on the SHIFTED sequence
// [sinks (s) | raw (T) | gists (n)]; a tile never straddles two of these segments.
//   bwd_prep_kernel            Delta = rowsum(dO o O) (fp32) and, for an fp32 dO, its bf16 copy; zeroes the fp32
//                              dQ accumulator of the fused kernel.
// head_dim 128: attn_bwd_fused_sm100_kernel (described where it is defined) and dq_convert_kernel.
// head_dim 64: two kernels (a 64-row dQ^T accumulator would halve the fused kernel's tensor throughput):
//   attn_bwd_dkdv_sm100_kernel one thread block owns a 128-key tile of one KV head and walks every
//                              128-query tile of every query head of the group that can see it:
//                              S^T = K Q^T and dP^T = V dO^T (TMEM), P^T = exp2(S^T c - LSE),
//                              dS^T = P^T o (dP^T - Delta), dV += P^T dO, dK += dS^T Q.  dK and dV
//                              live in TMEM for the whole block: no atomics, deterministic.
//   attn_bwd_dq_sm100_kernel   one thread block owns a 128-query tile of one query head and walks
//                              the visible 64-key tiles: S, dP, dS as above, dQ += dS K in TMEM.
// Tiles without a visible pair are never loaded; only "partial" tiles evaluate the mask.
#include <algorithm>
#include <vector>

#include "sm100_ptx.cuh"
#include "ug_common.cuh"

namespace ug {
namespace {

using namespace sm100;

constexpr float kLog2e = 1.4426950408889634f;
__device__ unsigned int g_bwd_timeout = 0;

// ------------------------------------------------------------------------------------------------
// A run of equal sequences as the per-token kernels see it: its geometry, its first packed token and its
// [batch, Hq, N] block of Delta.  One problem is one run; a packed sample (cross-document masking) has several
// and a warp finds its token's run by scanning the (at most twelve) first-token indices.
struct TokRun {
  Geom g;
  long long tok_begin;
  float* delta;
};
template <int kRuns>
struct TokRuns {
  TokRun run[kRuns];
  int n;
};


// Delta and dO conversion: one warp per token.  The token's batch index and shifted position are worked out
// once (the divisions cost more than a row's loads), then its Hq rows go by four at a time, all loads of the
// four issued before the first use; 4 elements per lane and pass.
template <bool kF32, int kRuns>
__global__ void __launch_bounds__(256)
bwd_prep_kernel(const __grid_constant__ TokRuns<kRuns> P, int interleaved, int Hq, int D, long long tokens,
                const void* __restrict__ d_o, const __nv_bfloat16* __restrict__ o,
                __nv_bfloat16* __restrict__ d_o_bf16, float* __restrict__ dq32) {
  constexpr int kHeads = 4;  // rows in flight
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long tk = warp; tk < tokens; tk += nwarps) {  // tk = packed token index (run's first token + b * N + t)
    int ri = 0;
    if constexpr (kRuns > 1)
      while (ri + 1 < P.n && tk >= P.run[ri + 1].tok_begin) ++ri;
    const Geom g = P.run[ri].g;
    const long long local = tk - P.run[ri].tok_begin;
    const long long b = local / g.N;
    const int t = (int)(local - b * g.N);
    // Delta is kept in shifted order, whatever the order of dO and O
    float* delta_tok = P.run[ri].delta + b * Hq * g.N + (interleaved ? unshift_perm(g, t) : t);
    const long long row0 = tk * Hq;
    for (int h0 = 0; h0 < Hq; h0 += kHeads) {
      float acc[kHeads];
#pragma unroll
      for (int u = 0; u < kHeads; ++u) acc[u] = 0.f;
      for (int d = lane * 4; d < D; d += 128) {
        uint2 dbits[kHeads], obits[kHeads];  // 4 bf16 of dO and of O
#pragma unroll
        for (int u = 0; u < kHeads; ++u) {
          if (h0 + u >= Hq) continue;
          const long long at = (row0 + h0 + u) * D + d;
          if (kF32) {
            const float4 x = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(d_o) + at));
            const __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y), hi = __floats2bfloat162_rn(x.z, x.w);
            dbits[u].x = *reinterpret_cast<const uint32_t*>(&lo);
            dbits[u].y = *reinterpret_cast<const uint32_t*>(&hi);
          } else {
            dbits[u] = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(d_o) + at);
          }
          obits[u] = *reinterpret_cast<const uint2*>(o + at);
        }
#pragma unroll
        for (int u = 0; u < kHeads; ++u) {
          if (h0 + u >= Hq) continue;
          const long long at = (row0 + h0 + u) * D + d;
          // the fused backward accumulates dQ into this fp32 buffer: start it at zero
          if (dq32) __stcs(reinterpret_cast<float4*>(dq32 + at), make_float4(0.f, 0.f, 0.f, 0.f));
          if (kF32) *reinterpret_cast<uint2*>(d_o_bf16 + at) = dbits[u];
          // a bf16 is the high half of an fp32
          acc[u] += __uint_as_float(dbits[u].x << 16) * __uint_as_float(obits[u].x << 16) +
                    __uint_as_float(dbits[u].x & 0xffff0000u) * __uint_as_float(obits[u].x & 0xffff0000u) +
                    __uint_as_float(dbits[u].y << 16) * __uint_as_float(obits[u].y << 16) +
                    __uint_as_float(dbits[u].y & 0xffff0000u) * __uint_as_float(obits[u].y & 0xffff0000u);
        }
      }
#pragma unroll
      for (int u = 0; u < kHeads; ++u) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], off);
      }
      if (lane < kHeads && h0 + lane < Hq) {
        float mine = acc[0];
#pragma unroll
        for (int u = 1; u < kHeads; ++u) mine = lane == u ? acc[u] : mine;
        delta_tok[(long long)(h0 + lane) * g.N] = mine;
      }
    }
  }
}

// Query rows (numbered inside the raw or the gist segment, inclusive) that see a given key:
// Eq. 3 read column-wise.  An empty interval has lo > hi.
__device__ __forceinline__ void key_q_interval(const Geom& g, bool key_is_raw, int key, bool key_valid,
                                               bool q_is_raw, int& lo, int& hi) {
  if (!key_valid) {
    lo = 1;
    hi = 0;
    return;
  }
  if (key_is_raw) {
    const int u = key / g.r;
    if (q_is_raw) {
      lo = key;
      hi = min(g.T - 1, (u + g.k + 1) * g.r - 1);
    } else {
      lo = u;
      hi = min(g.n - 1, u + g.k);
    }
  } else {
    if (q_is_raw) {
      lo = (key + 1) * g.r;
      hi = g.T - 1;
    } else {
      lo = key;
      hi = g.n - 1;
    }
  }
}

// Query rows of segment qseg (numbered inside it, inclusive) that see key `key` of segment kseg:
// Eq. 3 read column-wise, sinks included.  An empty interval has lo > hi.
__device__ __forceinline__ void key_q_interval3(const Geom& g, int kseg, int key, bool key_valid, int qseg, int& lo,
                                                int& hi) {
  lo = 1;
  hi = 0;
  if (!key_valid) return;
  if (kseg == kSegSink) {  // a sink is seen by the sinks from itself on and by every raw and gist query
    lo = qseg == kSegSink ? key : 0;
    hi = seg_len(g, qseg) - 1;
    return;
  }
  if (qseg == kSegSink) return;  // sink queries see sinks only
  key_q_interval(g, kseg == kSegRaw, key, true, qseg == kSegRaw, lo, hi);
}

// ------------------------------------------------------------------------------------------------
// dK / dV kernel
constexpr int KV_BM = 128;       // keys per block (TMEM lanes)
constexpr int KV_BN = 128;       // queries per step
constexpr int kKvThreads = 320;  // 8 compute warps, 1 TMA warp, 1 MMA warp

template <int D>
struct KvSmem {
  static constexpr int kSlab = 128 * 128;
  static constexpr int kTile = kSlab * (D / 64);
  static constexpr int kStats = 2 * 2 * KV_BN * 4;  // [stage][lse2 | delta][128] fp32
  static constexpr int kBytes = 6 * kTile + kStats + 1024 + 256;
};

template <int D>
__global__ void __launch_bounds__(kKvThreads, 1)
attn_bwd_dkdv_sm100_kernel(const __grid_constant__ CUtensorMap tm_q_sink, const __grid_constant__ CUtensorMap tm_q_raw,
                           const __grid_constant__ CUtensorMap tm_q_gist, const __grid_constant__ CUtensorMap tm_do_sink,
                           const __grid_constant__ CUtensorMap tm_do_raw, const __grid_constant__ CUtensorMap tm_do_gist,
                           const __grid_constant__ CUtensorMap tm_k_sink, const __grid_constant__ CUtensorMap tm_k_raw,
                           const __grid_constant__ CUtensorMap tm_k_gist, const __grid_constant__ CUtensorMap tm_v_sink,
                           const __grid_constant__ CUtensorMap tm_v_raw, const __grid_constant__ CUtensorMap tm_v_gist,
                           Geom g, int Hq, int Hkv, float scale, const float* __restrict__ lse,
                           const float* __restrict__ delta, __nv_bfloat16* __restrict__ dk,
                           __nv_bfloat16* __restrict__ dv, int n_sink_kt, int n_gist_kt) {
  using SM = KvSmem<D>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* gen = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t sK = base, sV = base + SM::kTile;
  const uint32_t sQ[2] = {base + 2 * SM::kTile, base + 4 * SM::kTile};
  const uint32_t sDO[2] = {base + 3 * SM::kTile, base + 5 * SM::kTile};
  float* stats = reinterpret_cast<float*>(gen + 6 * SM::kTile);  // [stage][2][128]
  const uint32_t bars = base + 6 * SM::kTile + SM::kStats;
  const uint32_t bar_kv = bars, bar_full[2] = {bars + 8, bars + 16}, bar_empty[2] = {bars + 24, bars + 32},
                 bar_S = bars + 40, bar_dP = bars + 48, bar_P = bars + 56, bar_dS = bars + 64, bar_final = bars + 72,
                 tmem_slot = bars + 80;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(gen + 6 * SM::kTile + SM::kStats + 80);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int hk = blockIdx.y, b = blockIdx.z, G = Hq / Hkv;
  // sink and gist key tiles are seen by every later query: heaviest, scheduled first
  const int rank = blockIdx.x;
  const int kseg = rank < n_sink_kt ? kSegSink : (rank < n_sink_kt + n_gist_kt ? kSegGist : kSegRaw);
  const int kt = rank - (kseg == kSegSink ? 0 : (kseg == kSegGist ? n_sink_kt : n_sink_kt + n_gist_kt));
  const int key_seg_len = seg_len(g, kseg);
  const int key_seg_base = seg_base(g, kseg);
  const int key_a = kt * KV_BM, key_b = min(key_a + KV_BM - 1, key_seg_len - 1);
  const bool key_tile_whole = key_a + KV_BM - 1 <= key_seg_len - 1;

  // query tiles that see this key tile, per query segment: first tile and count, and the bounds inside which a
  // tile is "full" (seen by the last key from t_lo on, by the first key up to t_hi)
  int lo_a, hi_a, lo_b, hi_b;
  key_q_interval3(g, kseg, key_a, true, kSegRaw, lo_a, hi_a);
  key_q_interval3(g, kseg, key_b, true, kSegRaw, lo_b, hi_b);
  const int n_raw_q = hi_b >= lo_a ? hi_b / KV_BN - lo_a / KV_BN + 1 : 0, rq_lo = lo_a / KV_BN, raw_t_lo = lo_b, raw_t_hi = hi_a;
  key_q_interval3(g, kseg, key_a, true, kSegGist, lo_a, hi_a);
  key_q_interval3(g, kseg, key_b, true, kSegGist, lo_b, hi_b);
  const int n_gist_q = hi_b >= lo_a ? hi_b / KV_BN - lo_a / KV_BN + 1 : 0, gq_lo = lo_a / KV_BN, gist_t_lo = lo_b, gist_t_hi = hi_a;
  key_q_interval3(g, kseg, key_a, true, kSegSink, lo_a, hi_a);
  key_q_interval3(g, kseg, key_b, true, kSegSink, lo_b, hi_b);
  const int n_sink_q = hi_b >= lo_a ? hi_b / KV_BN - lo_a / KV_BN + 1 : 0, sq_lo = lo_a / KV_BN, sink_t_lo = lo_b, sink_t_hi = hi_a;
  const int n_iter = (n_raw_q + n_gist_q + n_sink_q) * G;

  if (threadIdx.x == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_full[0], 1);
    mbar_init(bar_full[1], 1);
    mbar_init(bar_empty[0], 1);
    mbar_init(bar_empty[1], 1);
    mbar_init(bar_S, 1);
    mbar_init(bar_dP, 1);
    mbar_init(bar_P, 256);
    mbar_init(bar_dS, 256);
    mbar_init(bar_final, 1);
    mbar_fence_init();
  }
  if (warp == 9) tmem_alloc(tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t t_dK = tmem, t_dV = tmem + 128, t_A = tmem + 256, t_B = tmem + 384;
  bool ok = true;

  auto tile_of = [&](int it, int& qseg, int& qt, int& head) {
    const int t = it / G;
    head = hk * G + (it - t * G);
    if (t < n_raw_q) {
      qseg = kSegRaw;
      qt = rq_lo + t;
    } else if (t < n_raw_q + n_gist_q) {
      qseg = kSegGist;
      qt = gq_lo + (t - n_raw_q);
    } else {
      qseg = kSegSink;
      qt = sq_lo + (t - n_raw_q - n_gist_q);
    }
  };

  if (warp == 8) {
    // ------------------------------------------------------------ producer: K, V once; Q, dO, LSE, Delta per step
    if (lane == 0) {
      mbar_arrive_expect_tx(bar_kv, 2 * SM::kTile);
      const CUtensorMap* mk = kseg == kSegRaw ? &tm_k_raw : (kseg == kSegGist ? &tm_k_gist : &tm_k_sink);
      const CUtensorMap* mv = kseg == kSegRaw ? &tm_v_raw : (kseg == kSegGist ? &tm_v_gist : &tm_v_sink);
#pragma unroll
      for (int sl = 0; sl < D / 64; ++sl) {
        tma_load_4d(sK + sl * SM::kSlab, mk, bar_kv, sl * 64, hk, key_a, b);
        tma_load_4d(sV + sl * SM::kSlab, mv, bar_kv, sl * 64, hk, key_a, b);
      }
    }
    for (int it = 0; it < n_iter; ++it) {
      const int st = it & 1;
      int qseg, qt, head;
      tile_of(it, qseg, qt, head);
      if (it >= 2) ok = mbar_wait_warp(bar_empty[st], ((it >> 1) - 1) & 1);
      if (!ok) break;
      const int q_seg_len = seg_len(g, qseg), q_seg_base = seg_base(g, qseg);
      float* ls = stats + st * 2 * KV_BN;
      const long long row_base = ((long long)b * Hq + head) * g.N + q_seg_base;
#pragma unroll
      for (int i = 0; i < KV_BN / 32; ++i) {
        const int c = lane + 32 * i, row = qt * KV_BN + c;
        const bool valid = row < q_seg_len;
        // rows past the segment get LSE = +inf, so their P is exactly zero
        ls[c] = valid ? lse[row_base + row] * kLog2e : INFINITY;
        ls[KV_BN + c] = valid ? delta[row_base + row] : 0.f;
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_expect_tx(bar_full[st], 2 * SM::kTile);
        const CUtensorMap* mq = qseg == kSegRaw ? &tm_q_raw : (qseg == kSegGist ? &tm_q_gist : &tm_q_sink);
        const CUtensorMap* md = qseg == kSegRaw ? &tm_do_raw : (qseg == kSegGist ? &tm_do_gist : &tm_do_sink);
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) {
          tma_load_4d(sQ[st] + sl * SM::kSlab, mq, bar_full[st], sl * 64, head, qt * KV_BN, b);
          tma_load_4d(sDO[st] + sl * SM::kSlab, md, bar_full[st], sl * 64, head, qt * KV_BN, b);
        }
      }
      __syncwarp();
    }
    if (!ok) atomicExch(&g_bwd_timeout, 1u);
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(KV_BM, KV_BN, false, false);
      constexpr uint32_t idesc_acc = make_idesc_bf16(KV_BM, D, false, true);
      // A operand of the accumulating MMAs: bf16 pairs in TMEM; query columns [0,64) are packed at
      // columns [0,32) of the buffer, query columns [64,128) at columns [64,96)
      auto a_col = [](int kk) { return (kk / 4) * 64 + (kk % 4) * 8; };
      ok = mbar_wait(bar_kv, 0);
      for (int it = 0; it < n_iter && ok; ++it) {
        const int st = it & 1;
        ok = mbar_wait(bar_full[st], (it >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk / 4) * SM::kSlab + (kk % 4) * 32;
          umma_ss(t_A, make_smem_desc(sK + off, 16, 1024), make_smem_desc(sQ[st] + off, 16, 1024), idesc_s, kk > 0);
        }
        umma_commit(bar_S);
        if (it > 0) {
          const int ps = (it - 1) & 1;
          ok = mbar_wait(bar_dS, (it - 1) & 1);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < KV_BN / 16; ++kk)
            umma_ts(t_dK, t_B + a_col(kk), make_smem_desc(sQ[ps] + kk * 2048, SM::kSlab, 1024), idesc_acc,
                    (it > 1 || kk > 0) ? 1u : 0u);
          umma_commit(bar_empty[ps]);
        }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk / 4) * SM::kSlab + (kk % 4) * 32;
          umma_ss(t_B, make_smem_desc(sV + off, 16, 1024), make_smem_desc(sDO[st] + off, 16, 1024), idesc_s, kk > 0);
        }
        umma_commit(bar_dP);
        ok = mbar_wait(bar_P, it & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < KV_BN / 16; ++kk)
          umma_ts(t_dV, t_A + a_col(kk), make_smem_desc(sDO[st] + kk * 2048, SM::kSlab, 1024), idesc_acc,
                  (it > 0 || kk > 0) ? 1u : 0u);
      }
      if (ok && n_iter > 0) {
        const int ps = (n_iter - 1) & 1;
        ok = mbar_wait(bar_dS, (n_iter - 1) & 1);
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < KV_BN / 16; ++kk)
            umma_ts(t_dK, t_B + a_col(kk), make_smem_desc(sQ[ps] + kk * 2048, SM::kSlab, 1024), idesc_acc,
                    (n_iter > 1 || kk > 0) ? 1u : 0u);
          umma_commit(bar_final);
        }
      }
      if (!ok) atomicExch(&g_bwd_timeout, 1u);
    }
  } else {
    // ------------------------------------------------------------ compute: thread = key (TMEM lane), 64 query columns
    const int qd = warp & 3, hf = warp >> 2;
    const int key = key_a + qd * 32 + lane;
    const bool key_valid = key <= key_b;
    const uint32_t lane_base = static_cast<uint32_t>(qd * 32) << 16;
    const float scale_log2 = scale * kLog2e;
    int my_lo_r, my_hi_r, my_lo_g, my_hi_g, my_lo_s, my_hi_s;  // queries that see this key, per query segment
    key_q_interval3(g, kseg, key, key_valid, kSegRaw, my_lo_r, my_hi_r);
    key_q_interval3(g, kseg, key, key_valid, kSegGist, my_lo_g, my_hi_g);
    key_q_interval3(g, kseg, key, key_valid, kSegSink, my_lo_s, my_hi_s);

    for (int it = 0; it < n_iter && ok; ++it) {
      const int st = it & 1;
      int qseg, qt, head;
      tile_of(it, qseg, qt, head);
      const int q0 = qt * KV_BN, q_seg_len = seg_len(g, qseg);
      const int qb = min(q0 + KV_BN - 1, q_seg_len - 1);
      // full: every (query, key) pair of the tile is visible -> no mask arithmetic
      const int t_lo = qseg == kSegRaw ? raw_t_lo : (qseg == kSegGist ? gist_t_lo : sink_t_lo);
      const int t_hi = qseg == kSegRaw ? raw_t_hi : (qseg == kSegGist ? gist_t_hi : sink_t_hi);
      const bool full = key_tile_whole && q0 >= t_lo && qb <= t_hi;
      const int lo = (qseg == kSegRaw ? my_lo_r : (qseg == kSegGist ? my_lo_g : my_lo_s)) - q0 - 64 * hf;
      const int hi = (qseg == kSegRaw ? my_hi_r : (qseg == kSegGist ? my_hi_g : my_hi_s)) - q0 - 64 * hf;
      const float* ls = stats + st * 2 * KV_BN + 64 * hf;
      const float* dl = ls + KV_BN;
      ok = mbar_wait_warp(bar_full[st], (it >> 1) & 1) && mbar_wait_warp(bar_S, it & 1);
      if (!ok) break;
      tc_fence_after();
      float p[64];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld(t_A + lane_base + 64 * hf + 32 * c, v);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 l4 = *reinterpret_cast<const float4*>(ls + 32 * c + i);
          const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float x = fmaf(__uint_as_float(v[i + e]), scale_log2, -lv[e]);
            if (!full) {
              const int col = 32 * c + i + e;
              x = (col >= lo && col <= hi) ? x : -INFINITY;
            }
            p[32 * c + i + e] = ex2(x);
          }
          pk[i / 2] = pack_bf16(p[32 * c + i], p[32 * c + i + 1]);
          pk[i / 2 + 1] = pack_bf16(p[32 * c + i + 2], p[32 * c + i + 3]);
        }
        tmem_st(t_A + lane_base + 64 * hf + 16 * c, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_P);
      ok = mbar_wait_warp(bar_dP, it & 1);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld(t_B + lane_base + 64 * hf + 32 * c, v);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
          const float4 d4 = *reinterpret_cast<const float4*>(dl + 32 * c + i);
          const float dv4[4] = {d4.x, d4.y, d4.z, d4.w};
          float ds[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) ds[e] = p[32 * c + i + e] * (__uint_as_float(v[i + e]) - dv4[e]);
          pk[i / 2] = pack_bf16(ds[0], ds[1]);
          pk[i / 2 + 1] = pack_bf16(ds[2], ds[3]);
        }
        tmem_st(t_B + lane_base + 64 * hf + 16 * c, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_dS);
    }
    if (ok && n_iter > 0) ok = mbar_wait_warp(bar_final, 0);
    if (ok) {
      tc_fence_after();
      const long long tok = (long long)b * g.N + key_seg_base + key;
      // D = 128: this warp stores columns [64 hf, 64 hf + 64) of dK and of dV; D = 64: hf picks dK or dV
      constexpr int kChunks = 2;
#pragma unroll
      for (int which = 0; which < (D == 128 ? 2 : 1); ++which) {
        const bool is_dk = D == 128 ? which == 0 : hf == 0;
        const int col0 = D == 128 ? 64 * hf : 0;
        const uint32_t tsrc = (is_dk ? t_dK : t_dV) + lane_base + col0;
        __nv_bfloat16* dst = (is_dk ? dk : dv) + (tok * Hkv + hk) * D + col0;
        const float mul = is_dk ? scale : 1.f;
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          uint32_t v[32];
          if (n_iter > 0) {
            tmem_ld(tsrc + 32 * c, v);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0u;
          }
          if (key_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 pk;
              pk.x = pack_bf16(__uint_as_float(v[i]) * mul, __uint_as_float(v[i + 1]) * mul);
              pk.y = pack_bf16(__uint_as_float(v[i + 2]) * mul, __uint_as_float(v[i + 3]) * mul);
              pk.z = pack_bf16(__uint_as_float(v[i + 4]) * mul, __uint_as_float(v[i + 5]) * mul);
              pk.w = pack_bf16(__uint_as_float(v[i + 6]) * mul, __uint_as_float(v[i + 7]) * mul);
              *reinterpret_cast<uint4*>(dst + 32 * c + i) = pk;
            }
          }
        }
      }
    } else {
      atomicExch(&g_bwd_timeout, 1u);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    __syncwarp();
    tmem_dealloc(tmem, 512);
  }
}

// ------------------------------------------------------------------------------------------------
// dQ kernel
constexpr int DQ_BM = 128;  // query rows per block
constexpr int DQ_BN = 64;   // keys per step
constexpr int kDqThreads = 192;

template <int D>
struct DqSmem {
  static constexpr int kQSlab = DQ_BM * 128, kQTile = kQSlab * (D / 64);
  static constexpr int kKSlab = DQ_BN * 128, kKTile = kKSlab * (D / 64);
  static constexpr int kBytes = 2 * kQTile + 2 * kKTile + 1024 + 128;
};

template <int D>
__global__ void __launch_bounds__(kDqThreads, 2)
attn_bwd_dq_sm100_kernel(const __grid_constant__ CUtensorMap tm_q_sink, const __grid_constant__ CUtensorMap tm_q_raw,
                         const __grid_constant__ CUtensorMap tm_q_gist, const __grid_constant__ CUtensorMap tm_do_sink,
                         const __grid_constant__ CUtensorMap tm_do_raw, const __grid_constant__ CUtensorMap tm_do_gist,
                         const __grid_constant__ CUtensorMap tm_k_sink, const __grid_constant__ CUtensorMap tm_k_raw,
                         const __grid_constant__ CUtensorMap tm_k_gist, const __grid_constant__ CUtensorMap tm_v_sink,
                         const __grid_constant__ CUtensorMap tm_v_raw, const __grid_constant__ CUtensorMap tm_v_gist,
                         Geom g, int Hq, int Hkv, float scale, const float* __restrict__ lse,
                         const float* __restrict__ delta, __nv_bfloat16* __restrict__ dq, int n_sink_qt, int n_raw_qt) {
  using SM = DqSmem<D>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* gen = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t sQ = base, sDO = base + SM::kQTile, sK = base + 2 * SM::kQTile, sV = sK + SM::kKTile;
  const uint32_t bars = sV + SM::kKTile;
  const uint32_t bar_q = bars, bar_k = bars + 8, bar_v = bars + 16, bar_s = bars + 24, bar_p = bars + 32,
                 bar_pv = bars + 40, tmem_slot = bars + 48;
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(gen + 2 * SM::kQTile + 2 * SM::kKTile + 48);

  const int warp = threadIdx.x >> 5;
  const int h = blockIdx.y, b = blockIdx.z, hk = h / (Hq / Hkv);
  // heaviest tiles first: gist query tiles from the end, then raw query tiles from the end, sink tiles last
  const int qt_lin = gridDim.x - 1 - blockIdx.x;
  const int qseg = qt_lin < n_sink_qt ? kSegSink : (qt_lin < n_sink_qt + n_raw_qt ? kSegRaw : kSegGist);
  const int qt = qt_lin - (qseg == kSegSink ? 0 : (qseg == kSegRaw ? n_sink_qt : n_sink_qt + n_raw_qt));
  const int q_len = seg_len(g, qseg);
  const int q_base = seg_base(g, qseg);
  const int row_a = qt * DQ_BM, row_b = min(row_a + DQ_BM - 1, q_len - 1);
  const RowIv iv_a = row_intervals(g, q_base + row_a), iv_b = row_intervals(g, q_base + row_b);
  // visible 64-key tiles: sink tiles [0, n_sink), raw tiles [raw_lo, raw_lo + n_raw), gist tiles [0, n_gist)
  const int n_sink = iv_b.hi_sink >= 0 ? iv_b.hi_sink / DQ_BN + 1 : 0;
  const int raw_lo = iv_a.lo_raw / DQ_BN, n_raw = iv_b.hi_raw >= iv_a.lo_raw ? iv_b.hi_raw / DQ_BN - raw_lo + 1 : 0;
  const int n_gist = iv_b.hi_gist >= 0 ? iv_b.hi_gist / DQ_BN + 1 : 0;
  const int nt = n_sink + n_raw + n_gist;
  // step j: its key segment and 64-key tile
  auto key_tile = [&](int j, int& sg, int& idx) {
    if (j < n_raw) {
      sg = kSegRaw;
      idx = raw_lo + j;
    } else if (j < n_raw + n_gist) {
      sg = kSegGist;
      idx = j - n_raw;
    } else {
      sg = kSegSink;
      idx = j - n_raw - n_gist;
    }
  };

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_k, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 128);
    mbar_init(bar_pv, 1);
    mbar_fence_init();
  }
  if (warp == 5) tmem_alloc(tmem_slot, 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t t_S = tmem, t_dP = tmem + 64, t_dQ = tmem + 128;
  bool ok = true;

  if (warp == 4) {
    if (elect_one()) {
      mbar_arrive_expect_tx(bar_q, 2 * SM::kQTile);
      const CUtensorMap* mq = qseg == kSegRaw ? &tm_q_raw : (qseg == kSegGist ? &tm_q_gist : &tm_q_sink);
      const CUtensorMap* md = qseg == kSegRaw ? &tm_do_raw : (qseg == kSegGist ? &tm_do_gist : &tm_do_sink);
#pragma unroll
      for (int sl = 0; sl < D / 64; ++sl) {
        tma_load_4d(sQ + sl * SM::kQSlab, mq, bar_q, sl * 64, h, row_a, b);
        tma_load_4d(sDO + sl * SM::kQSlab, md, bar_q, sl * 64, h, row_a, b);
      }
      for (int j = 0; j < nt && ok; ++j) {
        int sg, idx;
        key_tile(j, sg, idx);
        const CUtensorMap* mk = sg == kSegRaw ? &tm_k_raw : (sg == kSegGist ? &tm_k_gist : &tm_k_sink);
        const CUtensorMap* mv = sg == kSegRaw ? &tm_v_raw : (sg == kSegGist ? &tm_v_gist : &tm_v_sink);
        if (j > 0) ok = mbar_wait(bar_s, (j - 1) & 1);  // dP(j-1) done: V buffer free
        if (!ok) break;
        mbar_arrive_expect_tx(bar_v, SM::kKTile);
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) tma_load_4d(sV + sl * SM::kKSlab, mv, bar_v, sl * 64, hk, idx * DQ_BN, b);
        if (j > 0) ok = mbar_wait(bar_pv, (j - 1) & 1);  // dQ MMA (j-1) done: K buffer free
        if (!ok) break;
        mbar_arrive_expect_tx(bar_k, SM::kKTile);
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) tma_load_4d(sK + sl * SM::kKSlab, mk, bar_k, sl * 64, hk, idx * DQ_BN, b);
      }
      if (!ok) atomicExch(&g_bwd_timeout, 1u);
    }
  } else if (warp == 5) {
    if (elect_one()) {
      constexpr uint32_t idesc_s = make_idesc_bf16(DQ_BM, DQ_BN, false, false);
      constexpr uint32_t idesc_dq = make_idesc_bf16(DQ_BM, D, false, true);
      ok = mbar_wait(bar_q, 0);
      for (int j = 0; j < nt && ok; ++j) {
        ok = mbar_wait(bar_k, j & 1) && mbar_wait(bar_v, j & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t qoff = (kk / 4) * SM::kQSlab + (kk % 4) * 32, koff = (kk / 4) * SM::kKSlab + (kk % 4) * 32;
          umma_ss(t_S, make_smem_desc(sQ + qoff, 16, 1024), make_smem_desc(sK + koff, 16, 1024), idesc_s, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t qoff = (kk / 4) * SM::kQSlab + (kk % 4) * 32, koff = (kk / 4) * SM::kKSlab + (kk % 4) * 32;
          umma_ss(t_dP, make_smem_desc(sDO + qoff, 16, 1024), make_smem_desc(sV + koff, 16, 1024), idesc_s, kk > 0);
        }
        umma_commit(bar_s);
        ok = mbar_wait(bar_p, j & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < DQ_BN / 16; ++kk)
          umma_ts(t_dQ, t_S + kk * 8, make_smem_desc(sK + kk * 2048, SM::kKSlab, 1024), idesc_dq,
                  (j > 0 || kk > 0) ? 1u : 0u);
        umma_commit(bar_pv);
      }
      if (!ok) atomicExch(&g_bwd_timeout, 1u);
    }
  } else {
    const int r_in_tile = threadIdx.x;
    const int row = min(row_a + r_in_tile, row_b);
    const bool valid = row_a + r_in_tile <= row_b;
    const RowIv my = row_intervals(g, q_base + row);
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    const float scale_log2 = scale * kLog2e;
    const long long stat_idx = ((long long)b * Hq + h) * g.N + q_base + row;
    const float lse2 = lse[stat_idx] * kLog2e, dl = delta[stat_idx];
    for (int j = 0; j < nt && ok; ++j) {
      int sg, idx;
      key_tile(j, sg, idx);
      const int col0 = idx * DQ_BN;
      bool full;
      int lo, hi;
      if (sg == kSegRaw) {
        full = col0 >= iv_b.lo_raw && col0 + DQ_BN - 1 <= iv_a.hi_raw;
        lo = my.lo_raw - col0;
        hi = my.hi_raw - col0;
      } else if (sg == kSegGist) {
        full = col0 + DQ_BN - 1 <= iv_a.hi_gist;
        lo = 0;
        hi = my.hi_gist - col0;
      } else {
        full = col0 + DQ_BN - 1 <= iv_a.hi_sink;
        lo = 0;
        hi = my.hi_sink - col0;
      }
      ok = mbar_wait_warp(bar_s, j & 1);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < DQ_BN / 32; ++c) {
        uint32_t sv[32], dv_[32];
        tmem_ld(t_S + lane_base + 32 * c, sv);
        tmem_ld(t_dP + lane_base + 32 * c, dv_);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float x0 = fmaf(__uint_as_float(sv[i]), scale_log2, -lse2);
          float x1 = fmaf(__uint_as_float(sv[i + 1]), scale_log2, -lse2);
          if (!full) {
            const int col = 32 * c + i;
            x0 = (col >= lo && col <= hi) ? x0 : -INFINITY;
            x1 = (col + 1 >= lo && col + 1 <= hi) ? x1 : -INFINITY;
          }
          const float ds0 = ex2(x0) * (__uint_as_float(dv_[i]) - dl);
          const float ds1 = ex2(x1) * (__uint_as_float(dv_[i + 1]) - dl);
          pk[i / 2] = pack_bf16(ds0, ds1);
        }
        tmem_st(t_S + lane_base + 16 * c, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p);
    }
    if (ok) ok = mbar_wait_warp(bar_pv, (nt - 1) & 1);
    if (ok) {
      tc_fence_after();
      const long long tok = (long long)b * g.N + q_base + row_a + r_in_tile;
      __nv_bfloat16* drow = dq + (tok * Hq + h) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        tmem_ld(t_dQ + lane_base + 32 * c, v);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(v[i]) * scale, __uint_as_float(v[i + 1]) * scale);
            pk.y = pack_bf16(__uint_as_float(v[i + 2]) * scale, __uint_as_float(v[i + 3]) * scale);
            pk.z = pack_bf16(__uint_as_float(v[i + 4]) * scale, __uint_as_float(v[i + 5]) * scale);
            pk.w = pack_bf16(__uint_as_float(v[i + 6]) * scale, __uint_as_float(v[i + 7]) * scale);
            *reinterpret_cast<uint4*>(drow + 32 * c + i) = pk;
          }
        }
      }
    } else {
      atomicExch(&g_bwd_timeout, 1u);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    __syncwarp();
    tmem_dealloc(tmem, 256);
  }
}

// ------------------------------------------------------------------------------------------------
// Fused backward for head_dim 128: one kernel, five matrix products per (key tile, query tile) pair.
//
// A thread block owns a 128-key tile of one KV head (dK, dV in TMEM for its lifetime: no atomics,
// deterministic) and walks every 128-query tile of every query head of the group that sees it:
//   S^T = K Q^T, dP^T = V dO^T        (both operands in shared memory)          -> TMEM
//   P^T = exp2(S^T c - LSE)            bf16, written over S^T in TMEM
//   dV += P^T dO                       (P^T read from TMEM)
//   dS^T = P^T o (dP^T - Delta)        bf16, written to shared memory [key][query]
//   dK += dS^T Q                       (dS^T from shared memory, query-contiguous = K-major A)
//   dQ^T = K^T dS^T                    (K tile as MN-major A, dS^T as MN-major B) -> TMEM, over dP^T
// dQ^T (head_dim x queries, fp32) is then added into an fp32 dQ buffer in global memory by TMA
// reductions from small staging buffers, since several key tiles contribute to one query tile; a
// small kernel scales and rounds that buffer to bf16 afterwards.
// MMA issue order per step i:  dV(i), S(i+1), dQ(i), dK(i), dP(i+1)  so that the exponentials of
// step i+1 and the dQ read-out of step i run under matrix products.
// Warps: 0-7 compute (thread = key, 64 query columns each), 8-15 dQ read-out (two warps per TMEM lane
// quarter, 64 query columns each, so the dQ^T columns are free again after two TMEM loads), 16 TMA, 17 MMA.
constexpr int kFuThreads = 640;
constexpr int kFuTmaWarp = 16, kFuMmaWarp = 17;
constexpr int kFuRegsLaunch = 96, kFuRegsCompute = 128, kFuRegsReadout = 80, kFuRegsOther = 64;
static_assert(kFuThreads * kFuRegsLaunch <= 65536 && kFuThreads * (kFuRegsLaunch + 8) > 65536,
              "launch register count is stale");
static_assert(2 * kFuRegsCompute + 2 * kFuRegsReadout + kFuRegsOther <= 5 * kFuRegsLaunch,
              "register split exceeds the block's allocation");

// One 32-query chunk of P^T for one key: p = 2^(s * c - lse2[q]); kMasked: bit e of `bits` says query e sees the key.
template <bool kMasked>
__device__ __forceinline__ void fused_p_chunk(const uint32_t (&v)[32], const float* __restrict__ ls, float scale_log2,
                                              uint32_t bits, float* __restrict__ p, uint32_t (&pk)[16]) {
#pragma unroll
  for (int i = 0; i < 32; i += 4) {
    const float4 l4 = *reinterpret_cast<const float4*>(ls + i);
    const float lv[4] = {l4.x, l4.y, l4.z, l4.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float x = fmaf(__uint_as_float(v[i + e]), scale_log2, -lv[e]);
      if (kMasked) x = (bits >> (i + e)) & 1u ? x : -INFINITY;
      p[i + e] = ex2(x);
    }
    pk[i / 2] = pack_bf16(p[i], p[i + 1]);
    pk[i / 2 + 1] = pack_bf16(p[i + 2], p[i + 3]);
  }
}

struct FuSmem {
  static constexpr int kSlab = 128 * 128;    // [128 rows x 64 bf16]
  static constexpr int kTile = 2 * kSlab;    // [128 x 128] bf16
  static constexpr int kOffK = 0, kOffV = kTile, kOffQ = 2 * kTile /* 2 stages */, kOffDO = 4 * kTile, kOffDS = 5 * kTile;
  static constexpr int kOffStage = 6 * kTile;             // dQ staging: [8 warps][32 queries][32 floats]
  static constexpr int kOffStats = 7 * kTile;             // [stage][lse2 | delta][128] fp32
  static constexpr int kOffBars = kOffStats + 2 * 2 * 128 * 4;
  static constexpr int kUsed = kOffBars + 192;
  static constexpr int kBytes = 232448;  // all a block may have; the 1024-byte alignment slack comes out of it
};

// One launch unit of the fused backward: a batch of sequences of one geometry with its own tensor maps (one per
// segment) and output pointers.  A call on one problem is one unit with a (blocks, 1, batch) grid; a packed
// sample under cross-document masking is several units in ONE launch with a flat grid, and a block finds its
// unit from the units' first block indices.
struct alignas(64) BwdRun {
  CUtensorMap q[3], dout[3], k[3], v[3], dq[3];
  Geom g;
  const float* lse;
  const float* delta;
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
  int n_sink_kt, n_gist_kt, n_raw_kt;
  int plane;  // blocks per batch index
  // flat grid (several units in one launch): the sink / gist blocks of ALL units come first, then the raw blocks;
  // the unit's first block in each of the two ranges, and its blocks per batch index there
  int heavy_begin, raw_begin, heavy_plane, raw_plane;
  FastDiv heavy_plane_div, raw_plane_div;
  // A sink or gist key tile's walk over its query tiles is cut into n_chunks chunks of chunk_tiles tiles, one
  // block each; `partial` receives the fp32 dK / dV of the chunks of key tiles that have more than one
  // ([batch][KV head][heavy key tile][chunk][dK | dV][128 keys][128]).
  int n_chunks, chunk_tiles;
  float* partial;
  FastDiv heavy_div /* by n_chunks * heavy tiles */, tile_div /* by heavy tiles */, raw_div;
};
template <int kRuns>
struct BwdRuns {
  BwdRun run[kRuns];
  int n;
  int total_heavy;  // flat grid: blocks of the sink / gist range
};
constexpr int kMaxRunsPerLaunch = 12;  // 12 units are 24 KB of kernel parameters (the limit is 32 KB)
static_assert(sizeof(BwdRuns<kMaxRunsPerLaunch>) + 256 <= 32764, "the launch units must fit the kernel parameter space");

template <int kRuns>
__global__ void __launch_bounds__(kFuThreads, 1)
attn_bwd_fused_sm100_kernel(const __grid_constant__ BwdRuns<kRuns> P, int Hq, int Hkv, float scale, int interleaved,
                            FastDiv rdiv) {
  int ri = 0, bx, b;
  if constexpr (kRuns == 1) {
    bx = blockIdx.x, b = blockIdx.z;
  } else {
    const int c = blockIdx.x;
    if (c < P.total_heavy) {
      while (ri + 1 < P.n && c >= P.run[ri + 1].heavy_begin) ++ri;
      const int local = c - P.run[ri].heavy_begin;
      b = fdiv(P.run[ri].heavy_plane_div, local);
      bx = local - b * P.run[ri].heavy_plane;  // < heavy_plane: a sink / gist block of the unit
    } else {
      while (ri + 1 < P.n && c >= P.run[ri + 1].raw_begin) ++ri;
      const int local = c - P.run[ri].raw_begin;
      b = fdiv(P.run[ri].raw_plane_div, local);
      bx = P.run[ri].heavy_plane + (local - b * P.run[ri].raw_plane);
    }
  }
  const BwdRun& R = P.run[ri];
  const Geom g = R.g;
  const float* __restrict__ lse = R.lse;
  const float* __restrict__ delta = R.delta;
  __nv_bfloat16* __restrict__ dk = R.dk;
  __nv_bfloat16* __restrict__ dv = R.dv;
  const int n_sink_kt = R.n_sink_kt, n_gist_kt = R.n_gist_kt, n_raw_kt = R.n_raw_kt;
  using SM = FuSmem;
  constexpr int D = 128;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw_base = smem_u32(smem_dyn);
  const uint32_t base = (raw_base + 1023u) & ~1023u;
  if (base - raw_base + SM::kUsed > SM::kBytes) {  // cannot happen with a 1024-aligned window; never run past it
    if (threadIdx.x == 0) atomicExch(&g_bwd_timeout, 1u);
    return;
  }
  unsigned char* gen = smem_dyn + (base - raw_base);
  const uint32_t sK = base + SM::kOffK, sV = base + SM::kOffV, sDS = base + SM::kOffDS;
  const uint32_t sQ0 = base + SM::kOffQ /* stage st at + st * kTile */, sDO = base + SM::kOffDO;
  float* stats = reinterpret_cast<float*>(gen + SM::kOffStats);
  const uint32_t bars = base + SM::kOffBars;
  const uint32_t bar_kv = bars, bar_S = bars + 8, bar_dP = bars + 16, bar_P = bars + 24, bar_dS = bars + 32,
                 bar_dSfree = bars + 40, bar_dQ = bars + 48, bar_dQfree = bars + 56, bar_final = bars + 64;
  const uint32_t full_q0 = bars + 72, empty_q0 = bars + 88 /* + 8 * st */, full_do = bars + 104, empty_do = bars + 120;
  const uint32_t tmem_slot = bars + 136;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(gen + SM::kOffBars + 136);
  // number of Q tiles whose load the producer has issued so far (a scheduling hint for the dQ read-out, see there)
  volatile int* q_issued = reinterpret_cast<volatile int*>(gen + SM::kOffBars + 144);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Block order (the hardware starts blocks in the order of their index).  Sink and gist key tiles are seen by
  // every later query: they are the heaviest and come first, before any raw key tile.  Their walk over the query
  // tiles (which starts at the last query tile for every one of them) is cut into chunks of the same query tiles,
  // one block per (key tile, chunk), ordered KV head, chunk, key tile: the blocks that run side by side are the key
  // tiles of ONE KV head over ONE chunk of queries, they start together, take the same time and read the same
  // Q / dO / dQ tiles, which therefore come from DRAM once and from L2 for every other block.  (One block per
  // key tile over all its queries had blocks of very different lengths start whenever an SM fell free, each
  // sweeping the head's queries on its own: 7 times the algorithmic DRAM traffic.)  The raw key tiles of one KV
  // head are consecutive too; their windows of query tiles overlap.
  const int G = Hq / Hkv;
  const int n_heavy_kt = n_sink_kt + n_gist_kt;
  int hk, rank, chunk = 0;
  if (bx < n_heavy_kt * R.n_chunks * Hkv) {
    hk = fdiv(R.heavy_div, bx);
    const int rem = bx - hk * n_heavy_kt * R.n_chunks;
    chunk = fdiv(R.tile_div, rem);
    rank = rem - chunk * n_heavy_kt;
  } else {
    const int y = bx - n_heavy_kt * R.n_chunks * Hkv;
    hk = fdiv(R.raw_div, y);
    rank = n_heavy_kt + (y - hk * n_raw_kt);
  }
  const int kseg = rank < n_sink_kt ? kSegSink : (rank < n_sink_kt + n_gist_kt ? kSegGist : kSegRaw);
  const int kt = rank - (kseg == kSegSink ? 0 : (kseg == kSegGist ? n_sink_kt : n_sink_kt + n_gist_kt));
  const int key_seg_len = seg_len(g, kseg);
  const int key_a = kt * 128, key_b = min(key_a + 127, key_seg_len - 1);
  const bool key_tile_whole = key_a + 127 <= key_seg_len - 1;

  // query tiles that see this key tile, per query segment: [first tile, count], and the bounds inside
  // which a tile is "full" (seen by the last key from t_lo on, by the first key up to t_hi)
  int lo_a, hi_a, lo_b, hi_b;
  key_q_interval3(g, kseg, key_a, true, kSegRaw, lo_a, hi_a);
  key_q_interval3(g, kseg, key_b, true, kSegRaw, lo_b, hi_b);
  const int n_raw_q = hi_b >= lo_a ? hi_b / 128 - lo_a / 128 + 1 : 0, rq_lo = lo_a / 128, raw_t_lo = lo_b, raw_t_hi = hi_a;
  key_q_interval3(g, kseg, key_a, true, kSegGist, lo_a, hi_a);
  key_q_interval3(g, kseg, key_b, true, kSegGist, lo_b, hi_b);
  const int n_gist_q = hi_b >= lo_a ? hi_b / 128 - lo_a / 128 + 1 : 0, gq_lo = lo_a / 128, gist_t_lo = lo_b, gist_t_hi = hi_a;
  key_q_interval3(g, kseg, key_a, true, kSegSink, lo_a, hi_a);
  key_q_interval3(g, kseg, key_b, true, kSegSink, lo_b, hi_b);
  const int n_sink_q = hi_b >= lo_a ? hi_b / 128 - lo_a / 128 + 1 : 0, sq_lo = lo_a / 128, sink_t_lo = lo_b, sink_t_hi = hi_a;
  // this block's part of the walk: tiles [t_begin, t_end) of the order below (all of them for a raw key tile)
  const int n_tiles = n_raw_q + n_gist_q + n_sink_q;
  const bool heavy = kseg != kSegRaw;
  const int t_begin = heavy ? chunk * R.chunk_tiles : 0;
  const int t_end = heavy ? min(t_begin + R.chunk_tiles, n_tiles) : n_tiles;
  if (chunk > 0 && t_begin >= n_tiles) return;  // this key tile has no such chunk (whole block, before any barrier)
  const bool to_partial = heavy && n_tiles > R.chunk_tiles;  // several chunks: fp32 partial sums, reduced afterwards
  const int n_iter = (t_end - t_begin) * G;

  if (threadIdx.x == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_S, 1);
    mbar_init(bar_dP, 1);
    mbar_init(bar_P, 256);
    mbar_init(bar_dS, 256);
    mbar_init(bar_dSfree, 1);
    mbar_init(bar_dQ, 1);
    mbar_init(bar_dQfree, 256);
    mbar_init(bar_final, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(full_q0 + 8 * i, 1);
      mbar_init(empty_q0 + 8 * i, 1);
    }
    mbar_init(full_do, 1);
    mbar_init(empty_do, 1);
    *q_issued = 0;
    mbar_fence_init();
  }
  if (warp == kFuMmaWarp) tmem_alloc(tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t t_dK = tmem, t_dV = tmem + 128, t_S = tmem + 256, t_dP = tmem + 384;
  bool ok = true;

  // Step order.  Tiles: raw query tiles from the last one down, then gist query tiles, then sink query tiles.
  // A sink or gist key tile is seen up to the last tile of every segment, so the blocks of one KV head that start
  // together walk the same tiles: with the G heads of a tile back to back they stay in step until each runs out,
  // and share Q / dO / dQ lines in L2.  A raw key tile sees a window of query tiles that moves with the key tile:
  // its neighbour is one tile behind, i.e. G steps with the heads innermost but a single step with the tiles
  // innermost (head by head), which keeps the shared lines in L2 between the two uses.
  const bool tiles_inner = kseg == kSegRaw;
  struct StepIter {
    int t, hd;  // tile index in the order above, head of the group
  };
  auto advance = [&](StepIter& x) {  // no division: the walk is sequential for every role
    if (tiles_inner) {
      if (++x.t == n_tiles) x.t = 0, ++x.hd;
    } else {
      if (++x.hd == G) x.hd = 0, ++x.t;
    }
  };
  auto tile_of = [&](const StepIter& x, int& qseg, int& qt, int& head) {
    const int t = x.t;
    head = hk * G + x.hd;
    if (t < n_raw_q) {
      qseg = kSegRaw;
      qt = rq_lo + (n_raw_q - 1 - t);
    } else if (t < n_raw_q + n_gist_q) {
      qseg = kSegGist;
      qt = gq_lo + (n_gist_q - 1 - (t - n_raw_q));
    } else {
      qseg = kSegSink;
      qt = sq_lo + (n_sink_q - 1 - (t - n_raw_q - n_gist_q));
    }
  };

  if (warp >= 16) {
    reg_dealloc<kFuRegsOther>();
    if (warp == kFuTmaWarp) {
      // ---------------------------------------------------------- producer: K, V once; Q, dO, LSE, Delta per step
      // tile coordinate: its first unit (a raw tile of an interleaved tensor spans 128 / r gist units)
      auto first_unit = [&](int sg, int row0) { return interleaved && sg == kSegRaw ? fdiv(rdiv, row0) : row0; };
      if (lane == 0) {
        mbar_arrive_expect_tx(bar_kv, 2 * SM::kTile);
        const CUtensorMap* mk = &R.k[kseg];
        const CUtensorMap* mv = &R.v[kseg];
#pragma unroll
        for (int sl = 0; sl < 2; ++sl) {
          tma_load_5d(sK + sl * SM::kSlab, mk, bar_kv, sl * 64, hk, 0, first_unit(kseg, key_a), b);
          tma_load_5d(sV + sl * SM::kSlab, mv, bar_kv, sl * 64, hk, 0, first_unit(kseg, key_a), b);
        }
      }
      // LSE (in log2 units) and Delta of the step's 128 query rows, 4 rows per lane, fetched one step ahead
      float st_l[4], st_d[4];
      auto fetch_stats = [&](const StepIter& at) {
        int qseg, qt, head;
        tile_of(at, qseg, qt, head);
        const int q_seg_len = seg_len(g, qseg), q_seg_base = seg_base(g, qseg);
        const long long row_base = ((long long)b * Hq + head) * g.N + q_seg_base;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int row = qt * 128 + lane + 32 * i;
          const bool valid = row < q_seg_len;
          // rows past the segment get LSE = +inf, so their P is exactly zero
          st_l[i] = valid ? lse[row_base + row] * kLog2e : INFINITY;
          st_d[i] = valid ? delta[row_base + row] : 0.f;
        }
      };
      StepIter cur{t_begin, 0}, ahead{t_begin, 0};
      if (n_iter > 0) fetch_stats(ahead);
      for (int it = 0; it < n_iter; ++it, advance(cur)) {
        const int st = it & 1;
        int qseg, qt, head;
        tile_of(cur, qseg, qt, head);
        if (it >= 2) ok = mbar_wait_warp(empty_q0 + 8 * st, ((it >> 1) - 1) & 1);
        if (!ok) break;
        float* ls = stats + st * 256;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          ls[lane + 32 * i] = st_l[i];
          ls[128 + lane + 32 * i] = st_d[i];
        }
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_expect_tx(full_q0 + 8 * st, SM::kTile);
          const CUtensorMap* mq = &R.q[qseg];
#pragma unroll
          for (int sl = 0; sl < 2; ++sl)
            tma_load_5d(sQ0 + st * SM::kTile + sl * SM::kSlab, mq, full_q0 + 8 * st, sl * 64, head, 0,
                        first_unit(qseg, qt * 128), b);
          *q_issued = it + 1;
        }
        advance(ahead);
        if (it + 1 < n_iter) fetch_stats(ahead);
        if (it >= 1) ok = mbar_wait_warp(empty_do, (it - 1) & 1);  // one dO buffer: free once dV of the step before is done
        if (!ok) break;
        if (lane == 0) {
          mbar_arrive_expect_tx(full_do, SM::kTile);
          const CUtensorMap* md = &R.dout[qseg];
#pragma unroll
          for (int sl = 0; sl < 2; ++sl)
            tma_load_5d(sDO + sl * SM::kSlab, md, full_do, sl * 64, head, 0, first_unit(qseg, qt * 128), b);
        }
        __syncwarp();
      }
      if (!ok && lane == 0) atomicExch(&g_bwd_timeout, 1u);
    } else if (warp == kFuMmaWarp) {
      // ---------------------------------------------------------- MMA issuer
      if (lane == 0) {
        constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);   // K-major A and B
        constexpr uint32_t idesc_acc = make_idesc_bf16(128, 128, false, true);  // K-major A, MN-major B
        constexpr uint32_t idesc_dq = make_idesc_bf16(128, 128, true, true);    // MN-major A and B
        constexpr uint32_t kHi = smem_desc_hi(1024);
        constexpr uint32_t kStage = SM::kTile >> 4;  // stage st of Q / dO: + st * kStage on the low word
        const uint32_t k_lo = smem_desc_lo(sK, 16), v_lo = smem_desc_lo(sV, 16);
        const uint32_t kT_lo = smem_desc_lo(sK, SM::kSlab);    // K tile read as MN-major A (head_dim contiguous)
        const uint32_t ds_lo = smem_desc_lo(sDS, 16);          // dS^T as K-major A (queries contiguous)
        const uint32_t dsT_lo = smem_desc_lo(sDS, SM::kSlab);  // dS^T as MN-major B
        const uint32_t q_lo = smem_desc_lo(sQ0, 16), qT_lo = smem_desc_lo(sQ0, SM::kSlab);
        const uint32_t do_lo = smem_desc_lo(sDO, 16), doT_lo = smem_desc_lo(sDO, SM::kSlab);
        // K-major operands step 32 B per 16 elements inside a 64-element slab; MN-major ones 2048 B
        auto koff = [](int kk) { return (uint32_t)(((kk / 4) * SM::kSlab + (kk % 4) * 32) >> 4); };
        auto moff = [](int kk) { return (uint32_t)((kk * 2048) >> 4); };
        // bf16 pairs of P^T in TMEM: query columns [0,64) packed at [0,32), [64,128) at [64,96)
        auto a_col = [](int kk) { return (uint32_t)((kk / 4) * 64 + (kk % 4) * 8); };
        auto issue_S = [&](int st) {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ss(t_S, smem_desc_join(k_lo + koff(kk), kHi), smem_desc_join(q_lo + st * kStage + koff(kk), kHi),
                    idesc_s, kk > 0);
          umma_commit(bar_S);
        };
        auto issue_dP = [&]() {
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            umma_ss(t_dP, smem_desc_join(v_lo + koff(kk), kHi), smem_desc_join(do_lo + koff(kk), kHi), idesc_s, kk > 0);
          umma_commit(bar_dP);
        };
        ok = mbar_wait(bar_kv, 0);
        if (ok && n_iter > 0) {
          ok = mbar_wait(full_q0, 0);
          if (ok) {
            tc_fence_after();
            issue_S(0);
            ok = mbar_wait(full_do, 0);
          }
          if (ok) {
            tc_fence_after();
            issue_dP();
          }
        }
        for (int it = 0; it < n_iter && ok; ++it) {
          const int st = it & 1, ph = it & 1;
          const bool has_next = it + 1 < n_iter;
          ok = mbar_wait(bar_P, ph);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)  // dV += P^T dO
            umma_ts(t_dV, t_S + a_col(kk), smem_desc_join(doT_lo + moff(kk), kHi), idesc_acc,
                    (it > 0 || kk > 0) ? 1u : 0u);
          umma_commit(empty_do);
          if (has_next) {
            ok = mbar_wait(full_q0 + 8 * (st ^ 1), ((it + 1) >> 1) & 1);
            if (!ok) break;
            tc_fence_after();
            issue_S(st ^ 1);
          }
          ok = mbar_wait(bar_dS, ph);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)  // dQ^T = K^T dS^T  (contraction over the 128 keys)
            umma_ss(t_dP, smem_desc_join(kT_lo + moff(kk), kHi), smem_desc_join(dsT_lo + moff(kk), kHi), idesc_dq,
                    kk > 0);
          umma_commit(bar_dQ);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)  // dK += dS^T Q  (contraction over the 128 queries)
            umma_ss(t_dK, smem_desc_join(ds_lo + koff(kk), kHi), smem_desc_join(qT_lo + st * kStage + moff(kk), kHi),
                    idesc_acc, (it > 0 || kk > 0) ? 1u : 0u);
          umma_commit(empty_q0 + 8 * st);
          umma_commit(bar_dSfree);
          if (has_next) {
            ok = mbar_wait(bar_dQfree, ph) && mbar_wait(full_do, (it + 1) & 1);
            if (!ok) break;
            tc_fence_after();
            issue_dP();
          }
        }
        if (ok) umma_commit(bar_final);
        if (!ok) atomicExch(&g_bwd_timeout, 1u);
      }
    }
  } else if (warp >= 8) {
    // ------------------------------------------------------------ dQ read-out: lane = head_dim index
    // Each warp moves its 32 head_dim rows x 64 queries of dQ^T, 32 queries at a time, through its own
    // staging buffer ([32 queries][32 floats]) and has the TMA unit add them into the fp32 dQ tensor.
    reg_dealloc<kFuRegsReadout>();
    const int qd = warp & 3, half = (warp >> 2) & 1;
    const uint32_t lane_base = static_cast<uint32_t>(qd * 32) << 16;
    float* stage_gen = reinterpret_cast<float*>(gen + SM::kOffStage) + (warp - 8) * 1024 + lane;
    const uint32_t stage_sh = base + SM::kOffStage + (warp - 8) * 4096;
    StepIter cur{t_begin, 0};
    for (int it = 0; it < n_iter && ok; ++it, advance(cur)) {
      int qseg, qt, head;
      tile_of(cur, qseg, qt, head);
      const CUtensorMap* mdq = &R.dq[qseg];
      const int nq = seg_len(g, qseg) - qt * 128;  // rows of this tile inside the segment (may exceed 128)
      ok = mbar_wait_warp(bar_dQ, it & 1);
      if (!ok) break;
      tc_fence_after();
      // both halves of this warp's 64 query columns into registers, then the dQ^T columns are free again: the
      // MMA warp never waits for the staging buffer or for the TMA unit
      uint32_t v0[32], v1[32];
      const int col0 = 64 * half;
      tmem_ld32(t_dP + lane_base + col0, v0);
      tmem_ld32(t_dP + lane_base + col0 + 32, v1);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive_relaxed(bar_dQfree);
      auto stage_rows = [&](const uint32_t (&v)[32]) {  // the reduction issued before has finished reading the staging buffer
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int e = 0; e < 32; ++e) stage_gen[e * 32] = __uint_as_float(v[e]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
      };
      auto reduce_rows = [&](int c0) {
        if (lane == 0 && c0 < nq) {  // rows past the segment's end are clipped by the tensor map
          tma_reduce_add_4d(mdq, stage_sh, qd * 32, head, qt * 128 + c0, b);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      };
      stage_rows(v0);
      // The TMA unit takes its work in order, and a step's 16 reduce-adds keep it busy for about 1200 clocks.
      // The Q tile of step it + 2 can be loaded once dK of this step is done, a few hundred clocks from now, and
      // S of that step waits for it: let that load go first.  A hint only: bounded, and no error if it runs out.
      if (lane == 0 && it + 2 < n_iter)
        for (int spin = 0; spin < 4096 && *q_issued < it + 3; ++spin) __nanosleep(20);
      __syncwarp();
      reduce_rows(col0);
      stage_rows(v1);
      reduce_rows(col0 + 32);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (!ok && lane == 0) atomicExch(&g_bwd_timeout, 1u);
  } else {
    // ------------------------------------------------------------ compute: thread = key (TMEM lane), 64 query columns
    reg_alloc<kFuRegsCompute>();
    const int qd = warp & 3, hf = warp >> 2;
    const int krow = qd * 32 + lane;
    const int key = key_a + krow;
    const bool key_valid = key <= key_b;
    const uint32_t lane_base = static_cast<uint32_t>(qd * 32) << 16;
    const float scale_log2 = scale * kLog2e;
    int my_lo_r, my_hi_r, my_lo_g, my_hi_g, my_lo_s, my_hi_s;  // queries that see this key, per query segment
    key_q_interval3(g, kseg, key, key_valid, kSegRaw, my_lo_r, my_hi_r);
    key_q_interval3(g, kseg, key, key_valid, kSegGist, my_lo_g, my_hi_g);
    key_q_interval3(g, kseg, key, key_valid, kSegSink, my_lo_s, my_hi_s);
    // this thread's row of the dS^T tile in shared memory: slab hf, row krow, 16-byte chunks swizzled by row
    unsigned char* ds_row = gen + SM::kOffDS + hf * SM::kSlab + krow * 128;
    const int swz = krow & 7;

    StepIter cur{t_begin, 0};
    for (int it = 0; it < n_iter && ok; ++it, advance(cur)) {
      const int st = it & 1;
      int qseg, qt, head;
      tile_of(cur, qseg, qt, head);
      const int q0 = qt * 128, q_seg_len = seg_len(g, qseg);
      const int qb = min(q0 + 127, q_seg_len - 1);
      // full: every (query, key) pair of the tile is visible -> no mask arithmetic
      const int t_lo = qseg == kSegRaw ? raw_t_lo : (qseg == kSegGist ? gist_t_lo : sink_t_lo);
      const int t_hi = qseg == kSegRaw ? raw_t_hi : (qseg == kSegGist ? gist_t_hi : sink_t_hi);
      const bool full = key_tile_whole && q0 >= t_lo && qb <= t_hi;
      const int lo = (qseg == kSegRaw ? my_lo_r : (qseg == kSegGist ? my_lo_g : my_lo_s)) - q0 - 64 * hf;
      const int hi = (qseg == kSegRaw ? my_hi_r : (qseg == kSegGist ? my_hi_g : my_hi_s)) - q0 - 64 * hf;
      const float* ls = stats + st * 256 + 64 * hf;
      const float* dl = ls + 128;
      ok = mbar_wait_warp(full_q0 + 8 * st, (it >> 1) & 1) && mbar_wait_warp(bar_S, it & 1);
      if (!ok) break;
      tc_fence_after();
      float p[64];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(t_S + lane_base + 64 * hf + 32 * c, v);
        tmem_wait_ld();
        uint32_t pk[16];
        if (full) {
          fused_p_chunk<false>(v, ls + 32 * c, scale_log2, 0u, p + 32 * c, pk);
        } else {
          const int a = max(lo - 32 * c, 0), bb = min(hi - 32 * c, 31);
          const uint32_t bits = a > bb ? 0u : ((0xffffffffu >> (31 - bb)) & (0xffffffffu << a));
          fused_p_chunk<true>(v, ls + 32 * c, scale_log2, bits, p + 32 * c, pk);
        }
        tmem_st(t_S + lane_base + 64 * hf + 16 * c, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_P);
      ok = mbar_wait_warp(bar_dP, it & 1);
      if (ok && it > 0) ok = mbar_wait_warp(bar_dSfree, (it - 1) & 1);  // the previous dS^T has been consumed
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(t_dP + lane_base + 64 * hf + 32 * c, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; i += 8) {  // 8 queries = one 16-byte chunk of this key's dS^T row
          const float4 d0 = *reinterpret_cast<const float4*>(dl + 32 * c + i);
          const float4 d1 = *reinterpret_cast<const float4*>(dl + 32 * c + i + 4);
          const float* pp = p + 32 * c + i;
          uint4 w;
          w.x = pack_bf16(pp[0] * (__uint_as_float(v[i]) - d0.x), pp[1] * (__uint_as_float(v[i + 1]) - d0.y));
          w.y = pack_bf16(pp[2] * (__uint_as_float(v[i + 2]) - d0.z), pp[3] * (__uint_as_float(v[i + 3]) - d0.w));
          w.z = pack_bf16(pp[4] * (__uint_as_float(v[i + 4]) - d1.x), pp[5] * (__uint_as_float(v[i + 5]) - d1.y));
          w.w = pack_bf16(pp[6] * (__uint_as_float(v[i + 6]) - d1.z), pp[7] * (__uint_as_float(v[i + 7]) - d1.w));
          const int chunk = 4 * c + i / 8;
          *reinterpret_cast<uint4*>(ds_row + ((chunk ^ swz) << 4)) = w;
        }
      }
      tc_fence_before();  // the dP^T columns may be overwritten (by dQ^T) once every thread has arrived
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // dS^T visible to the tensor core's reads
      mbar_arrive(bar_dS);
    }
    if (ok && n_iter > 0) ok = mbar_wait_warp(bar_final, 0);
    if (ok) {
      tc_fence_after();
      const long long tok = (long long)b * g.N + seg_row_to_token(g, interleaved != 0, kseg, key_valid ? key : key_a);
      // where this key's row of the chunk's fp32 partial sums goes when the key tile has several chunks
      float* part_row = R.partial + (((((long long)b * Hkv + hk) * n_heavy_kt + rank) * R.n_chunks + chunk) * 2 * 128 + krow) * 128 + 64 * hf;
      // this warp stores columns [64 hf, 64 hf + 64) of dK and of dV
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        const bool is_dk = which == 0;
        const uint32_t tsrc = (is_dk ? t_dK : t_dV) + lane_base + 64 * hf;
        __nv_bfloat16* dst = (is_dk ? dk : dv) + (tok * Hkv + hk) * D + 64 * hf;
        const float mul = is_dk ? scale : 1.f;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t v[32];
          if (n_iter > 0) {
            tmem_ld32(tsrc + 32 * c, v);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0u;
          }
          if (to_partial) {
            if (key_valid) {
              float4* pd = reinterpret_cast<float4*>(part_row + which * 128 * 128 + 32 * c);
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                pd[i / 4] = make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]), __uint_as_float(v[i + 2]),
                                        __uint_as_float(v[i + 3]));
            }
          } else if (key_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 pk;
              pk.x = pack_bf16(__uint_as_float(v[i]) * mul, __uint_as_float(v[i + 1]) * mul);
              pk.y = pack_bf16(__uint_as_float(v[i + 2]) * mul, __uint_as_float(v[i + 3]) * mul);
              pk.z = pack_bf16(__uint_as_float(v[i + 4]) * mul, __uint_as_float(v[i + 5]) * mul);
              pk.w = pack_bf16(__uint_as_float(v[i + 6]) * mul, __uint_as_float(v[i + 7]) * mul);
              *reinterpret_cast<uint4*>(dst + 32 * c + i) = pk;
            }
          }
        }
      }
    } else {
      atomicExch(&g_bwd_timeout, 1u);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kFuMmaWarp) {
    __syncwarp();
    tmem_dealloc(tmem, 512);
  }
}

// Number of 128-query tiles that see a key tile [key_a, key_b] of segment kseg (all query segments).
__device__ __forceinline__ int count_q_tiles(const Geom& g, int kseg, int key_a, int key_b) {
  int n = 0;
#pragma unroll
  for (int qseg = 0; qseg < 3; ++qseg) {
    int lo_a, hi_a, lo_b, hi_b;
    key_q_interval3(g, kseg, key_a, true, qseg, lo_a, hi_a);
    key_q_interval3(g, kseg, key_b, true, qseg, lo_b, hi_b);
    n += hi_b >= lo_a ? hi_b / 128 - lo_a / 128 + 1 : 0;
  }
  return n;
}

// dK, dV of the sink and gist key tiles whose walk was cut into several chunks: the chunks' fp32 partial sums
// added in chunk order (the same bits on every run), scaled, rounded to bf16 and stored at the keys' rows.
// One block per (16 rows of a heavy key tile, KV head, batch index), a warp per key row.
__global__ void __launch_bounds__(128)
dkdv_reduce_kernel(Geom g, int interleaved, int Hkv, int n_sink_kt, int n_gist_kt, int n_chunks, int chunk_tiles,
                   const float* __restrict__ partial, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                   float scale) {
  const int rank = blockIdx.x >> 3, row0 = (blockIdx.x & 7) * 16, hk = blockIdx.y, b = blockIdx.z;
  const int n_heavy_kt = n_sink_kt + n_gist_kt;
  const int kseg = rank < n_sink_kt ? kSegSink : kSegGist;
  const int kt = rank - (kseg == kSegSink ? 0 : n_sink_kt);
  const int key_a = kt * 128, key_b = min(key_a + 127, seg_len(g, kseg) - 1);
  const int n_tiles = count_q_tiles(g, kseg, key_a, key_b);
  if (n_tiles <= chunk_tiles) return;  // a single chunk: the fused kernel stored dK, dV itself
  const int chunks = (n_tiles + chunk_tiles - 1) / chunk_tiles;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* base = partial + ((((long long)b * Hkv + hk) * n_heavy_kt + rank) * n_chunks) * 2 * 128 * 128;
  for (int krow = row0 + warp; krow < row0 + 16 && key_a + krow <= key_b; krow += 4) {
    const long long tok = (long long)b * g.N + seg_row_to_token(g, interleaved != 0, kseg, key_a + krow);
#pragma unroll
    for (int which = 0; which < 2; ++which) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int c = 0; c < chunks; ++c) {
        const float4 x = __ldcs(reinterpret_cast<const float4*>(base + ((long long)(c * 2 + which) * 128 + krow) * 128) + lane);
        acc.x += x.x, acc.y += x.y, acc.z += x.z, acc.w += x.w;
      }
      const float mul = which == 0 ? scale : 1.f;
      __nv_bfloat16* dst = (which == 0 ? dk : dv) + (tok * Hkv + hk) * 128 + lane * 4;
      *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(acc.x * mul, acc.y * mul), pack_bf16(acc.z * mul, acc.w * mul));
    }
  }
}

// dQ (bf16) = scale * dQ accumulated in fp32 (shifted order, head_dim 128).  One warp per token: Hq rows of
// 128 floats, 4 per lane; the bf16 row goes to the token's shifted or interleaved position.
template <int kRuns>
__global__ void __launch_bounds__(256)
dq_convert_kernel(const __grid_constant__ TokRuns<kRuns> P, int interleaved, int Hq, long long tokens,
                  const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, float scale) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long tk = warp; tk < tokens; tk += nwarps) {  // tk = packed token index, shifted order inside a sequence
    int ri = 0;
    if constexpr (kRuns > 1)
      while (ri + 1 < P.n && tk >= P.run[ri + 1].tok_begin) ++ri;
    const Geom g = P.run[ri].g;
    const long long local = tk - P.run[ri].tok_begin;
    const long long b = local / g.N;
    const int sigma = (int)(local - b * g.N);
    const long long out_tk = P.run[ri].tok_begin + b * g.N + (interleaved ? shift_perm(g, sigma) : sigma);
    const float4* s4 = reinterpret_cast<const float4*>(src + tk * Hq * 128) + lane;
    uint2* d2 = reinterpret_cast<uint2*>(dst + out_tk * Hq * 128) + lane;
    for (int h0 = 0; h0 < Hq; h0 += 4) {
      float4 a[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (h0 + u < Hq) a[u] = __ldcs(s4 + (h0 + u) * 32);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (h0 + u < Hq)
          d2[(h0 + u) * 32] = make_uint2(pack_bf16(a[u].x * scale, a[u].y * scale), pack_bf16(a[u].z * scale, a[u].w * scale));
    }
  }
}

}  // namespace

namespace {

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// The backward's scratch for `tokens` packed tokens: Delta (fp32, per run a [batch, Hq, N] block that starts at
// float Hq * first token), the bf16 copy of an fp32 dO, and for the fused backward the fp32 dQ accumulator.
struct BwdScratch {
  float* delta;
  __nv_bfloat16* do_bf16;
  float* dq32;
};
BwdScratch carve_scratch(void* workspace, long long tokens, int Hq, int D, bool f32, bool fused) {
  char* ws = static_cast<char*>(workspace);
  BwdScratch sc;
  sc.delta = reinterpret_cast<float*>(ws);
  ws += align256((size_t)tokens * Hq * sizeof(float));
  sc.do_bf16 = f32 ? reinterpret_cast<__nv_bfloat16*>(ws) : nullptr;
  if (f32) ws += align256((size_t)tokens * Hq * D * 2);
  sc.dq32 = fused ? reinterpret_cast<float*>(ws) : nullptr;
  return sc;
}

template <int kRuns>
int32_t launch_prep(const TokRuns<kRuns>& T, const unigist_problem& p, long long tokens, const void* d_o, const void* o,
                    const BwdScratch& sc, cudaStream_t st) {
  const bool f32 = (p.flags & UNIGIST_FLAG_DOUT_FP32) != 0;
  const int il = (p.flags & UNIGIST_FLAG_INTERLEAVED) ? 1 : 0;
  const int blocks = (int)((tokens + 7) / 8 < sm_count() * 16 ? (tokens + 7) / 8 : sm_count() * 16);
  {
    KernelScope ks("bwd_prep_kernel", st);
    if (f32)
      bwd_prep_kernel<true, kRuns><<<blocks, 256, 0, st>>>(T, il, p.num_q_heads, p.head_dim, tokens, d_o,
                                                           (const __nv_bfloat16*)o, sc.do_bf16, sc.dq32);
    else
      bwd_prep_kernel<false, kRuns><<<blocks, 256, 0, st>>>(T, il, p.num_q_heads, p.head_dim, tokens, d_o,
                                                            (const __nv_bfloat16*)o, nullptr, sc.dq32);
  }
  return check_launch("backward prep kernel");
}

template <int kRuns>
int32_t launch_convert(const TokRuns<kRuns>& T, const unigist_problem& p, long long tokens, const BwdScratch& sc, void* dq,
                       float scale, cudaStream_t st) {
  const int blocks = (int)((tokens + 7) / 8 < sm_count() * 16 ? (tokens + 7) / 8 : sm_count() * 16);
  {
    KernelScope ks("dq_convert_kernel", st);
    dq_convert_kernel<kRuns><<<blocks, 256, 0, st>>>(T, (p.flags & UNIGIST_FLAG_INTERLEAVED) ? 1 : 0, p.num_q_heads, tokens,
                                                     sc.dq32, (__nv_bfloat16*)dq, scale);
  }
  return check_launch("dQ convert kernel");
}

// How the walk of a sink or gist key tile over its query tiles is cut (head_dim 128).  Not at all while the rows
// one KV head's blocks sweep (Q, dO and the fp32 dQ of its G query heads: 1 KB per token and head) fit in three
// quarters of the L2: however the blocks start, what one has read is still there for the next.  Otherwise into at
// most four chunks of at least 16 query tiles, fewer where the chunks' fp32 partial sums would take more than
// half the room of the dQ accumulator.
// -> tiles per chunk, number of chunks of the longest walk (1 = no cutting, no partial sums).
void bwd_chunking(const Geom& g, int batch, int Hq, int Hkv, int* n_chunks, int* chunk_tiles) {
  const int n_heavy = (g.s + 127) / 128 + (g.n + 127) / 128;
  const int max_tiles = n_heavy + (g.T + 127) / 128;  // the first sink / gist key tile is seen by every query tile
  const size_t dq_bytes = (size_t)batch * g.N * Hq * 128 * sizeof(float);
  const size_t sweep_bytes = (size_t)g.N * (Hq / Hkv) * 1024;
  int C = sweep_bytes > l2_bytes() / 4 * 3 ? 4 : 1;
  while (C > 1 && ((max_tiles + C - 1) / C < 16 ||
                   (size_t)batch * Hkv * n_heavy * C * 2 * 128 * 128 * sizeof(float) > dq_bytes / 2))
    --C;
  *chunk_tiles = (max_tiles + C - 1) / C;
  *n_chunks = (max_tiles + *chunk_tiles - 1) / *chunk_tiles;
}

// Tensor maps and tile counts of one launch unit of the fused backward: `batch` sequences of geometry g whose
// first rows are the given pointers.  128-row tile maps per segment (sinks, raw, gists) that read shifted or
// interleaved tensors, and reduction maps over the fp32 dQ tensor (always shifted).
int32_t fill_bwd_run(BwdRun* R, const Geom& g, const unigist_problem& p, int batch, const void* q, const void* do_src,
                     const void* k, const void* v, float* dq32, const float* lse, const float* delta, void* dk, void* dv,
                     float* partial) {
  const int D = p.head_dim, Hq = p.num_q_heads, Hkv = p.num_kv_heads;
  const bool il = (p.flags & UNIGIST_FLAG_INTERLEAVED) != 0;
  for (int sg = 0; sg < 3; ++sg) {
    if (int32_t rc = encode_tile_map(&R->q[sg], q, D, Hq, batch, g.s, g.T, g.r, g.n, il, sg)) return rc;
    if (int32_t rc = encode_tile_map(&R->dout[sg], do_src, D, Hq, batch, g.s, g.T, g.r, g.n, il, sg)) return rc;
    if (int32_t rc = encode_tile_map(&R->k[sg], k, D, Hkv, batch, g.s, g.T, g.r, g.n, il, sg)) return rc;
    if (int32_t rc = encode_tile_map(&R->v[sg], v, D, Hkv, batch, g.s, g.T, g.r, g.n, il, sg)) return rc;
    const int rows = seg_len(g, sg) > 0 ? seg_len(g, sg) : 1;  // a tensor map cannot be empty
    if (int32_t rc = encode_segment_map_f32(&R->dq[sg], dq32, D, Hq, g.N, batch, seg_base(g, sg), rows, 32, 32)) return rc;
  }
  R->g = g;
  R->lse = lse;
  R->delta = delta;
  R->dk = static_cast<__nv_bfloat16*>(dk);
  R->dv = static_cast<__nv_bfloat16*>(dv);
  R->n_sink_kt = (g.s + 127) / 128;
  R->n_gist_kt = (g.n + 127) / 128;
  R->n_raw_kt = (g.T + 127) / 128;
  bwd_chunking(g, batch, Hq, Hkv, &R->n_chunks, &R->chunk_tiles);
  R->partial = partial;
  const int n_heavy = R->n_sink_kt + R->n_gist_kt;
  R->heavy_plane = n_heavy * R->n_chunks * Hkv;
  R->raw_plane = R->n_raw_kt * Hkv;
  R->plane = R->heavy_plane + R->raw_plane;
  R->heavy_begin = R->raw_begin = 0;
  R->heavy_plane_div = make_fastdiv(R->heavy_plane);
  R->raw_plane_div = make_fastdiv(R->raw_plane);
  R->heavy_div = make_fastdiv(n_heavy * R->n_chunks);
  R->tile_div = make_fastdiv(n_heavy);
  R->raw_div = make_fastdiv(R->n_raw_kt);
  return UNIGIST_OK;
}

template <int kRuns>
int32_t launch_fused(const BwdRuns<kRuns>& P, dim3 grid, const unigist_problem& p, float scale, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(attn_bwd_fused_sm100_kernel<kRuns>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       FuSmem::kBytes);
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  {
    KernelScope ks("attn_bwd_fused_sm100_kernel", st);
    attn_bwd_fused_sm100_kernel<kRuns><<<grid, kFuThreads, FuSmem::kBytes, st>>>(
        P, p.num_q_heads, p.num_kv_heads, scale, (p.flags & UNIGIST_FLAG_INTERLEAVED) ? 1 : 0, make_fastdiv(p.ratio));
  }
  return check_launch("tcgen05 fused backward kernel");
}

// Adds up the chunks' partial dK / dV of one launch unit (nothing to do where no key tile has several chunks).
int32_t launch_dkdv_reduce(const BwdRun& R, int batch, const unigist_problem& p, float scale, cudaStream_t st) {
  if (R.n_chunks <= 1) return UNIGIST_OK;
  {
    KernelScope ks("dkdv_reduce_kernel", st);
    dkdv_reduce_kernel<<<dim3((R.n_sink_kt + R.n_gist_kt) * 8, p.num_kv_heads, batch), 128, 0, st>>>(
        R.g, (p.flags & UNIGIST_FLAG_INTERLEAVED) ? 1 : 0, p.num_kv_heads, R.n_sink_kt, R.n_gist_kt, R.n_chunks,
        R.chunk_tiles, R.partial, R.dk, R.dv, scale);
  }
  return check_launch("dK/dV reduce kernel");
}

// The two-kernel backward (head_dim 64; head_dim 128 when dQ has to be the same bit for bit from run to run): a
// block of the first kernel owns a key tile (dK, dV), a block of the second a query tile (dQ, over 64-key tiles).
template <int D>
int32_t launch_two_kernels(const Geom& g, const unigist_problem& p, float scale, const void* q, const void* do_src,
                           const void* k, const void* v, const float* lse, const float* delta, void* dq, void* dk,
                           void* dv, cudaStream_t st) {
  const int Hq = p.num_q_heads, Hkv = p.num_kv_heads, B = p.batch;
  const int n_sink_t = (g.s + 127) / 128, n_raw_t = (g.T + 127) / 128, n_gist_t = (g.n + 127) / 128;
  // one map per segment (sinks, raw, gists; a tensor map cannot be empty) with 128-row boxes, and 64-row boxes
  // over K and V for the dQ kernel
  CUtensorMap mq[3], md[3], mk[3], mv[3], mk64[3], mv64[3];
  for (int sg = 0; sg < 3; ++sg) {
    const long long first = seg_base(g, sg), len = seg_len(g, sg) > 0 ? seg_len(g, sg) : 1;
    if (int32_t rc = encode_segment_map(&mq[sg], q, D, Hq, g.N, B, first, len, 128)) return rc;
    if (int32_t rc = encode_segment_map(&md[sg], do_src, D, Hq, g.N, B, first, len, 128)) return rc;
    if (int32_t rc = encode_segment_map(&mk[sg], k, D, Hkv, g.N, B, first, len, 128)) return rc;
    if (int32_t rc = encode_segment_map(&mv[sg], v, D, Hkv, g.N, B, first, len, 128)) return rc;
    if (int32_t rc = encode_segment_map(&mk64[sg], k, D, Hkv, g.N, B, first, len, DQ_BN)) return rc;
    if (int32_t rc = encode_segment_map(&mv64[sg], v, D, Hkv, g.N, B, first, len, DQ_BN)) return rc;
  }
  const int n_tiles = n_sink_t + n_raw_t + n_gist_t;
  cudaError_t e = cudaFuncSetAttribute(attn_bwd_dkdv_sm100_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       KvSmem<D>::kBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(attn_bwd_dq_sm100_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSmem<D>::kBytes);
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  {
    KernelScope ks("attn_bwd_dkdv_sm100_kernel", st);
    attn_bwd_dkdv_sm100_kernel<D><<<dim3(n_tiles, Hkv, B), kKvThreads, KvSmem<D>::kBytes, st>>>(
        mq[0], mq[1], mq[2], md[0], md[1], md[2], mk[0], mk[1], mk[2], mv[0], mv[1], mv[2], g, Hq, Hkv, scale, lse, delta,
        (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, n_sink_t, n_gist_t);
  }
  if (int32_t rc = check_launch("tcgen05 dK/dV kernel")) return rc;
  {
    KernelScope ks("attn_bwd_dq_sm100_kernel", st);
    attn_bwd_dq_sm100_kernel<D><<<dim3(n_tiles, Hq, B), kDqThreads, DqSmem<D>::kBytes, st>>>(
        mq[0], mq[1], mq[2], md[0], md[1], md[2], mk64[0], mk64[1], mk64[2], mv64[0], mv64[1], mv64[2], g, Hq, Hkv, scale,
        lse, delta, (__nv_bfloat16*)dq, n_sink_t, n_raw_t);
  }
  return check_launch("tcgen05 dQ kernel");
}

}  // namespace

size_t bwd_scratch_bytes(long long tokens, int Hq, int D, bool dout_fp32, bool fused) {
  size_t b = align256((size_t)tokens * Hq * sizeof(float));
  if (dout_fp32) b += align256((size_t)tokens * Hq * D * 2);
  if (fused) b += align256((size_t)tokens * Hq * D * sizeof(float));
  return b;
}

size_t bwd_partial_bytes(const Geom& g, int batch, int Hq, int Hkv, bool fused) {
  if (!fused) return 0;
  int C, tiles;
  bwd_chunking(g, batch, Hq, Hkv, &C, &tiles);
  if (C <= 1) return 0;
  const size_t n_heavy = (g.s + 127) / 128 + (g.n + 127) / 128;
  return align256((size_t)batch * Hkv * n_heavy * C * 2 * 128 * 128 * sizeof(float));
}

int32_t launch_bwd_sm100(const Geom& g, const unigist_problem& p, float scale, const void* q, const void* k,
                         const void* v, const void* o, const float* lse, const void* d_o, void* dq, void* dk,
                         void* dv, void* workspace, cudaStream_t st) {
  const int D = p.head_dim, Hq = p.num_q_heads, Hkv = p.num_kv_heads, B = p.batch;
  const bool f32 = (p.flags & UNIGIST_FLAG_DOUT_FP32) != 0;
  const long long tokens = (long long)B * g.N;
  // head_dim 64 takes the two-kernel path, and so does head_dim 128 when dQ must not depend on the order in which
  // blocks arrive
  const bool fused = bwd_is_fused(D, p.flags);
  const BwdScratch sc = carve_scratch(workspace, tokens, Hq, D, f32, fused);
  float* delta = sc.delta;
  const void* do_src = f32 ? static_cast<const void*>(sc.do_bf16) : d_o;
  TokRuns<1> T;
  T.n = 1;
  T.run[0].g = g;
  T.run[0].tok_begin = 0;
  T.run[0].delta = delta;
  if (int32_t rc = launch_prep(T, p, tokens, d_o, o, sc, st)) return rc;

  if (!fused)
    return D == 64 ? launch_two_kernels<64>(g, p, scale, q, do_src, k, v, lse, delta, dq, dk, dv, st)
                   : launch_two_kernels<128>(g, p, scale, q, do_src, k, v, lse, delta, dq, dk, dv, st);
  BwdRuns<1> P;
  P.n = 1;
  P.total_heavy = 0;  // not used with the (blocks, 1, batch) grid
  float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + bwd_scratch_bytes(tokens, Hq, D, f32, true));
  if (int32_t rc = fill_bwd_run(&P.run[0], g, p, B, q, do_src, k, v, sc.dq32, lse, delta, dk, dv, partial)) return rc;
  if (int32_t rc = launch_fused(P, dim3(P.run[0].plane, 1, B), p, scale, st)) return rc;
  if (int32_t rc = launch_dkdv_reduce(P.run[0], B, p, scale, st)) return rc;
  return launch_convert(T, p, tokens, sc, dq, scale, st);
}

// Backward over a packed sample (head_dim 128): every run of equal documents is a launch unit; up to twelve
// units share one launch of the prep, fused and convert kernels.
int32_t launch_bwd_sm100_runs(const SeqRun* runs, int n_runs, long long tokens, const unigist_problem& p, float scale,
                              const void* q, const void* k, const void* v, const void* o, const float* lse,
                              const void* d_o, void* dq, void* dk, void* dv, void* workspace, cudaStream_t st) {
  const int D = p.head_dim, Hq = p.num_q_heads, Hkv = p.num_kv_heads;
  const bool f32 = (p.flags & UNIGIST_FLAG_DOUT_FP32) != 0;
  const BwdScratch sc = carve_scratch(workspace, tokens, Hq, D, f32, true);
  const void* do_src = f32 ? static_cast<const void*>(sc.do_bf16) : d_o;
  const size_t rq = (size_t)Hq * D * 2, rk = (size_t)Hkv * D * 2;
  // the chunks' partial dK / dV: one slice per run, behind the scratch of the packed tokens
  std::vector<float*> partial_of(n_runs);
  {
    char* at = static_cast<char*>(workspace) + bwd_scratch_bytes(tokens, Hq, D, f32, true);
    for (int i = 0; i < n_runs; ++i) {
      partial_of[i] = reinterpret_cast<float*>(at);
      at += bwd_partial_bytes(runs[i].g, runs[i].batch, Hq, Hkv, true);
    }
  }
  for (int first = 0; first < n_runs; first += kMaxRunsPerLaunch) {
    const int n = n_runs - first < kMaxRunsPerLaunch ? n_runs - first : kMaxRunsPerLaunch;
    // the runs of one launch hold consecutive packed tokens [tok_lo, tok_hi)
    const long long tok_lo = runs[first].first_row;
    const long long tok_hi = runs[first + n - 1].first_row + (long long)runs[first + n - 1].g.N * runs[first + n - 1].batch;
    TokRuns<kMaxRunsPerLaunch> T;
    BwdRuns<kMaxRunsPerLaunch> P;
    T.n = P.n = n;
    // the per-token kernels scan the runs in token order; the fused kernel starts the longest run's blocks first
    int order[kMaxRunsPerLaunch];
    for (int i = 0; i < n; ++i) order[i] = i;
    std::stable_sort(order, order + n, [&](int a, int b) {
      return (long long)runs[first + a].g.N * runs[first + a].batch > (long long)runs[first + b].g.N * runs[first + b].batch;
    });
    long long ctas = 0;
    for (int i = 0; i < n; ++i) {
      const SeqRun& t = runs[first + i];
      T.run[i].g = t.g;
      T.run[i].tok_begin = t.first_row - tok_lo;
      T.run[i].delta = sc.delta + t.first_row * Hq;
      const SeqRun& r = runs[first + order[i]];
      if (int32_t rc = fill_bwd_run(&P.run[i], r.g, p, r.batch, (const char*)q + r.first_row * rq,
                                    (const char*)do_src + r.first_row * rq, (const char*)k + r.first_row * rk,
                                    (const char*)v + r.first_row * rk, sc.dq32 + r.first_row * Hq * D,
                                    lse + r.first_row * Hq, sc.delta + r.first_row * Hq, (char*)dk + r.first_row * rk,
                                    (char*)dv + r.first_row * rk, partial_of[first + order[i]]))
        return rc;
      ctas += (long long)P.run[i].plane * r.batch;
      if (ctas > 0x7fffffffLL) return fail(UNIGIST_ERR_SHAPE, "packed sample too large for one grid");
    }
    // block ranges: every unit's sink / gist blocks (the long ones) before any unit's raw blocks
    int at = 0;
    for (int i = 0; i < n; ++i) {
      P.run[i].heavy_begin = at;
      at += P.run[i].heavy_plane * runs[first + order[i]].batch;
    }
    P.total_heavy = at;
    for (int i = 0; i < n; ++i) {
      P.run[i].raw_begin = at;
      at += P.run[i].raw_plane * runs[first + order[i]].batch;
    }
    for (int i = n; i < kMaxRunsPerLaunch; ++i) T.run[i] = T.run[0], P.run[i] = P.run[0];  // never selected
    // the per-token kernels of this launch see the tensors from packed token tok_lo on
    BwdScratch part = sc;
    if (part.do_bf16) part.do_bf16 += tok_lo * Hq * D;
    part.dq32 += tok_lo * Hq * D;
    const size_t rdo = f32 ? 2 * rq : rq;
    if (int32_t rc = launch_prep(T, p, tok_hi - tok_lo, (const char*)d_o + tok_lo * rdo, (const char*)o + tok_lo * rq, part, st))
      return rc;
    if (int32_t rc = launch_fused(P, dim3((unsigned)ctas, 1, 1), p, scale, st)) return rc;
    for (int i = 0; i < n; ++i)
      if (int32_t rc = launch_dkdv_reduce(P.run[i], runs[first + order[i]].batch, p, scale, st)) return rc;
    if (int32_t rc = launch_convert(T, p, tok_hi - tok_lo, part, (char*)dq + tok_lo * rq, scale, st)) return rc;
  }
  return UNIGIST_OK;
}

int32_t bwd_sm100_take_timeout(bool* timed_out) {
  unsigned int flag = 0, zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&flag, g_bwd_timeout, sizeof(flag));
  if (e == cudaSuccess && flag) e = cudaMemcpyToSymbol(g_bwd_timeout, &zero, sizeof(zero));
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "reading the device status: %s", cudaGetErrorString(e));
  *timed_out = flag != 0;
  return UNIGIST_OK;
}

}  // namespace ug
