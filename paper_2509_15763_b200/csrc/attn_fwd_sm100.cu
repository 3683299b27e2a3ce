// Forward gist-masked attention on Blackwell tensor cores (tcgen05 + TMEM + TMA), no sinks.
//
// The SHIFTED sequence is [raw (T) | gists (n)].  A thread block owns one 128-row query tile of one
// segment and one query head.  From the closed-form row intervals it derives the list of 128-key
// tiles that hold a visible pair: the tile of the query rows' own segment that contains the
// diagonal comes first (every row sees itself there, so the running maximum is finite from the
// first tile on), then the rest; masked-out tiles are never loaded.  Per key tile:
//   TMA:      K, V tiles -> shared memory (128-byte swizzle), one tensor map per segment so a tile
//             never straddles segments and rows past a segment's end read as zero.
//   tcgen05:  S = Q K^T into TMEM (fp32);   O += P V with P (bf16) read from TMEM.
//   softmax:  128 threads, one query row each: row max, lazy rescale of O, exp2, row sum, P -> TMEM.
//             Only tiles classified "partial" evaluate the mask; "full" tiles skip it.
// Roles: warps 0-3 softmax / epilogue, warp 4 TMA producer, warp 5 MMA issuer and TMEM owner.
// Two thread blocks share an SM (256 TMEM columns each) so one block's MMAs overlap the other's softmax.
#include "sm100_ptx.cuh"
#include "ug_common.cuh"

namespace ug {
namespace {

using namespace sm100;

constexpr int BM = 128;  // query rows per tile
constexpr int BN = 128;  // keys per tile
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 256;
constexpr float kRescaleThreshold = 8.0f;  // log2 units: O is rescaled only when the max grows by > 2^8

__device__ unsigned int g_fwd_timeout = 0;

template <int D>
struct FwdSmem {
  static constexpr int kSlab = BM * 128;          // bytes of one [128 rows x 64 bf16] slab
  static constexpr int kTile = kSlab * (D / 64);  // bytes of one [128 x D] tile
  static constexpr int kBytes = 3 * kTile + 1024 /*align*/ + 128 /*barriers*/;
};

// Key tiles a query tile visits: `n_first` tiles of its own segment in descending order starting
// at `first_hi`, then `n_second` tiles of the other segment ascending from `second_lo`.
struct TileSeq {
  int n_first, first_hi, n_second, second_lo;
  bool first_is_raw;
  __device__ int count() const { return n_first + n_second; }
  __device__ void at(int j, bool& is_raw, int& idx) const {
    if (j < n_first) {
      is_raw = first_is_raw;
      idx = first_hi - j;
    } else {
      is_raw = !first_is_raw;
      idx = second_lo + (j - n_first);
    }
  }
};

__device__ TileSeq make_tile_seq(const RowIv& iv_a, const RowIv& iv_b, bool q_is_raw) {
  const int raw_lo = iv_a.lo_raw / BN, raw_hi = iv_b.hi_raw / BN;  // hi_raw >= lo_raw always
  const int n_raw = raw_hi - raw_lo + 1;
  const int n_gist = iv_b.hi_gist >= 0 ? iv_b.hi_gist / BN + 1 : 0;
  TileSeq s;
  s.first_is_raw = q_is_raw;
  if (q_is_raw) {
    s.n_first = n_raw;
    s.first_hi = raw_hi;
    s.n_second = n_gist;
    s.second_lo = 0;
  } else {
    s.n_first = n_gist;
    s.first_hi = n_gist - 1;
    s.n_second = n_raw;
    s.second_lo = raw_lo;
  }
  return s;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
attn_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q_raw, const __grid_constant__ CUtensorMap tm_q_gist,
                      const __grid_constant__ CUtensorMap tm_k_raw, const __grid_constant__ CUtensorMap tm_k_gist,
                      const __grid_constant__ CUtensorMap tm_v_raw, const __grid_constant__ CUtensorMap tm_v_gist,
                      Geom g, int Hq, int Hkv, float scale_log2, __nv_bfloat16* __restrict__ o,
                      float* __restrict__ lse, int n_raw_qt) {
  using SM = FwdSmem<D>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const uint32_t sQ = base, sK = base + SM::kTile, sV = base + 2 * SM::kTile;
  const uint32_t bars = base + 3 * SM::kTile;
  const uint32_t bar_q = bars, bar_k = bars + 8, bar_v = bars + 16, bar_s = bars + 24, bar_p = bars + 32,
                 bar_pv = bars + 40, tmem_slot = bars + 48;
  unsigned char* gen_base = smem_dyn + (base - smem_u32(smem_dyn));
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(gen_base + 3 * SM::kTile + 48);

  const int warp = threadIdx.x >> 5;
  const int h = blockIdx.y, b = blockIdx.z, hk = h / (Hq / Hkv);
  // heaviest tiles first: gist tiles from the end, then raw tiles from the end
  const int qt_lin = gridDim.x - 1 - blockIdx.x;
  const bool q_is_raw = qt_lin < n_raw_qt;
  const int qt = q_is_raw ? qt_lin : qt_lin - n_raw_qt;
  const int seg_len = q_is_raw ? g.T : g.n;
  const int seg_base = q_is_raw ? g.s : g.s + g.T;  // shifted position of the segment's row 0
  const int row_a = qt * BM, row_b = min(row_a + BM - 1, seg_len - 1);
  const RowIv iv_a = row_intervals(g, seg_base + row_a), iv_b = row_intervals(g, seg_base + row_b);
  const TileSeq seq = make_tile_seq(iv_a, iv_b, q_is_raw);
  const int nt = seq.count();

  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_k, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 128);
    mbar_init(bar_pv, 1);
    mbar_fence_init();
  }
  if (warp == 5) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t tmem_S = tmem, tmem_P = tmem, tmem_O = tmem + 128;
  bool ok = true;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      const CUtensorMap* mq = q_is_raw ? &tm_q_raw : &tm_q_gist;
      mbar_arrive_expect_tx(bar_q, SM::kTile);
#pragma unroll
      for (int sl = 0; sl < D / 64; ++sl) tma_load_4d(sQ + sl * SM::kSlab, mq, bar_q, sl * 64, h, row_a, b);
      for (int j = 0; j < nt && ok; ++j) {
        bool is_raw;
        int idx;
        seq.at(j, is_raw, idx);
        const CUtensorMap* mk = is_raw ? &tm_k_raw : &tm_k_gist;
        const CUtensorMap* mv = is_raw ? &tm_v_raw : &tm_v_gist;
        if (j > 0) ok = mbar_wait(bar_s, (j - 1) & 1);  // S(j-1) done: K buffer free
        if (!ok) break;
        mbar_arrive_expect_tx(bar_k, SM::kTile);
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) tma_load_4d(sK + sl * SM::kSlab, mk, bar_k, sl * 64, hk, idx * BN, b);
        if (j > 0) ok = mbar_wait(bar_pv, (j - 1) & 1);  // PV(j-1) done: V buffer free
        if (!ok) break;
        mbar_arrive_expect_tx(bar_v, SM::kTile);
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) tma_load_4d(sV + sl * SM::kSlab, mv, bar_v, sl * 64, hk, idx * BN, b);
      }
      if (!ok) atomicExch(&g_fwd_timeout, 1u);
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc_qk = make_idesc_bf16(BM, BN, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(BM, D, false, true);
      ok = mbar_wait(bar_q, 0);
      for (int j = 0; j < nt && ok; ++j) {
        ok = mbar_wait(bar_k, j & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk / 4) * SM::kSlab + (kk % 4) * 32;
          umma_ss(tmem_S, make_smem_desc(sQ + off, 16, 1024), make_smem_desc(sK + off, 16, 1024), idesc_qk,
                  kk > 0);
        }
        umma_commit(bar_s);
        ok = mbar_wait(bar_p, j & 1) && mbar_wait(bar_v, j & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
          // V tile is MN-major: 16 keys = 2048 B per k step, 64-column groups SM::kSlab apart
          umma_ts(tmem_O, tmem_P + kk * 8, make_smem_desc(sV + kk * 2048, SM::kSlab, 1024), idesc_pv,
                  (j > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(bar_pv);
      }
      if (!ok) atomicExch(&g_fwd_timeout, 1u);
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue (one row per thread)
    const int r_in_tile = threadIdx.x;  // 0..127
    const int row = min(row_a + r_in_tile, row_b);
    const RowIv my = row_intervals(g, seg_base + row);
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    float m_run = -INFINITY, l_run = 0.f;

    for (int j = 0; j < nt && ok; ++j) {
      bool is_raw;
      int idx;
      seq.at(j, is_raw, idx);
      const int col0 = idx * BN;
      bool full;
      int lo, hi;  // visible columns of this row, relative to the tile
      if (is_raw) {
        full = col0 >= iv_b.lo_raw && col0 + BN - 1 <= iv_a.hi_raw;
        lo = my.lo_raw - col0;
        hi = my.hi_raw - col0;
      } else {
        full = col0 + BN - 1 <= iv_a.hi_gist;
        lo = 0;
        hi = my.hi_gist - col0;
      }
      ok = mbar_wait_warp(bar_s, j & 1);
      if (!ok) break;
      tc_fence_after();

      // pass 1: row maximum of the raw scores
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        tmem_ld(tmem_S + lane_base + c * 32, v);
        tmem_wait_ld();
        if (full) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(v[i]));
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int col = c * 32 + i;
            const float x = (col >= lo && col <= hi) ? __uint_as_float(v[i]) : -INFINITY;
            mx = fmaxf(mx, x);
          }
        }
      }
      const float mx_s = mx * scale_log2;
      const bool need = mx_s > m_run + kRescaleThreshold;  // also true for the first visible tile
      if (__any_sync(0xffffffffu, need)) {
        const float m_new = need ? mx_s : m_run;
        const float f = need ? ex2(m_run - m_new) : 1.f;  // m_run = -inf gives 0
        l_run *= f;
        m_run = m_new;
        if (j > 0) {  // S(j) complete implies PV(j-1) complete: O is stable here
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t v[32];
            tmem_ld(tmem_O + lane_base + c * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * f);
            tmem_st(tmem_O + lane_base + c * 32, v);
          }
        }
      }
      // pass 2: p = 2^(s * scale_log2 - m), row sum, bf16 P into TMEM (over the first 64 columns of S)
#pragma unroll
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        tmem_ld(tmem_S + lane_base + c * 32, v);
        tmem_wait_ld();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float x0 = fmaf(__uint_as_float(v[i]), scale_log2, -m_run);
          float x1 = fmaf(__uint_as_float(v[i + 1]), scale_log2, -m_run);
          if (!full) {
            const int col = c * 32 + i;
            x0 = (col >= lo && col <= hi) ? x0 : -INFINITY;
            x1 = (col + 1 >= lo && col + 1 <= hi) ? x1 : -INFINITY;
          }
          const float p0 = ex2(x0), p1 = ex2(x1);
          l_run += p0 + p1;
          pk[i / 2] = pack_bf16(p0, p1);
        }
        tmem_st(tmem_P + lane_base + c * 16, pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar_p);
    }
    if (ok) ok = mbar_wait_warp(bar_pv, (nt - 1) & 1);
    if (ok) {
      tc_fence_after();
      const float inv_l = 1.f / l_run;
      const bool valid = row_a + r_in_tile <= row_b;
      const long long tok = (long long)b * g.N + seg_base + row_a + r_in_tile;
      __nv_bfloat16* orow = o + (tok * Hq + h) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t v[32];
        tmem_ld(tmem_O + lane_base + c * 32, v);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(v[i]) * inv_l, __uint_as_float(v[i + 1]) * inv_l);
            pk.y = pack_bf16(__uint_as_float(v[i + 2]) * inv_l, __uint_as_float(v[i + 3]) * inv_l);
            pk.z = pack_bf16(__uint_as_float(v[i + 4]) * inv_l, __uint_as_float(v[i + 5]) * inv_l);
            pk.w = pack_bf16(__uint_as_float(v[i + 6]) * inv_l, __uint_as_float(v[i + 7]) * inv_l);
            *reinterpret_cast<uint4*>(orow + c * 32 + i) = pk;
          }
        }
      }
      if (valid)
        lse[((long long)b * Hq + h) * g.N + seg_base + row_a + r_in_tile] =
            (m_run + log2f(l_run)) * 0.6931471805599453f;
    } else {
      atomicExch(&g_fwd_timeout, 1u);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

int32_t encode_segment_map(CUtensorMap* map, const void* base, int D, int H, long long N, int B,
                           long long seg_first_row, long long seg_rows, int box_rows) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return fail(UNIGIST_ERR_CUDA, "cuTensorMapEncodeTiled is not available: %s", cudaGetErrorString(e));
    encode = reinterpret_cast<EncodeFn>(fn);
  }
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)seg_rows, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2, (cuuint64_t)N * H * D * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  void* addr = const_cast<char*>(static_cast<const char*>(base)) + seg_first_row * H * D * 2;
  CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, addr, dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(UNIGIST_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return UNIGIST_OK;
}

int32_t launch_fwd_sm100(const Geom& g, const unigist_problem& p, float scale, const void* q, const void* k,
                         const void* v, void* o, float* lse, cudaStream_t st) {
  const int D = p.head_dim, Hq = p.num_q_heads, Hkv = p.num_kv_heads, B = p.batch;
  CUtensorMap mq_raw, mq_gist, mk_raw, mk_gist, mv_raw, mv_gist;
  if (int32_t rc = encode_segment_map(&mq_raw, q, D, Hq, g.N, B, g.s, g.T, BM)) return rc;
  if (int32_t rc = encode_segment_map(&mq_gist, q, D, Hq, g.N, B, g.s + g.T, g.n, BM)) return rc;
  if (int32_t rc = encode_segment_map(&mk_raw, k, D, Hkv, g.N, B, g.s, g.T, BN)) return rc;
  if (int32_t rc = encode_segment_map(&mk_gist, k, D, Hkv, g.N, B, g.s + g.T, g.n, BN)) return rc;
  if (int32_t rc = encode_segment_map(&mv_raw, v, D, Hkv, g.N, B, g.s, g.T, BN)) return rc;
  if (int32_t rc = encode_segment_map(&mv_gist, v, D, Hkv, g.N, B, g.s + g.T, g.n, BN)) return rc;
  const int n_raw_qt = (g.T + BM - 1) / BM, n_gist_qt = (g.n + BM - 1) / BM;
  dim3 grid(n_raw_qt + n_gist_qt, Hq, B);
  const float scale_log2 = scale * 1.4426950408889634f;
  auto go = [&](auto kern, size_t smem) -> int32_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
    {
      KernelScope ks("attn_fwd_sm100_kernel", st);
      kern<<<grid, kThreads, smem, st>>>(mq_raw, mq_gist, mk_raw, mk_gist, mv_raw, mv_gist, g, Hq, Hkv, scale_log2,
                                         (__nv_bfloat16*)o, lse, n_raw_qt);
    }
    return check_launch("tcgen05 forward kernel");
  };
  return D == 64 ? go(attn_fwd_sm100_kernel<64>, FwdSmem<64>::kBytes) : go(attn_fwd_sm100_kernel<128>, FwdSmem<128>::kBytes);
}

int32_t fwd_sm100_take_timeout(bool* timed_out) {
  unsigned int flag = 0, zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&flag, g_fwd_timeout, sizeof(flag));
  if (e == cudaSuccess && flag) e = cudaMemcpyToSymbol(g_fwd_timeout, &zero, sizeof(zero));
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "reading the device status: %s", cudaGetErrorString(e));
  *timed_out = flag != 0;
  return UNIGIST_OK;
}

}  // namespace ug
