// Forward gist-masked attention on Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// The SHIFTED sequence is [sinks (s) | raw (T) | gists (n)]; a tile never straddles two of these segments.
// A thread block runs TWO query streams at once,
// each a 128-row query tile of one query head: either the same tile of two neighbouring heads of
// one KV group (when the group size is even: both streams then walk the same key tiles under the
// same mask), or two neighbouring tiles of one head.  Both streams read the same K / V tiles, which
// are loaded once into a ring in shared memory.  From the closed-form row intervals each stream
// derives, per segment, the interval of 128-key tiles that hold a visible pair; the block walks the union
// (own segment first, downwards from the diagonal, then the other segments) and a stream skips the tiles
// outside its own intervals.  Masked-out tiles are never loaded.  Per key tile and stream:
//   TMA:      K, V tiles -> shared memory (128-byte swizzle), one tensor map per segment so a tile
//             never straddles segments and rows past a segment's end read as zero.
//   tcgen05:  S = Q K^T into TMEM (fp32);   O += P V with P (bf16) read from TMEM.
//   softmax:  one warpgroup per stream, one query row per thread.  One pass over the 128 scores of
//             the row takes 2^(s - m) against the RUNNING maximum m, the row sum and the tile's own
//             maximum together; only when some row's maximum outgrew m by more than the lazy-rescale
//             threshold (always checked, seldom true after the first tile) is O rescaled and the
//             pass repeated.  Only tiles classified "partial" evaluate the mask (hidden scores are
//             set to -inf before the pass).
// The MMA issue order PV0(j), S0(j+1), PV1(j), S1(j+1) lets one stream's softmax run under the
// other stream's matrix products.
// Roles: one softmax warpgroup per stream (a thread owns a whole query row and keeps its 128 scores
// of a tile in registers), then one more warpgroup
// with the TMA producer warp and the MMA issuer / TMEM owner warp, which hands most of its registers
// to the softmax warpgroups.  TMEM: S0 | S1 | O0 | O1, 128 columns each.
#include <algorithm>

#include "sm100_ptx.cuh"
#include "ug_common.cuh"

namespace ug {
namespace {

using namespace sm100;

constexpr int BM = 128;  // query rows per tile
constexpr int BN = 128;  // keys per tile
constexpr int kStages = 4;  // ring slots; K and V tiles alternate through them
constexpr int kCols = BN;     // score columns per thread and tile
constexpr int kSmWarps = 8;   // softmax warps: 2 streams x 4 lane quarters
constexpr int kTmaWarp = kSmWarps, kMmaWarp = kSmWarps + 1;
constexpr int kThreads = (kSmWarps + 4) * 32;  // the last warpgroup: TMA warp, MMA warp, 2 idle warps
constexpr uint32_t kTmemCols = 512;
// Register split after launch: the softmax warpgroups grow, the last warpgroup shrinks.  The total must not exceed what the block was launched with, or the growing
// warpgroups would wait forever.
constexpr int kRegsLaunch = 168;  // 65536 / kThreads, rounded down to a multiple of 8
constexpr int kRegsSoftmax = 216, kRegsOther = 72;
static_assert(kThreads * (kRegsLaunch + 8) > 65536 && kThreads * kRegsLaunch <= 65536, "kRegsLaunch is stale");
static_assert((kSmWarps / 4) * kRegsSoftmax + kRegsOther <= (kSmWarps / 4 + 1) * kRegsLaunch,
              "register split exceeds the block's allocation");
constexpr float kRescaleThreshold = 8.0f;  // log2 units: O is rescaled only when the max grows by > 2^8

__device__ unsigned int g_fwd_timeout = 0;

template <int D>
struct FwdSmem {
  static constexpr int kSlab = BM * 128;          // bytes of one [128 rows x 64 bf16] slab
  static constexpr int kTile = kSlab * (D / 64);  // bytes of one [128 x D] tile
  static constexpr int kBarOff = (2 + kStages) * kTile;
  static constexpr int kBytes = kBarOff + 256 + 1024 /*align*/;
};

// One query stream: a 128-row tile of one head, with the key tiles it can see in each segment.
struct Stream {
  bool valid;
  int h, row_a, row_b;      // head; first / last row inside the segment
  RowIv iv_a, iv_b;         // visible intervals of the first / last row
  int n_sink;               // sink key tiles [0, n_sink)
  int raw_lo, raw_hi;       // raw key tiles [raw_lo, raw_hi] (none if raw_hi < raw_lo)
  int n_gist;               // gist key tiles [0, n_gist)
  __device__ bool sees(int seg, int idx) const {
    if (!valid) return false;
    if (seg == kSegRaw) return idx >= raw_lo && idx <= raw_hi;
    return idx < (seg == kSegGist ? n_gist : n_sink);
  }
};

__device__ Stream make_stream(const Geom& g, const FastDiv& rdiv, bool valid, int h, int qt, int qseg, int q_off) {
  Stream s;
  s.valid = valid;
  s.h = h;
  s.row_a = q_off + qt * BM;  // rows are numbered inside the key segment; the queries may start at q_off
  s.row_b = min(s.row_a + BM - 1, seg_len(g, qseg) - 1);
  if (!valid) {
    s.row_a = s.row_b = 0;
  }
  auto div_r = [&](int x) { return fdiv(rdiv, x); };
  s.iv_a = row_intervals_with(g, seg_base(g, qseg) + s.row_a, div_r);
  s.iv_b = row_intervals_with(g, seg_base(g, qseg) + s.row_b, div_r);
  s.n_sink = s.iv_b.hi_sink >= 0 ? s.iv_b.hi_sink / BN + 1 : 0;
  s.raw_lo = s.iv_a.lo_raw / BN;
  s.raw_hi = s.iv_b.hi_raw >= 0 ? s.iv_b.hi_raw / BN : -1;
  s.n_gist = s.iv_b.hi_gist >= 0 ? s.iv_b.hi_gist / BN + 1 : 0;
  return s;
}

// Key tiles the block visits: the union of its streams' tiles, in three runs.  First the query rows' own
// segment downwards from the tile that holds the diagonal (every row sees itself there, so the running
// maximum is finite from a stream's first tile on), then the other segments upwards.
struct TileSeq {
  int seg[3], cnt[3], start[3];  // run i: cnt[i] tiles of segment seg[i]; run 0 counts down from start[0]
  __device__ int count() const { return cnt[0] + cnt[1] + cnt[2]; }
  __device__ void at(int j, int& sg, int& idx) const {
    if (j < cnt[0]) {
      sg = seg[0];
      idx = start[0] - j;
    } else if (j < cnt[0] + cnt[1]) {
      sg = seg[1];
      idx = start[1] + (j - cnt[0]);
    } else {
      sg = seg[2];
      idx = start[2] + (j - cnt[0] - cnt[1]);
    }
  }
};

__device__ TileSeq make_tile_seq(const Stream& a, const Stream& b, int qseg) {
  int n_sink, raw_lo, raw_hi, n_gist;
  if (a.valid && b.valid) {
    n_sink = max(a.n_sink, b.n_sink);
    raw_lo = min(a.raw_lo, b.raw_lo);
    raw_hi = max(a.raw_hi, b.raw_hi);
    n_gist = max(a.n_gist, b.n_gist);
  } else {
    const Stream& s = a.valid ? a : b;
    n_sink = s.n_sink;
    raw_lo = s.raw_lo;
    raw_hi = s.raw_hi;
    n_gist = s.n_gist;
  }
  const int n_raw = raw_hi >= raw_lo ? raw_hi - raw_lo + 1 : 0;
  TileSeq t;
  if (qseg == kSegRaw) {
    t.seg[0] = kSegRaw, t.cnt[0] = n_raw, t.start[0] = raw_hi;
    t.seg[1] = kSegGist, t.cnt[1] = n_gist, t.start[1] = 0;
    t.seg[2] = kSegSink, t.cnt[2] = n_sink, t.start[2] = 0;
  } else if (qseg == kSegGist) {
    t.seg[0] = kSegGist, t.cnt[0] = n_gist, t.start[0] = n_gist - 1;
    t.seg[1] = kSegRaw, t.cnt[1] = n_raw, t.start[1] = raw_lo;
    t.seg[2] = kSegSink, t.cnt[2] = n_sink, t.start[2] = 0;
  } else {  // sink queries see sinks only
    t.seg[0] = kSegSink, t.cnt[0] = n_sink, t.start[0] = n_sink - 1;
    t.seg[1] = kSegRaw, t.cnt[1] = 0, t.start[1] = 0;
    t.seg[2] = kSegGist, t.cnt[2] = 0, t.start[2] = 0;
  }
  return t;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Bit e of the result: column 32 * c + e lies inside [lo, hi].
__device__ __forceinline__ uint32_t chunk_mask(int lo, int hi, int c) {
  const int a = max(lo - 32 * c, 0), b = min(hi - 32 * c, 31);
  return a > b ? 0u : ((0xffffffffu >> (31 - b)) & (0xffffffffu << a));
}

// Hidden columns (outside [lo, hi]) of a row of raw scores become -inf.
__device__ __forceinline__ void mask_row(uint32_t (&sc)[kCols], int lo, int hi) {
#pragma unroll
  for (int c = 0; c < kCols / 32; ++c) {
    const uint32_t bits = chunk_mask(lo, hi, c);
#pragma unroll
    for (int e = 0; e < 32; ++e) sc[c * 32 + e] = (bits >> e) & 1u ? sc[c * 32 + e] : 0xff800000u;
  }
}

// Row maximum of the raw scores of one tile.
__device__ __forceinline__ float row_max(const uint32_t (&sc)[kCols]) {
  float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
  for (int e = 0; e < kCols; e += 8) {
    m0 = max3(m0, __uint_as_float(sc[e]), __uint_as_float(sc[e + 1]));
    m1 = max3(m1, __uint_as_float(sc[e + 2]), __uint_as_float(sc[e + 3]));
    m2 = max3(m2, __uint_as_float(sc[e + 4]), __uint_as_float(sc[e + 5]));
    m3 = max3(m3, __uint_as_float(sc[e + 6]), __uint_as_float(sc[e + 7]));
  }
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// Half a pass over a row of raw scores (columns 64 * kHalf .. + 63): p = 2^(s * scale_log2 - m) written to
// TMEM as bf16 pairs; returns the sum of the half row.  The first half also leaves the maximum raw score of
// the WHOLE row in mx, so that the caller knows whether m still serves before it hands any of P over.
// m must be finite; a score of -inf gives p = 0 (or about 2^-126 where the exponential is taken on the FMA
// pipe).  The special-function unit (16 exponentials per clock and SM) bounds this loop, so kEmuNum of every
// kEmuDen column pairs go to the FMA pipe (ex2_fma2) and the maximum rides along on the ALU pipe.
constexpr int kEmuNum = 2, kEmuDen = 8;
template <int kHalf>
__device__ __forceinline__ float row_exp(const uint32_t (&sc)[kCols], uint32_t t_p, float scale_log2, float m, float& mx) {
  uint64_t l01 = f32x2(0.f, 0.f), l23 = l01;
  const uint64_t scale2 = f32x2(scale_log2, scale_log2), negm2 = f32x2(-m, -m);
  float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
  for (int c = kHalf * (kCols / 64); c < (kHalf + 1) * (kCols / 64); ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
      const int i0 = c * 32 + e;
      float x[4];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int pair = i0 / 2 + q;
        f32x2_split(fma2(f32x2(__uint_as_float(sc[i0 + 2 * q]), __uint_as_float(sc[i0 + 2 * q + 1])), scale2, negm2),
                    x[2 * q], x[2 * q + 1]);
        if ((pair * kEmuNum) % kEmuDen < kEmuNum) {
          ex2_fma2(x[2 * q], x[2 * q + 1]);
        } else {
          x[2 * q] = ex2(x[2 * q]);
          x[2 * q + 1] = ex2(x[2 * q + 1]);
        }
      }
      if (kHalf == 0) {  // the maximum of both halves: 8 columns per 4 exponentials
        const int j0 = 2 * i0;
        m0 = max3(m0, __uint_as_float(sc[j0]), __uint_as_float(sc[j0 + 1]));
        m1 = max3(m1, __uint_as_float(sc[j0 + 2]), __uint_as_float(sc[j0 + 3]));
        m0 = max3(m0, __uint_as_float(sc[j0 + 4]), __uint_as_float(sc[j0 + 5]));
        m1 = max3(m1, __uint_as_float(sc[j0 + 6]), __uint_as_float(sc[j0 + 7]));
      }
      l01 = add2(l01, f32x2(x[0], x[1]));
      l23 = add2(l23, f32x2(x[2], x[3]));
      pk[e / 2] = pack_bf16(x[0], x[1]);
      pk[e / 2 + 1] = pack_bf16(x[2], x[3]);
    }
    tmem_st(t_p + c * 16, pk);
  }
  if (kHalf == 0) mx = fmaxf(m0, m1);
  float l0, l1, l2, l3;
  f32x2_split(l01, l0, l1);
  f32x2_split(l23, l2, l3);
  return (l0 + l1) + (l2 + l3);
}

// One launch unit: a batch of sequences of one geometry with its own tensor maps (one per segment, so that
// tiles never straddle segments, ragged ends read as zero and stores past a segment's end are dropped).
// A call on one problem is one unit with a (tiles, heads, batch) grid.  A packed sample under cross-document
// masking (Section 5.1) is several units in ONE launch: the grid is flat and a block finds its unit from the
// units' first block indices.
struct alignas(64) FwdRun {
  CUtensorMap q[3], k[3], v[3], o[3];
  Geom g;
  QueryRows qr;
  float* lse;
  int n_sink_units, n_raw_units, n_units;  // n_units: x extent of the unit's grid
  int cta_begin;                           // flat grid: first block of the unit
  int plane;                               // n_units * (y extent)
  FastDiv units_div, plane_div;
};
template <int kRuns>
struct FwdRuns {
  FwdRun run[kRuns];
  int n;
};
constexpr int kMaxRunsPerLaunch = 12;  // 12 units are 20 KB of kernel parameters (the limit is 32 KB)
static_assert(sizeof(FwdRuns<kMaxRunsPerLaunch>) + 256 <= 32764, "the launch units must fit the kernel parameter space");

template <int D, int kRuns>
__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_sm100_kernel(const __grid_constant__ FwdRuns<kRuns> P, int Hq, FastDiv rdiv, FastDiv hkdiv, float scale_log2,
                      int pair_heads, int interleaved) {
  int ri = 0, bx, by, bz;
  if constexpr (kRuns == 1) {
    bx = blockIdx.x, by = blockIdx.y, bz = blockIdx.z;
  } else {
    const int c = blockIdx.x;
    while (ri + 1 < P.n && c >= P.run[ri + 1].cta_begin) ++ri;
    const int local = c - P.run[ri].cta_begin;
    bz = fdiv(P.run[ri].plane_div, local);
    const int rem = local - bz * P.run[ri].plane;
    by = fdiv(P.run[ri].units_div, rem);
    bx = rem - by * P.run[ri].n_units;
  }
  const FwdRun& R = P.run[ri];
  const Geom g = R.g;
  const QueryRows qr = R.qr;
  float* __restrict__ lse = R.lse;
  const int n_sink_units = R.n_sink_units, n_raw_units = R.n_raw_units;
  using SM = FwdSmem<D>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const uint32_t sQ[2] = {base, base + SM::kTile};
  const uint32_t ring = base + 2 * SM::kTile;
  const uint32_t bars = base + SM::kBarOff;
  const uint32_t bar_q = bars, bar_o = bars + 8;
  const uint32_t bar_s[2] = {bars + 16, bars + 24}, bar_p[2] = {bars + 32, bars + 40};  // bar_p: first half of P stored
  const uint32_t bar_p2[2] = {bars + 64 + 16 * kStages, bars + 72 + 16 * kStages};          // second half of P stored
  const uint32_t bar_full = bars + 48, bar_empty = bars + 48 + 8 * kStages;  // arrays of kStages
  const uint32_t tmem_slot = bars + 48 + 16 * kStages;
  unsigned char* gen_base = smem_dyn + (base - smem_u32(smem_dyn));
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(gen_base + SM::kBarOff + 48 + 16 * kStages);

  const int warp = threadIdx.x >> 5;
  const int b = bz;
  // heaviest units first: gist units from the end, then raw units from the end, sink units last
  const int u_lin = R.n_units - 1 - bx;
  const int qseg = u_lin < n_sink_units ? kSegSink : (u_lin < n_sink_units + n_raw_units ? kSegRaw : kSegGist);
  const int u = u_lin - (qseg == kSegSink ? 0 : (qseg == kSegRaw ? n_sink_units : n_sink_units + n_raw_units));
  const int q_off = qr.off[qseg];  // first query row of the segment (0 unless this is a prefill chunk)
  const int n_qt = (seg_len(g, qseg) - q_off + BM - 1) / BM;
  const int q_seg_base = seg_base(g, qseg);  // shifted position of the segment's row 0
  int qt[2], hh[2];
  bool sv[2];
  if (pair_heads) {
    qt[0] = qt[1] = u;
    hh[0] = 2 * by;
    hh[1] = hh[0] + 1;
    sv[0] = sv[1] = true;
  } else {
    qt[0] = 2 * u;
    qt[1] = 2 * u + 1;
    hh[0] = hh[1] = by;
    sv[0] = true;
    sv[1] = qt[1] < n_qt;
  }

  // Barriers, tensor memory and the Q loads come before the rest of the index arithmetic, which then runs
  // under the latency of those loads.
  if (threadIdx.x == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_o, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_s[i], 1);
      mbar_init(bar_p[i], 128);
      mbar_init(bar_p2[i], 128);
    }
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_fence_init();
  }
  if (warp == kMmaWarp) tmem_alloc(tmem_slot, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  bool ok = true;
  const int hk = fdiv(hkdiv, by);  // both streams share the KV head
  // tile coordinate: its first unit (a raw tile of an interleaved tensor spans 128 / r gist units)
  auto first_unit = [&](int sg, int row0) { return interleaved && sg == kSegRaw ? fdiv(rdiv, row0) : row0; };
  if (warp == kTmaWarp && elect_one()) {
    const CUtensorMap* mq = &R.q[qseg];
    mbar_arrive_expect_tx(bar_q, (sv[1] ? 2 : 1) * SM::kTile);
    for (int i = 0; i < 2; ++i) {
      if (!sv[i]) continue;
      const int row0 = qt[i] * BM;
#pragma unroll
      for (int sl = 0; sl < D / 64; ++sl)
        tma_load_5d(sQ[i] + sl * SM::kSlab, mq, bar_q, sl * 64, hh[i], 0, first_unit(qseg, row0), b);
    }
    // The first key tile is the one with the diagonal of the later stream (every stream starts in its own
    // segment, at its last row's tile): its K and V loads need none of the interval arithmetic below.
    const int last = sv[1] ? 1 : 0;
    const int idx0 = min(q_off + qt[last] * BM + BM - 1, seg_len(g, qseg) - 1) / BN;
    const CUtensorMap* mk0 = &R.k[qseg];
    const CUtensorMap* mv0 = &R.v[qseg];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      mbar_arrive_expect_tx(bar_full + 8 * t, SM::kTile);
#pragma unroll
      for (int sl = 0; sl < D / 64; ++sl)
        tma_load_5d(ring + t * SM::kTile + sl * SM::kSlab, t ? mv0 : mk0, bar_full + 8 * t, sl * 64, hk, 0,
                    first_unit(qseg, idx0 * BN), b);
    }
  }
  const Stream str0 = make_stream(g, rdiv, sv[0], hh[0], qt[0], qseg, q_off),
               str1 = make_stream(g, rdiv, sv[1], hh[1], qt[1], qseg, q_off);
  const TileSeq seq = make_tile_seq(str0, str1, qseg);
  const int nt = seq.count();
  if (warp >= kSmWarps) {
    reg_dealloc<kRegsOther>();
  if (warp == kTmaWarp) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      for (int t = 2; t < 2 * nt && ok; ++t) {  // item t: K tile of step t/2 (even t) or its V tile (odd t); 0, 1 are on their way
        int sg, idx;
        seq.at(t >> 1, sg, idx);
        const CUtensorMap* m = (t & 1) ? &R.v[sg] : &R.k[sg];
        const int slot = t % kStages, use = t / kStages;
        if (use > 0) ok = mbar_wait(bar_empty + 8 * slot, (use - 1) & 1);
        if (!ok) break;
        mbar_arrive_expect_tx(bar_full + 8 * slot, SM::kTile);
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl)
          tma_load_5d(ring + slot * SM::kTile + sl * SM::kSlab, m, bar_full + 8 * slot, sl * 64, hk, 0,
                      first_unit(sg, idx * BN), b);
      }
      if (!ok) atomicExch(&g_fwd_timeout, 1u);
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc_qk = make_idesc_bf16(BM, BN, false, false);
      constexpr uint32_t idesc_pv = make_idesc_bf16(BM, D, false, true);
      int n_s[2] = {0, 0}, n_pv[2] = {0, 0};  // products issued so far per stream
      // descriptors: constant high word, low word = start address / 16 stepped per 16-element k step
      constexpr uint32_t kHi = smem_desc_hi(1024);
      const uint32_t q_lo[2] = {smem_desc_lo(sQ[0], 16), smem_desc_lo(sQ[1], 16)};
      auto issue_s = [&](int i, uint32_t sK) {
        const uint32_t k_lo = smem_desc_lo(sK, 16);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk / 4) * SM::kSlab + (kk % 4) * 32) >> 4;
          umma_ss(tmem + i * 128, smem_desc_join(q_lo[i] + off, kHi), smem_desc_join(k_lo + off, kHi), idesc_qk,
                  kk > 0);
        }
        umma_commit(bar_s[i]);
        ++n_s[i];
      };
      auto issue_pv = [&](int i, uint32_t sV, int half) {  // the k steps of one half of the keys of the tile
        // V tile is MN-major: 16 keys = 2048 B per k step, 64-column groups SM::kSlab apart
        const uint32_t v_lo = smem_desc_lo(sV, SM::kSlab);
#pragma unroll
        for (int k4 = 0; k4 < BN / 32; ++k4) {
          const int kk = half * (BN / 32) + k4;
          umma_ts(tmem + 256 + i * 128, tmem + i * 128 + kk * 8, smem_desc_join(v_lo + kk * (2048 >> 4), kHi),
                  idesc_pv, (n_pv[i] > 0 || kk > 0) ? 1u : 0u);
        }
        n_pv[i] += half;
      };
      auto slot_of = [&](int t) { return t % kStages; };
      auto wait_full = [&](int t) { return mbar_wait(bar_full + 8 * slot_of(t), (t / kStages) & 1); };
      int sg, nx_sg = 0, idx, nx_idx = 0;
      ok = mbar_wait(bar_q, 0);
      if (ok && nt > 0) {
        seq.at(0, sg, idx);
        ok = wait_full(0);
        if (ok) {
          tc_fence_after();
          if (str0.sees(sg, idx)) issue_s(0, ring + slot_of(0) * SM::kTile);
          if (str1.sees(sg, idx)) issue_s(1, ring + slot_of(0) * SM::kTile);
          umma_commit(bar_empty + 8 * slot_of(0));
        }
      }
      for (int j = 0; j < nt && ok; ++j) {
        seq.at(j, sg, idx);
        const bool has_next = j + 1 < nt;
        if (has_next) seq.at(j + 1, nx_sg, nx_idx);
        const int tv = 2 * j + 1, tk = 2 * j + 2;
        ok = wait_full(tv);
        if (!ok) break;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const Stream& si = i ? str1 : str0;
          if (si.sees(sg, idx)) {
            // the first half of P is handed over while the softmax still works on the second
            ok = mbar_wait(bar_p[i], n_pv[i] & 1);
            if (!ok) break;
            tc_fence_after();
            issue_pv(i, ring + slot_of(tv) * SM::kTile, 0);
            ok = mbar_wait(bar_p2[i], n_pv[i] & 1);
            if (!ok) break;
            tc_fence_after();
            issue_pv(i, ring + slot_of(tv) * SM::kTile, 1);
          }
          if (i == 1) umma_commit(bar_empty + 8 * slot_of(tv));
          if (has_next) {
            if (i == 0) {
              ok = wait_full(tk);
              if (!ok) break;
              tc_fence_after();
            }
            if (si.sees(nx_sg, nx_idx)) issue_s(i, ring + slot_of(tk) * SM::kTile);
            if (i == 1) umma_commit(bar_empty + 8 * slot_of(tk));
          }
        }
      }
      if (ok) umma_commit(bar_o);
      if (!ok) atomicExch(&g_fwd_timeout, 1u);
    }
  }
  } else {
    reg_alloc<kRegsSoftmax>();
    // ------------------------------------------------------------ softmax + epilogue (one row per thread)
    const int i = warp / 4;  // stream
    const Stream me = i ? str1 : str0;
    if (me.valid) {
      const int r_in_tile = (warp & 3) * 32 + (threadIdx.x & 31);
      const int row = min(me.row_a + r_in_tile, me.row_b);
      const RowIv my = row_intervals(g, q_seg_base + row);
      const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
      const uint32_t tS = tmem + i * 128 + lane_base, tO = tmem + 256 + i * 128 + lane_base;
      float m_run = -INFINITY, l_run = 0.f;
      int cnt = 0;

      for (int j = 0; j < nt && ok; ++j) {
        int sg, idx;
        seq.at(j, sg, idx);
        if (!me.sees(sg, idx)) continue;
        const int col0 = idx * BN;
        bool full;
        int lo, hi;  // visible columns of this row, relative to the tile
        if (sg == kSegSink) {
          full = col0 + BN - 1 <= me.iv_a.hi_sink;
          lo = 0;
          hi = my.hi_sink - col0;
        } else if (sg == kSegRaw) {
          full = col0 >= me.iv_b.lo_raw && col0 + BN - 1 <= me.iv_a.hi_raw;
          lo = my.lo_raw - col0;
          hi = my.hi_raw - col0;
        } else {
          full = col0 + BN - 1 <= me.iv_a.hi_gist;
          lo = 0;
          hi = my.hi_gist - col0;
        }
        ok = mbar_wait_warp(bar_s[i], cnt & 1);
        if (!ok) break;
        tc_fence_after();

        // the whole score row of this tile sits in registers between the two passes
        uint32_t sc[kCols];
#pragma unroll
        for (int c = 0; c < kCols / 32; ++c) tmem_ld32(tS + c * 32, sc + c * 32);
        tmem_wait_ld();
        if (!full) mask_row(sc, lo, hi);
        // the first tile has no running maximum to go by: take its own first
        if (cnt == 0) m_run = row_max(sc) * scale_log2;
        float tile_sum;
        for (int pass = 0; pass < 2; ++pass) {
          // first half of the row: p = 2^(s * scale_log2 - m) against the running maximum, bf16 P into TMEM
          // (over the first 64 columns of S), and the whole row's own maximum
          float mx;
          tile_sum = row_exp<0>(sc, tS, scale_log2, m_run == -INFINITY ? 0.f : m_run, mx);
          const float mx_s = mx * scale_log2;
          const bool need = mx_s > m_run + kRescaleThreshold;
          if (!__any_sync(0xffffffffu, need)) break;
          // some row of this warp outgrew its running maximum: rescale and take the half again
          const float m_new = need ? mx_s : m_run;
          const float f = need ? ex2(m_run - m_new) : 1.f;  // m_run = -inf gives 0
          l_run *= f;
          m_run = m_new;
          tmem_wait_st();
          if (cnt > 0) {  // S of this step complete implies the previous PV complete: O is stable here
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t v[32];
              tmem_ld(tO + c * 32, v);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * f);
              tmem_st(tO + c * 32, v);
            }
          }
        }
        // hand the first half of P over, so that its part of P V runs under the second half's exponentials
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p[i]);
        float unused;
        tile_sum += row_exp<1>(sc, tS, scale_log2, m_run == -INFINITY ? 0.f : m_run, unused);
        l_run += tile_sum;
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p2[i]);
        ++cnt;
      }
      if (ok) ok = mbar_wait_warp(bar_o, 0);
      if (ok) {
        tc_fence_after();
        const float inv_l = 1.f / l_run;
        // O leaves through shared memory and TMA stores: a thread's row-wise 16-byte stores to global memory
        // would touch 32 rows per warp instruction.  Every product has completed, so the stream's Q tile is free:
        // the normalised rows go there in the tile layout of the loads (128-byte swizzle, one slab per 64 columns).
        const uint32_t srow = sQ[i] + r_in_tile * 128;
        uint32_t v[D];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) tmem_ld32(tO + c * 32, v + c * 32);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
#pragma unroll
          for (int e0 = 0; e0 < 32; e0 += 8) {
            const int e = c * 32 + e0;
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(v[e]) * inv_l, __uint_as_float(v[e + 1]) * inv_l);
            pk.y = pack_bf16(__uint_as_float(v[e + 2]) * inv_l, __uint_as_float(v[e + 3]) * inv_l);
            pk.z = pack_bf16(__uint_as_float(v[e + 4]) * inv_l, __uint_as_float(v[e + 5]) * inv_l);
            pk.w = pack_bf16(__uint_as_float(v[e + 6]) * inv_l, __uint_as_float(v[e + 7]) * inv_l);
            const int chunk = e / 8;  // 16-byte chunk of the row: slab chunk / 8, position (chunk % 8) ^ (row % 8)
            st_shared_v4(srow + (chunk >> 3) * SM::kSlab + (((chunk & 7) ^ (r_in_tile & 7)) << 4), pk);
          }
        }
        if (me.row_a + r_in_tile <= me.row_b)
          lse[((long long)b * Hq + me.h) * qr.n_out + qr.out_base[qseg] + (me.row_a + r_in_tile - q_off)] =
              (m_run + log2f(l_run)) * 0.6931471805599453f;
      } else {
        atomicExch(&g_fwd_timeout, 1u);
      }
      // all four warps of the stream get here, whatever their waits returned
      fence_proxy_async_smem();
      named_barrier_sync(1 + i, 128);
      if (ok && (warp & 3) == 0 && elect_one()) {
        // rows past the end of the segment lie outside the map and are not written
        const CUtensorMap* mo = &R.o[qseg];
        const int row0 = qt[i] * BM;
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl)
          tma_store_5d(mo, sQ[i] + sl * SM::kSlab, sl * 64, me.h, 0, first_unit(qseg, row0), b);
        bulk_commit_group();
        bulk_wait_group_read0();  // shared memory must outlive the reads of the store
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}

}  // namespace

namespace {
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
int32_t get_encode_fn(EncodeFn* out) {
  static EncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return fail(UNIGIST_ERR_CUDA, "cuTensorMapEncodeTiled is not available: %s", cudaGetErrorString(e));
    encode = reinterpret_cast<EncodeFn>(fn);
  }
  *out = encode;
  return UNIGIST_OK;
}
int32_t encode_map(CUtensorMap* map, const void* base, int D, int H, long long N, int B, long long seg_first_row,
                   long long seg_rows, int box_cols, int box_rows, int elem_bytes) {
  EncodeFn encode;
  if (int32_t rc = get_encode_fn(&encode)) return rc;
  const cuuint64_t eb = (cuuint64_t)elem_bytes;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)seg_rows, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)D * eb, (cuuint64_t)H * D * eb, (cuuint64_t)N * H * D * eb};
  const cuuint32_t box[4] = {(cuuint32_t)box_cols, 1, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  void* addr = const_cast<char*>(static_cast<const char*>(base)) + seg_first_row * H * D * elem_bytes;
  const bool bf16 = elem_bytes == 2;
  CUresult r = encode(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, addr, dims,
                      strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      bf16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(UNIGIST_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return UNIGIST_OK;
}
}  // namespace

int32_t encode_segment_map(CUtensorMap* map, const void* base, int D, int H, long long N, int B,
                           long long seg_first_row, long long seg_rows, int box_rows) {
  return encode_map(map, base, D, H, N, B, seg_first_row, seg_rows, 64, box_rows, 2);
}

int32_t encode_segment_map_f32(CUtensorMap* map, const void* base, int D, int H, long long N, int B,
                               long long seg_first_row, long long seg_rows, int box_cols, int box_rows) {
  return encode_map(map, base, D, H, N, B, seg_first_row, seg_rows, box_cols, box_rows, 4);
}

int32_t encode_tile_map(CUtensorMap* map, const void* base, int D, int H, int B, int s, int T, int r, int n_gists,
                        bool interleaved, int segment) {
  const bool raw_segment = segment == kSegRaw;
  EncodeFn encode;
  if (int32_t rc = get_encode_fn(&encode)) return rc;
  const long long n = n_gists, N = (long long)s + T + n;
  const cuuint64_t row_bytes = (cuuint64_t)H * D * 2;
  long long first_row, units, unit_rows, unit_stride_rows;
  if (segment == kSegSink) {  // the sinks are a prefix in either order; a tensor map cannot be empty
    first_row = 0;
    units = s > 0 ? s : 1;
    unit_rows = 1;
    unit_stride_rows = 1;
  } else if (!interleaved) {
    first_row = raw_segment ? s : (long long)s + T;
    units = raw_segment ? T : n;
    unit_rows = 1;
    unit_stride_rows = 1;
  } else if (raw_segment) {
    first_row = s;
    units = n;
    unit_rows = r;
    unit_stride_rows = r + 1;
  } else {
    first_row = (long long)s + r;  // the first gist sits after the first r raw rows
    units = n;
    unit_rows = 1;
    unit_stride_rows = r + 1;
  }
  const cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)unit_rows, (cuuint64_t)units, (cuuint64_t)B};
  const cuuint64_t strides[4] = {(cuuint64_t)D * 2, row_bytes, row_bytes * (cuuint64_t)unit_stride_rows,
                                 row_bytes * (cuuint64_t)N};
  const cuuint32_t box[5] = {64, 1, (cuuint32_t)unit_rows, (cuuint32_t)(128 / unit_rows), 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  void* addr = const_cast<char*>(static_cast<const char*>(base)) + first_row * row_bytes;
  CUresult rc = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, addr, dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) return fail(UNIGIST_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)rc);
  return UNIGIST_OK;
}

int32_t encode_map_2d_bf16(CUtensorMap* map, const void* base, long long rows, int cols, int box_rows, int box_cols) {
  EncodeFn encode;
  if (int32_t rc = get_encode_fn(&encode)) return rc;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(UNIGIST_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return UNIGIST_OK;
}

namespace {

// Two streams per block: neighbouring heads of a KV group when the group size is even, otherwise
// neighbouring query tiles of one head.
int fwd_pair_heads(const unigist_problem& p) { return (p.num_q_heads / p.num_kv_heads) % 2 == 0 ? 1 : 0; }

// Tensor maps and tile counts of one launch unit: `batch` sequences of geometry g whose first rows are
// q, k, v, o (and lse).  With `chunk` the queries are the tail of each segment only (chunk-wise prefill).
int32_t fill_fwd_run(FwdRun* R, const Geom& g, const unigist_problem& p, int batch, bool il, const void* q, const void* k,
                     const void* v, void* o, float* lse, const QueryRows* chunk) {
  const int D = p.head_dim, Hq = p.num_q_heads, Hkv = p.num_kv_heads;
  if (chunk) {
    R->qr = *chunk;
  } else {
    for (int sg = 0; sg < 3; ++sg) R->qr.off[sg] = 0, R->qr.out_base[sg] = seg_base(g, sg);
    R->qr.n_out = g.N;
  }
  // the Q tensor holds the query rows only: the tail of each segment from qr.off on
  const int sq = g.s - R->qr.off[kSegSink], Tq = g.T - R->qr.off[kSegRaw], nq = g.n - R->qr.off[kSegGist];
  for (int sg = 0; sg < 3; ++sg) {  // per segment: sinks, raw, gists (O has the geometry of Q)
    if (int32_t rc = encode_tile_map(&R->q[sg], q, D, Hq, batch, sq, Tq, g.r, nq, il, sg)) return rc;
    if (int32_t rc = encode_tile_map(&R->o[sg], o, D, Hq, batch, sq, Tq, g.r, nq, il, sg)) return rc;
    if (int32_t rc = encode_tile_map(&R->k[sg], k, D, Hkv, batch, g.s, g.T, g.r, g.n, il, sg)) return rc;
    if (int32_t rc = encode_tile_map(&R->v[sg], v, D, Hkv, batch, g.s, g.T, g.r, g.n, il, sg)) return rc;
  }
  const int n_sink_qt = (sq + BM - 1) / BM, n_raw_qt = (Tq + BM - 1) / BM, n_gist_qt = (nq + BM - 1) / BM;
  const int pair = fwd_pair_heads(p);
  R->n_sink_units = pair ? n_sink_qt : (n_sink_qt + 1) / 2;
  R->n_raw_units = pair ? n_raw_qt : (n_raw_qt + 1) / 2;
  const int n_gist_units = pair ? n_gist_qt : (n_gist_qt + 1) / 2;
  R->n_units = R->n_sink_units + R->n_raw_units + n_gist_units;
  R->g = g;
  R->lse = lse;
  const int ydim = pair ? Hq / 2 : Hq;
  R->plane = R->n_units * ydim;
  R->units_div = make_fastdiv(R->n_units);
  R->plane_div = make_fastdiv(R->plane);
  R->cta_begin = 0;
  return UNIGIST_OK;
}

template <typename Kern, typename Params>
int32_t go_fwd(Kern kern, size_t smem, dim3 grid, const Params& P, const unigist_problem& p, float scale, bool il,
               cudaStream_t st) {
  const int Hq = p.num_q_heads, Hkv = p.num_kv_heads, pair = fwd_pair_heads(p);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  {
    KernelScope ks("attn_fwd_sm100_kernel", st);
    kern<<<grid, kThreads, smem, st>>>(P, Hq, make_fastdiv(p.ratio), make_fastdiv(pair ? (Hq / Hkv) / 2 : Hq / Hkv),
                                       scale * 1.4426950408889634f, pair, il ? 1 : 0);
  }
  return check_launch("tcgen05 forward kernel");
}

}  // namespace

int32_t launch_fwd_sm100(const Geom& g, const unigist_problem& p, float scale, const void* q, const void* k,
                         const void* v, void* o, float* lse, cudaStream_t st, const QueryRows* chunk) {
  const bool il = (p.flags & UNIGIST_FLAG_INTERLEAVED) != 0 && !chunk;
  FwdRuns<1> P;
  P.n = 1;
  if (int32_t rc = fill_fwd_run(&P.run[0], g, p, p.batch, il, q, k, v, o, lse, chunk)) return rc;
  const dim3 grid(P.run[0].n_units, fwd_pair_heads(p) ? p.num_q_heads / 2 : p.num_q_heads, p.batch);
  return p.head_dim == 64 ? go_fwd(attn_fwd_sm100_kernel<64, 1>, FwdSmem<64>::kBytes, grid, P, p, scale, il, st)
                          : go_fwd(attn_fwd_sm100_kernel<128, 1>, FwdSmem<128>::kBytes, grid, P, p, scale, il, st);
}

int32_t launch_fwd_sm100_runs(const SeqRun* runs, int n_runs, const unigist_problem& p, float scale, const void* q,
                              const void* k, const void* v, void* o, float* lse, cudaStream_t st) {
  const bool il = (p.flags & UNIGIST_FLAG_INTERLEAVED) != 0;
  const size_t rq = (size_t)p.num_q_heads * p.head_dim * 2, rk = (size_t)p.num_kv_heads * p.head_dim * 2;
  for (int first = 0; first < n_runs; first += kMaxRunsPerLaunch) {  // one launch per kMaxRunsPerLaunch units
    FwdRuns<kMaxRunsPerLaunch> P;
    P.n = n_runs - first < kMaxRunsPerLaunch ? n_runs - first : kMaxRunsPerLaunch;
    int order[kMaxRunsPerLaunch];  // the longest run's blocks start first
    for (int i = 0; i < P.n; ++i) order[i] = i;
    std::stable_sort(order, order + P.n, [&](int a, int b) {
      return (long long)runs[first + a].g.N * runs[first + a].batch > (long long)runs[first + b].g.N * runs[first + b].batch;
    });
    long long ctas = 0;
    for (int i = 0; i < P.n; ++i) {
      const SeqRun& r = runs[first + order[i]];
      if (int32_t rc = fill_fwd_run(&P.run[i], r.g, p, r.batch, il, (const char*)q + r.first_row * rq,
                                    (const char*)k + r.first_row * rk, (const char*)v + r.first_row * rk,
                                    (char*)o + r.first_row * rq, lse + r.first_row * p.num_q_heads, nullptr))
        return rc;
      P.run[i].cta_begin = (int)ctas;
      ctas += (long long)P.run[i].plane * r.batch;
      if (ctas > 0x7fffffffLL) return fail(UNIGIST_ERR_SHAPE, "packed sample too large for one grid");
    }
    for (int i = P.n; i < kMaxRunsPerLaunch; ++i) P.run[i] = P.run[0];  // unused slots: defined contents, never selected
    const dim3 grid((unsigned)ctas, 1, 1);
    const int32_t rc = p.head_dim == 64 ? go_fwd(attn_fwd_sm100_kernel<64, kMaxRunsPerLaunch>, FwdSmem<64>::kBytes, grid, P, p, scale, il, st)
                                        : go_fwd(attn_fwd_sm100_kernel<128, kMaxRunsPerLaunch>, FwdSmem<128>::kBytes, grid, P, p, scale, il, st);
    if (rc) return rc;
  }
  return UNIGIST_OK;
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
