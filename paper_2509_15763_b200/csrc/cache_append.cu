// Token-by-token maintenance of the compressed paged cache during decoding (Section 4.3): raw tokens that
// leave the local window at a compression point are dropped, and no cache entry ever moves.  Decode
// attends to every entry, in any order, so the r slots of the unit that leaves the window (when the first
// raw token after a gist arrives) are handed to the next r raw tokens; the cache stays dense and grows by
// one entry per gist unit.  Per sequence a small state array remembers the window's slots in arrival
// order:  [0] ring head  [1] ring count  [2] free count  [3] raw tokens of the open unit  [4] error
//         ring[(k + 1) * r]  slots of the window's raw tokens, oldest first (circular)
//         free[r]            evicted slots not yet reused
#include "ug_common.cuh"

namespace ug {
namespace {

constexpr int PG = UNIGIST_PAGE_TOKENS;
constexpr int kHdr = 8;

__host__ __device__ inline int state_ints(int r, int k) { return kHdr + (k + 1) * r + r; }

// After a prefix of `units_done` whole units in the cache order of compaction [sinks | gists | window raw].
__global__ void cache_state_init_kernel(int B, int s, int r, int k, int units_done, int32_t* __restrict__ state) {
  const int b = blockIdx.x;
  int32_t* st = state + (long long)b * state_ints(r, k);
  const int w_units = units_done < k ? units_done : k;
  const int cap = (k + 1) * r;
  for (int i = threadIdx.x; i < cap; i += blockDim.x) st[kHdr + i] = i < w_units * r ? s + units_done + i : -1;
  for (int i = threadIdx.x; i < r; i += blockDim.x) st[kHdr + cap + i] = -1;
  if (threadIdx.x == 0) {
    st[0] = 0;
    st[1] = w_units * r;
    st[2] = 0;
    st[3] = 0;
    st[4] = 0;
  }
}

// One block per sequence: thread 0 picks the slot and updates the state, then the block copies the token's
// K and V rows (Hkv * D bf16 each) into the page.
__global__ void __launch_bounds__(128)
cache_append_kernel(int Hkv, int vecs, int r, int k, int is_gist, const uint4* __restrict__ k_new,
                    const uint4* __restrict__ v_new, uint4* __restrict__ kc, uint4* __restrict__ vc, int num_blocks,
                    const int32_t* __restrict__ table, int max_blocks, int32_t* __restrict__ seq_lens,
                    int32_t* __restrict__ state) {
  const int b = blockIdx.x;
  int32_t* st = state + (long long)b * state_ints(r, k);
  int32_t* ring = st + kHdr;
  const int cap = (k + 1) * r;
  int32_t* freel = ring + cap;
  __shared__ int slot_sh;
  if (threadIdx.x == 0) {
    int slot = -1;
    if (!is_gist) {
      if (st[3] >= r) {
        st[4] = 1;  // a raw token after a complete unit: the gist is missing
      } else {
        // a new unit opens while the window holds k + 1 earlier units: the oldest one is seen by no token
        // from here on (its own window ended with the gist just before), so its r slots are free
        const bool evicts = st[3] == 0 && st[1] > k * r;
        if (!evicts && st[2] == 0 && seq_lens[b] >= max_blocks * PG) {
          st[4] = 3;  // the block table is too short; nothing has changed
        } else {
          if (evicts) {
            for (int i = 0; i < r; ++i) freel[st[2]++] = ring[(st[0] + i) % cap];
            st[0] = (st[0] + r) % cap;
            st[1] -= r;
          }
          if (st[2] > 0) slot = freel[--st[2]];
          else slot = seq_lens[b]++;
          ring[(st[0] + st[1]) % cap] = slot;
          ++st[1];
          ++st[3];
        }
      }
    } else {
      if (st[3] != r) {
        st[4] = 2;  // a gist before its unit is complete
      } else {
        // the gist still attends to all k + 1 units of the window; eviction waits for the next raw token
        if (st[2] == 0 && seq_lens[b] >= max_blocks * PG) {
          st[4] = 3;  // the block table is too short; nothing has changed
        } else {
          if (st[2] > 0) slot = freel[--st[2]];
          else slot = seq_lens[b]++;
          st[3] = 0;
        }
      }
    }
    slot_sh = slot;
  }
  __syncthreads();
  const int slot = slot_sh;
  if (slot < 0) return;
  int blk = table[(long long)b * max_blocks + slot / PG];
  if (blk < 0 || blk >= num_blocks) return;  // never write outside the cache
  for (int e = threadIdx.x; e < Hkv * vecs; e += blockDim.x) {
    const int hk = e / vecs, vec = e - hk * vecs;
    const long long d = (((long long)blk * Hkv + hk) * PG + slot % PG) * vecs + vec;
    kc[d] = k_new[(long long)b * Hkv * vecs + e];
    vc[d] = v_new[(long long)b * Hkv * vecs + e];
  }
}

}  // namespace

void cache_state_layout(int r, int k, int* stride_ints, int* free_list_off) {
  *stride_ints = state_ints(r, k);
  *free_list_off = kHdr + (k + 1) * r;
}

size_t cache_state_bytes(int B, int r, int k) { return (size_t)B * state_ints(r, k) * sizeof(int32_t); }

int32_t launch_cache_state_init(const Geom& g, int B, int units_done, int32_t* state, cudaStream_t st) {
  {
    KernelScope ks("cache_state_init_kernel", st);
    cache_state_init_kernel<<<B, 128, 0, st>>>(B, g.s, g.r, g.k, units_done, state);
  }
  return check_launch("cache state init kernel");
}

int32_t launch_cache_append(const Geom& g, const unigist_problem& p, int is_gist, const void* k_new, const void* v_new,
                            void* kc, void* vc, int num_blocks, const int32_t* table, int max_blocks,
                            int32_t* seq_lens, int32_t* state, cudaStream_t st) {
  {
    KernelScope ks("cache_append_kernel", st);
    cache_append_kernel<<<p.batch, 128, 0, st>>>(p.num_kv_heads, p.head_dim / 8, g.r, g.k, is_gist,
                                                 (const uint4*)k_new, (const uint4*)v_new, (uint4*)kc, (uint4*)vc,
                                                 num_blocks, table, max_blocks, seq_lens, state);
  }
  return check_launch("cache append kernel");
}

}  // namespace ug
