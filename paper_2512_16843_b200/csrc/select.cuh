// Victim selection of the replacement controller (Sec. III-E, Sec. IV-D), as a block-level device
// routine: which slots receive the misses of the current batch.  Free slots first, then occupied
// slots, least valuable first (stale entries ahead, then lower decayed match rate, then least
// recently used).  Integer arithmetic only.
#pragma once
#include "llmcache_internal.cuh"

namespace llmc {

constexpr int SEL_THREADS = 512;
constexpr uint32_t SEL_SMEM = 2048;            // candidates / cached keys kept in shared memory

// Exclusive rank of `pred` among the threads of the block (in thread order) and the block total.
__device__ __forceinline__ uint32_t sel_rank(bool pred, uint32_t* warp_tot, uint32_t& total) {
  const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const uint32_t bal = __ballot_sync(0xFFFFFFFFu, pred);
  const uint32_t in_warp = __popc(bal & ((1u << lane) - 1u));
  __syncthreads();
  if (lane == 0) warp_tot[w] = __popc(bal);
  __syncthreads();
  uint32_t before = 0, tot = 0;
#pragma unroll
  for (uint32_t i = 0; i < (SEL_THREADS >> 5); ++i) {
    const uint32_t c = warp_tot[i];
    if (i < w) before += c;
    tot += c;
  }
  total = tot;
  return before + in_warp;
}

struct MetaView {
  const uint8_t* valid;
  const uint32_t *last_use, *insert_tick, *rate, *rate_epoch;
};

// Order in which slots are taken: free slots first (key 0), then occupied slots by ascending eviction
// key (bit 63 set, which no eviction key has); ties go to the lower slot.
// Keys of SEL_U consecutive slots starting at j0 (slots >= N: all ones, which sorts after every real key).
// All loads are issued before the first key is formed, so that a thread has them in flight together.
constexpr int SEL_U = 4;
__device__ __forceinline__ void take_keys(const MetaView& mv, const PolicyParams& p, uint32_t j0, uint32_t N,
                                          uint32_t tick, uint32_t epoch, unsigned long long (&key)[SEL_U]) {
  uint8_t v[SEL_U];
  uint32_t r[SEL_U], re[SEL_U], it[SEL_U], lu[SEL_U];
#pragma unroll
  for (int u = 0; u < SEL_U; ++u) {
    const uint32_t j = min(j0 + u, N - 1);
    v[u] = mv.valid[j]; r[u] = mv.rate[j]; re[u] = mv.rate_epoch[j]; it[u] = mv.insert_tick[j]; lu[u] = mv.last_use[j];
  }
#pragma unroll
  for (int u = 0; u < SEL_U; ++u)
    key[u] = j0 + u >= N ? ~0ull : (v[u] ? (evict_key(p, tick, epoch, r[u], re[u], it[u], lu[u]) | (1ull << 63)) : 0ull);
}

// Exclusive prefix sum of `v` over the threads of the block (in thread order) and the block total.
__device__ __forceinline__ uint32_t sel_scan(uint32_t v, uint32_t* warp_tot, uint32_t& total) {
  const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= (uint32_t)o) incl += t;
  }
  __syncthreads();
  if (lane == 31) warp_tot[w] = incl;
  __syncthreads();
  uint32_t before = 0, tot = 0;
#pragma unroll
  for (uint32_t i = 0; i < (SEL_THREADS >> 5); ++i) {
    const uint32_t c = warp_tot[i];
    if (i < w) before += c;
    tot += c;
  }
  total = tot;
  return before + incl - v;
}

// In-place bitonic sort of (key, slot) pairs, ascending by key then slot.  len is a power of two;
// the arrays may live in shared or global memory.  Thread t handles the pair (i, i + stride) with
// i = (t / stride) * 2 * stride + t % stride, so for stride <= 32 a warp only touches elements that
// no other warp touches in that step and a warp-level sync is enough.
template <int THREADS = SEL_THREADS>
__device__ __forceinline__ void bitonic_steps(unsigned long long* key, uint32_t* val, uint32_t len, uint32_t g0,
                                              uint32_t size, uint32_t first_stride) {
  // the steps of merge size `size` with strides first_stride, first_stride / 2, ..., 1 on `len` elements whose
  // first one has index g0 in the whole sequence (the direction of a pair depends on that index)
  for (uint32_t stride = first_stride, lg = 31 - __clz(stride);; stride >>= 1, --lg) {
    for (uint32_t t = threadIdx.x; t < (len >> 1); t += THREADS) {
      const uint32_t i = ((t >> lg) << (lg + 1)) | (t & (stride - 1)), l = i + stride;
      const unsigned long long ka = key[i], kb = key[l];
      const uint32_t va = val[i], vb = val[l];
      const bool a_gt_b = (ka > kb) || (ka == kb && va > vb);
      const bool ascending = ((g0 + i) & size) == 0;
      if (a_gt_b == ascending) {
        key[i] = kb; key[l] = ka;
        val[i] = vb; val[l] = va;
      }
    }
    // a step with stride <= 32 stays inside the warp's own 64 elements; a block-level sync is only
    // needed when this step or the next one reaches further
    const uint32_t next = stride > 1 ? (stride >> 1) : size;
    if (stride > 32 || next > 32) __syncthreads(); else __syncwarp();
    if (stride == 1) break;
  }
}

__device__ __forceinline__ void bitonic_sort(unsigned long long* key, uint32_t* val, uint32_t len) {
  __syncthreads();
  for (uint32_t size = 2; size <= len; size <<= 1) bitonic_steps(key, val, len, 0, size, size >> 1);
  __syncthreads();
}

// The same sort for a sequence in global memory that is longer than the shared-memory buffers (cap elements,
// a power of two; len a larger power of two).  Every step whose stride is below cap stays inside aligned
// pieces of cap elements, so those steps run on one piece at a time in shared memory; only the steps with
// strides of cap and more (log2(len / cap) * (log2(len / cap) + 1) / 2 of them) work on global memory.
__device__ __forceinline__ void bitonic_sort_large(unsigned long long* gkey, uint32_t* gval, uint32_t len,
                                                   unsigned long long* skey, uint32_t* sval, uint32_t cap) {
  __syncthreads();
  auto pieces = [&](uint32_t size_lo, uint32_t size_hi) {
    // on every piece: the steps with strides < cap of the merge sizes size_lo .. size_hi
    for (uint32_t g0 = 0; g0 < len; g0 += cap) {
      for (uint32_t i = threadIdx.x; i < cap; i += SEL_THREADS) { skey[i] = gkey[g0 + i]; sval[i] = gval[g0 + i]; }
      __syncthreads();
      for (uint32_t size = size_lo; size <= size_hi; size <<= 1)
        bitonic_steps(skey, sval, cap, g0, size, min(size >> 1, cap >> 1));
      __syncthreads();
      for (uint32_t i = threadIdx.x; i < cap; i += SEL_THREADS) { gkey[g0 + i] = skey[i]; gval[g0 + i] = sval[i]; }
      __syncthreads();
    }
  };
  pieces(2, cap);                                                    // sorted pieces, directions alternating
  for (uint32_t size = cap << 1; size <= len; size <<= 1) {
    for (uint32_t stride = size >> 1, lg = 31 - __clz(stride); stride >= cap; stride >>= 1, --lg) {
      for (uint32_t t = threadIdx.x; t < (len >> 1); t += SEL_THREADS) {
        const uint32_t i = ((t >> lg) << (lg + 1)) | (t & (stride - 1)), l = i + stride;
        const unsigned long long ka = gkey[i], kb = gkey[l];
        const uint32_t va = gval[i], vb = gval[l];
        const bool a_gt_b = (ka > kb) || (ka == kb && va > vb);
        const bool ascending = (i & size) == 0;
        if (a_gt_b == ascending) {
          gkey[i] = kb; gkey[l] = ka;
          gval[i] = vb; gval[l] = va;
        }
      }
      __syncthreads();
    }
    pieces(size, size);
  }
}

// One block.  Output: new_slot[m] for every miss m (in miss order): the slot it is stored in, or -1
// when it is dropped.  The `take` slots that come first in the taking order are found with a radix
// select over the 64-bit keys (bytes on which all keys agree are skipped), gathered in slot order,
// sorted, and handed to the insertable misses in miss order.
// Must be called by all SEL_THREADS threads of one block.  tally[0..2] receive the number of
// inserts, of evictions among them, and of dropped misses (added to the counters at commit).
struct SelectArgs {
  MetaView mv;
  PolicyParams pol;
  uint32_t N, tick, epoch;
  const int32_t* miss_idx;
  const float* rq;
  const uint32_t* counts;
  int32_t* new_slot;
  int32_t* victims;
  unsigned long long* g_key;
  uint32_t* g_val;
  uint32_t sort_cap;
  uint32_t* tally;
  uint32_t* status;
};

__device__ __forceinline__ void select_victims_block(const SelectArgs& A) {
  const MetaView& mv = A.mv;
  const PolicyParams& pol = A.pol;
  const uint32_t N = A.N, tick = A.tick, epoch = A.epoch, sort_cap = A.sort_cap;
  const int32_t* __restrict__ miss_idx = A.miss_idx;
  const float* __restrict__ rq = A.rq;
  const uint32_t* __restrict__ counts = A.counts;
  int32_t* __restrict__ new_slot = A.new_slot;
  int32_t* __restrict__ victims = A.victims;
  unsigned long long* __restrict__ g_key = A.g_key;
  uint32_t* __restrict__ g_val = A.g_val;
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t hist[256];
  __shared__ unsigned long long s_cache[SEL_SMEM];   // keys of all slots when N <= SEL_SMEM
  __shared__ unsigned long long s_key[SEL_SMEM];     // chosen candidates
  __shared__ uint32_t s_val[SEL_SMEM];
  __shared__ unsigned long long s_and, s_or, s_prefix;
  __shared__ uint32_t s_need, s_evict;

  const uint32_t M = counts[1];
  const bool cached = N <= SEL_SMEM;
  auto keys_at = [&](uint32_t j0, unsigned long long (&key)[SEL_U]) {
    if (cached) {
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) key[u] = j0 + u < N ? s_cache[j0 + u] : ~0ull;
    } else {
      take_keys(mv, pol, j0, N, tick, epoch, key);
    }
  };
  if (threadIdx.x == 0) { s_and = ~0ull; s_or = 0ull; s_evict = 0; }
  __syncthreads();

  // keys of all slots; bitwise AND / OR over them tells which bytes differ at all
  {
    unsigned long long a = ~0ull, o = 0ull;
    for (uint32_t base = 0; base < N; base += SEL_THREADS * SEL_U) {
      const uint32_t j0 = base + threadIdx.x * SEL_U;
      if (j0 >= N) break;
      unsigned long long key[SEL_U];
      take_keys(mv, pol, j0, N, tick, epoch, key);
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) {
        if (j0 + u < N) {
          if (cached) s_cache[j0 + u] = key[u];
          a &= key[u]; o |= key[u];
        }
      }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      a &= __shfl_xor_sync(0xFFFFFFFFu, a, off);
      o |= __shfl_xor_sync(0xFFFFFFFFu, o, off);
    }
    if ((threadIdx.x & 31) == 0) { atomicAnd(&s_and, a); atomicOr(&s_or, o); }
  }
  // how many misses can be inserted at all
  uint32_t n_ins = 0;
  for (uint32_t base = 0; base < M; base += SEL_THREADS) {
    const uint32_t m = base + threadIdx.x;
    const bool ok = m < M && rq[miss_idx[m]] > 0.f;
    n_ins += (uint32_t)__syncthreads_count(ok);
  }
  __syncthreads();
  const uint32_t take = min(n_ins, N);
  const unsigned long long differ = s_and ^ s_or;

  if (take > 0) {
    // radix select, most significant byte first: the take-th key in taking order
    unsigned long long prefix = 0ull;
    uint32_t need = take;                            // rank still to locate inside the current bucket
    for (int shift = 56; shift >= 0; shift -= 8) {
      if (((differ >> shift) & 0xFFull) == 0ull) {   // every key has the same byte here
        prefix |= s_and & (0xFFull << shift);
        continue;
      }
      for (uint32_t i = threadIdx.x; i < 256; i += SEL_THREADS) hist[i] = 0;
      __syncthreads();
      const unsigned long long hi_mask = shift == 56 ? 0ull : (~0ull << (shift + 8));
      for (uint32_t base = 0; base < N; base += SEL_THREADS * SEL_U) {
        const uint32_t j0 = base + threadIdx.x * SEL_U;
        if (j0 >= N) break;
        unsigned long long key[SEL_U];
        keys_at(j0, key);
#pragma unroll
        for (int u = 0; u < SEL_U; ++u)
          if (j0 + u < N && (key[u] & hi_mask) == prefix) atomicAdd(&hist[(uint32_t)(key[u] >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (threadIdx.x < 32) {
        // warp 0 finds the bin that holds the need-th candidate: each lane sums 8 bins, an inclusive
        // scan over the lanes locates the lane, the lane walks its 8 bins
        const uint32_t lane = threadIdx.x;
        uint32_t mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) mine += hist[lane * 8 + i];
        uint32_t incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
          if (lane >= (uint32_t)o) incl += t;
        }
        const uint32_t excl = incl - mine;
        if (excl < need && need <= incl) {           // exactly one lane
          uint32_t acc = excl, digit = lane * 8;
          for (int i = 0; i < 8; ++i, ++digit) {
            if (acc + hist[digit] >= need) break;
            acc += hist[digit];
          }
          s_prefix = prefix | ((unsigned long long)digit << shift);
          s_need = need - acc;
        }
      }
      __syncthreads();
      prefix = s_prefix;
      need = s_need;
    }
    const unsigned long long T = prefix;             // threshold key; `need` slots equal to T are taken
    // collect the chosen slots in slot order, then sort them by (key, slot)
    uint32_t pow2 = 1;
    while (pow2 < take) pow2 <<= 1;
    const bool in_smem = pow2 <= SEL_SMEM;
    unsigned long long* skey = in_smem ? s_key : g_key;
    uint32_t* sval = in_smem ? s_val : g_val;
    if (!in_smem && pow2 > sort_cap) pow2 = sort_cap;   // cannot happen: sort_cap >= pow2(min(B, N))
    uint32_t n_eq_seen = 0, n_out = 0, n_occ = 0;
    for (uint32_t base = 0; base < N; base += SEL_THREADS * SEL_U) {
      // every thread takes SEL_U consecutive slots, so thread order is slot order
      const uint32_t j0 = base + threadIdx.x * SEL_U;
      unsigned long long key[SEL_U];
      if (j0 < N) {
        keys_at(j0, key);
      } else {
#pragma unroll
        for (int u = 0; u < SEL_U; ++u) key[u] = ~0ull;
      }
      uint32_t c_eq = 0;
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) c_eq += (j0 + u < N && key[u] == T) ? 1u : 0u;
      uint32_t tot_eq;
      uint32_t eq_before = n_eq_seen + sel_scan(c_eq, warp_tot, tot_eq);
      uint32_t chosen = 0, c_ch = 0;                                 // bit u: slot j0 + u is taken
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) {
        const bool in = j0 + u < N, eq = in && key[u] == T;
        if (in && (key[u] < T || (eq && eq_before < need))) { chosen |= 1u << u; ++c_ch; }
        if (eq) ++eq_before;
      }
      uint32_t tot_ch;
      uint32_t pos = n_out + sel_scan(c_ch, warp_tot, tot_ch);
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) {
        if (chosen & (1u << u)) {
          if (pos < pow2) {
            skey[pos] = key[u];
            sval[pos] = j0 + u;
            if (key[u] >> 63) ++n_occ;
          }
          ++pos;
        }
      }
      n_eq_seen += tot_eq;
      n_out += tot_ch;
    }
    if (n_occ) atomicAdd(&s_evict, n_occ);
    for (uint32_t i = take + threadIdx.x; i < pow2; i += SEL_THREADS) {
      skey[i] = ~0ull;
      sval[i] = 0xFFFFFFFFu;
    }
    if (in_smem) bitonic_sort(skey, sval, pow2);
    else         bitonic_sort_large(skey, sval, pow2, s_key, s_val, SEL_SMEM);
    for (uint32_t i = threadIdx.x; i < take; i += SEL_THREADS)
      victims[i] = bounds_ok(sval[i] < N, A.status, SITE_SELECT) ? (int32_t)sval[i] : -1;
  }
  __syncthreads();

  // hand the victims to the insertable misses in miss order
  uint32_t given = 0;
  for (uint32_t base = 0; base < M; base += SEL_THREADS) {
    const uint32_t m = base + threadIdx.x;
    const bool ok = m < M && rq[miss_idx[m]] > 0.f;
    uint32_t tot;
    const uint32_t r = sel_rank(ok, warp_tot, tot);
    if (m < M) new_slot[m] = (ok && given + r < take) ? victims[given + r] : -1;
    given += tot;
  }
  if (threadIdx.x == 0) {
    A.tally[0] = take;
    A.tally[1] = s_evict;
    A.tally[2] = M - take;
  }
}

}  // namespace llmc
