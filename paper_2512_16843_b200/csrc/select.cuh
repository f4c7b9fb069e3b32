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
// key (bit 63 set, which no eviction key has); ties go to the lower slot.  All loads are issued
// unconditionally so that they overlap.
__device__ __forceinline__ unsigned long long take_key(const MetaView& mv, const PolicyParams& p,
                                                       uint32_t j, uint32_t tick, uint32_t epoch) {
  const uint8_t v = mv.valid[j];
  const uint32_t r = mv.rate[j], re = mv.rate_epoch[j], it = mv.insert_tick[j], lu = mv.last_use[j];
  return v ? (evict_key(p, tick, epoch, r, re, it, lu) | (1ull << 63)) : 0ull;
}

// In-place bitonic sort of (key, slot) pairs, ascending by key then slot.  len is a power of two;
// the arrays may live in shared or global memory.  Thread t handles the pair (i, i + stride) with
// i = (t / stride) * 2 * stride + t % stride, so for stride <= 32 a warp only touches elements that
// no other warp touches in that step and a warp-level sync is enough.
__device__ __forceinline__ void bitonic_sort(unsigned long long* key, uint32_t* val, uint32_t len) {
  __syncthreads();
  for (uint32_t size = 2; size <= len; size <<= 1) {
    for (uint32_t stride = size >> 1, lg = 31 - __clz(stride);; stride >>= 1, --lg) {
      for (uint32_t t = threadIdx.x; t < (len >> 1); t += SEL_THREADS) {
        const uint32_t i = ((t >> lg) << (lg + 1)) | (t & (stride - 1)), l = i + stride;
        const unsigned long long ka = key[i], kb = key[l];
        const uint32_t va = val[i], vb = val[l];
        const bool a_gt_b = (ka > kb) || (ka == kb && va > vb);
        const bool ascending = (i & size) == 0;
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
  __syncthreads();
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
  auto key_at = [&](uint32_t j) -> unsigned long long {
    return cached ? s_cache[j] : take_key(mv, pol, j, tick, epoch);
  };
  if (threadIdx.x == 0) { s_and = ~0ull; s_or = 0ull; s_evict = 0; }
  __syncthreads();

  // keys of all slots; bitwise AND / OR over them tells which bytes differ at all
  {
    unsigned long long a = ~0ull, o = 0ull;
    for (uint32_t j = threadIdx.x; j < N; j += SEL_THREADS) {
      const unsigned long long key = take_key(mv, pol, j, tick, epoch);
      if (cached) s_cache[j] = key;
      a &= key; o |= key;
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
      for (uint32_t j = threadIdx.x; j < N; j += SEL_THREADS) {
        const unsigned long long key = key_at(j);
        if ((key & hi_mask) == prefix) atomicAdd(&hist[(uint32_t)(key >> shift) & 255u], 1u);
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
    for (uint32_t base = 0; base < N; base += SEL_THREADS) {
      const uint32_t j = base + threadIdx.x;
      const unsigned long long key = j < N ? key_at(j) : ~0ull;
      const bool eq = j < N && key == T;
      uint32_t tot_eq;
      const uint32_t r_eq = sel_rank(eq, warp_tot, tot_eq);
      const bool chosen = j < N && (key < T || (eq && n_eq_seen + r_eq < need));
      uint32_t tot_ch;
      const uint32_t r_ch = sel_rank(chosen, warp_tot, tot_ch);
      if (chosen && n_out + r_ch < pow2) {
        skey[n_out + r_ch] = key;
        sval[n_out + r_ch] = j;
        if (key >> 63) ++n_occ;
      }
      n_eq_seen += tot_eq;
      n_out += tot_ch;
    }
    if (n_occ) atomicAdd(&s_evict, n_occ);
    for (uint32_t i = take + threadIdx.x; i < pow2; i += SEL_THREADS) {
      skey[i] = ~0ull;
      sval[i] = 0xFFFFFFFFu;
    }
    bitonic_sort(skey, sval, pow2);
    for (uint32_t i = threadIdx.x; i < take; i += SEL_THREADS) victims[i] = (int32_t)sval[i];
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
