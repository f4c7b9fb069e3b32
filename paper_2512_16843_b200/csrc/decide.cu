// Threshold decision, hit/miss compaction and metadata refresh (one kernel).
//   Sec. IV-A case equation / Algorithm 1: hit iff sim > tau (">=" selectable, Sec. III-C).
//   Sec. III-E / IV-D: recency, match count and decayed match rate of matched slots.
#include "llmcache_internal.cuh"

namespace llmc {

constexpr int DEC_THREADS = 1024;
constexpr uint32_t DEC_SINGLE_BLOCK_MAX = 2048;   // batches up to this size are decided by one block

// Exclusive rank of `pred` among the threads of the block (in thread order) and
// the block total.  warp_tot is a 32-word shared array.
__device__ __forceinline__ uint32_t block_rank(bool pred, uint32_t* warp_tot, uint32_t& total) {
  const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const uint32_t bal = __ballot_sync(0xFFFFFFFFu, pred);
  const uint32_t in_warp = __popc(bal & ((1u << lane) - 1u));
  __syncthreads();
  if (lane == 0) warp_tot[w] = __popc(bal);
  __syncthreads();
  uint32_t before = 0, tot = 0;
  const uint32_t nw = blockDim.x >> 5;
  for (uint32_t i = 0; i < nw; ++i) {
    const uint32_t c = warp_tot[i];
    if (i < w) before += c;
    tot += c;
  }
  total = tot;
  return before + in_warp;
}

// One block walks the batch in order, so hit_idx and miss_idx come out ascending.
__global__ void __launch_bounds__(DEC_THREADS)
k_decide_compact(unsigned long long* __restrict__ best, const float* __restrict__ rq,
                 uint32_t B, float tau, int cmp_ge,
                 uint8_t* __restrict__ hit, int32_t* __restrict__ slot, float* __restrict__ score,
                 int32_t* __restrict__ hit_idx, int32_t* __restrict__ miss_idx,
                 uint32_t* __restrict__ counts, uint32_t* __restrict__ hitcnt,
                 unsigned long long* __restrict__ stats,
                 uint32_t* __restrict__ last_use, uint32_t* __restrict__ hits_total, uint32_t* __restrict__ rate,
                 uint32_t* __restrict__ rate_epoch, uint32_t tick, uint32_t epoch,
                 uint32_t sim_k, int32_t ham_max, uint32_t* __restrict__ status, uint32_t N,
                 uint32_t slot_base, uint32_t n_total) {
  // slot_base, n_total: this bank holds the slots [slot_base, slot_base + N) of a bank of n_total slots that is
  // split over several (0 and N for a whole bank).  The best words carry slot numbers of the whole bank; the
  // decision, the reported slot and the index lists are the same in every part, the metadata refresh touches
  // only the slots this part owns.
  griddep_sync();
  __shared__ uint32_t warp_tot[32];
  uint32_t hbase = 0, mbase = 0, ndegen = 0;
  const uint32_t n_chunks = (B + DEC_THREADS - 1) / DEC_THREADS;
  int32_t my_slot = -1;                                  // this thread's slot when the batch fits one chunk
  for (uint32_t base = 0; base < B; base += DEC_THREADS) {
    const uint32_t b = base + threadIdx.x;
    bool is_hit = false, in_range = b < B;
    if (in_range) {
      const unsigned long long pk = best[b];
      best[b] = 0ull;                                   // ready for the next probe
      const float r = rq[b];
      float sc;
      int32_t sl = -1;
      if (!(r > 0.f)) {
        sc = 0.f;                                       // degenerate fingerprint: never a hit
        ++ndegen;
      } else if (pk == 0ull) {
        sc = -INFINITY;                                 // no occupied slot
      } else {
        sl = (int32_t)(0xFFFFFFFFu - (uint32_t)pk);
        if (sim_k) {
          // SimHash scan: the upper word is the inverted Hamming distance; the angle estimate is pi * ham / k
          const uint32_t ham = 0xFFFFFFFFu - (uint32_t)(pk >> 32);
          sc = cospif((float)ham / (float)sim_k);
          is_hit = (int32_t)ham <= ham_max;
        } else {
          sc = orderable_float((uint32_t)(pk >> 32)) * r;
          is_hit = cmp_ge ? (sc >= tau) : (sc > tau);
        }
        if (!bounds_ok((uint32_t)sl < n_total, status, SITE_DECIDE)) is_hit = false;
      }
      if (!is_hit) sl = -1;
      hit[b] = is_hit ? 1 : 0;
      slot[b] = sl;
      score[b] = sc;
      my_slot = sl;
      if (is_hit && (uint32_t)sl - slot_base < N) atomicAdd(hitcnt + ((uint32_t)sl - slot_base), 1u);
    }
    uint32_t nh;
    const uint32_t r = block_rank(is_hit, warp_tot, nh);
    if (in_range) {
      if (is_hit) hit_idx[hbase + r] = (int32_t)b;
      else        miss_idx[mbase + (threadIdx.x - r)] = (int32_t)b;
    }
    const uint32_t chunk = min((uint32_t)DEC_THREADS, B - base);
    hbase += nh;
    mbase += chunk - nh;
  }
  // Metadata refresh of matched slots (Sec. III-E / IV-D).  All matches of the batch are counted by
  // now; for each matched slot exactly one thread (the one whose exchange returns the count) applies
  // "one decay step, + 256 per match", so the result does not depend on the order of the batch, and
  // the counter is back at zero for the next probe.  The slot's metadata is fetched next to the
  // exchange, not after it.
  __syncthreads();
  for (uint32_t base = 0; base < B; base += DEC_THREADS) {
    const uint32_t b = base + threadIdx.x;
    if (b >= B) continue;
    const int32_t jg = n_chunks == 1 ? my_slot : slot[b];
    if (jg < 0 || (uint32_t)jg - slot_base >= N) continue;
    const uint32_t j = (uint32_t)jg - slot_base;
    const uint32_t c = atomicExch(hitcnt + j, 0u);
    const uint32_t old_rate = rate[j], old_epoch = rate_epoch[j], old_hits = hits_total[j];
    if (c == 0) continue;
    const unsigned long long m = (unsigned long long)rate_now(old_rate, old_epoch, epoch) + (unsigned long long)HIT_Q8 * c;
    rate[j] = m > M_CAP ? M_CAP : (uint32_t)m;
    rate_epoch[j] = epoch;
    last_use[j] = tick;
    const unsigned long long h = (unsigned long long)old_hits + c;
    hits_total[j] = h > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)h;
  }
  // degenerate count: block reduction by atomics on shared memory
  __shared__ uint32_t sdeg;
  if (threadIdx.x == 0) sdeg = 0;
  __syncthreads();
  if (ndegen) atomicAdd(&sdeg, ndegen);
  __syncthreads();
  if (threadIdx.x == 0) {
    counts[0] = hbase;
    counts[1] = mbase;
    stats[ST_SEQ] += B;
    stats[ST_HIT] += hbase;
    stats[ST_MISS] += mbase;
    stats[ST_DEGEN] += sdeg;
  }
}

// ---------------------------------------------------------------------------
// The same step for large batches, as two grids of DEC_THREADS sequences per block.
//   k_decide_flags    decision per sequence, matches per slot, hits and degenerate inputs per block
//   k_compact_touch   every block adds up the hit counts of the blocks before it (so the index lists come out
//                     ascending over the whole batch), writes its part of hit_idx / miss_idx and refreshes
//                     the metadata of the slots its sequences matched
// No block waits for another: the second grid starts when the first has finished.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(DEC_THREADS)
k_decide_flags(unsigned long long* __restrict__ best, const float* __restrict__ rq, uint32_t B, float tau, int cmp_ge,
               uint8_t* __restrict__ hit, int32_t* __restrict__ slot, float* __restrict__ score,
               uint32_t* __restrict__ hitcnt, uint32_t* __restrict__ blk_cnt, uint32_t sim_k, int32_t ham_max,
               uint32_t* __restrict__ status, uint32_t N, uint32_t slot_base, uint32_t n_total) {
  griddep_sync();
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t sdeg;
  if (threadIdx.x == 0) sdeg = 0;
  const uint32_t b = blockIdx.x * DEC_THREADS + threadIdx.x;
  bool is_hit = false, degen = false;
  if (b < B) {
    const unsigned long long pk = best[b];
    best[b] = 0ull;
    const float r = rq[b];
    float sc;
    int32_t sl = -1;
    if (!(r > 0.f)) {
      sc = 0.f;
      degen = true;
    } else if (pk == 0ull) {
      sc = -INFINITY;
    } else {
      sl = (int32_t)(0xFFFFFFFFu - (uint32_t)pk);
      if (sim_k) {
        const uint32_t ham = 0xFFFFFFFFu - (uint32_t)(pk >> 32);
        sc = cospif((float)ham / (float)sim_k);
        is_hit = (int32_t)ham <= ham_max;
      } else {
        sc = orderable_float((uint32_t)(pk >> 32)) * r;
        is_hit = cmp_ge ? (sc >= tau) : (sc > tau);
      }
      if (!bounds_ok((uint32_t)sl < n_total, status, SITE_DECIDE)) is_hit = false;
    }
    if (!is_hit) sl = -1;
    hit[b] = is_hit ? 1 : 0;
    slot[b] = sl;
    score[b] = sc;
    if (is_hit && (uint32_t)sl - slot_base < N) atomicAdd(hitcnt + ((uint32_t)sl - slot_base), 1u);
  }
  uint32_t nh;
  block_rank(is_hit, warp_tot, nh);
  const uint32_t bal = __ballot_sync(0xFFFFFFFFu, degen);
  if ((threadIdx.x & 31) == 0 && bal) atomicAdd(&sdeg, __popc(bal));
  __syncthreads();
  if (threadIdx.x == 0) {
    blk_cnt[2 * blockIdx.x] = nh;
    blk_cnt[2 * blockIdx.x + 1] = sdeg;
  }
}

// Sum of v over the threads of the block (every thread receives it).  red: 32 words of shared memory.
__device__ __forceinline__ uint32_t block_sum(uint32_t v, uint32_t* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  uint32_t tot = 0;
  const uint32_t nw = blockDim.x >> 5;
  for (uint32_t i = 0; i < nw; ++i) tot += red[i];
  return tot;
}

__global__ void __launch_bounds__(DEC_THREADS)
k_compact_touch(const uint8_t* __restrict__ hit, const int32_t* __restrict__ slot, uint32_t B,
                const uint32_t* __restrict__ blk_cnt, int32_t* __restrict__ hit_idx, int32_t* __restrict__ miss_idx,
                uint32_t* __restrict__ counts, uint32_t* __restrict__ hitcnt, unsigned long long* __restrict__ stats,
                uint32_t* __restrict__ last_use, uint32_t* __restrict__ hits_total, uint32_t* __restrict__ rate,
                uint32_t* __restrict__ rate_epoch, uint32_t tick, uint32_t epoch, uint32_t N, uint32_t slot_base) {
  griddep_sync();
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t red[32];
  const uint32_t b = blockIdx.x * DEC_THREADS + threadIdx.x;
  const bool in_range = b < B;
  const bool is_hit = in_range && hit[b] != 0;
  const int32_t jg = is_hit ? slot[b] : -1;
  const int32_t j = (jg >= 0 && (uint32_t)jg - slot_base < N) ? (int32_t)((uint32_t)jg - slot_base) : -1;   // owned: local index
  // hits in the blocks before this one
  uint32_t part = 0;
  for (uint32_t i = threadIdx.x; i < blockIdx.x; i += DEC_THREADS) part += blk_cnt[2 * i];
  const uint32_t hbase = block_sum(part, red);
  uint32_t nh;
  const uint32_t r = block_rank(is_hit, warp_tot, nh);
  if (in_range) {
    if (is_hit) hit_idx[hbase + r] = (int32_t)b;
    else        miss_idx[(blockIdx.x * DEC_THREADS - hbase) + (threadIdx.x - r)] = (int32_t)b;
  }
  if (j >= 0) {
    const uint32_t c = atomicExch(hitcnt + j, 0u);
    const uint32_t old_rate = rate[j], old_epoch = rate_epoch[j], old_hits = hits_total[j];
    if (c) {
      const unsigned long long m = (unsigned long long)rate_now(old_rate, old_epoch, epoch) + (unsigned long long)HIT_Q8 * c;
      rate[j] = m > M_CAP ? M_CAP : (uint32_t)m;
      rate_epoch[j] = epoch;
      last_use[j] = tick;
      const unsigned long long h = (unsigned long long)old_hits + c;
      hits_total[j] = h > 0xFFFFFFFFull ? 0xFFFFFFFFu : (uint32_t)h;
    }
  }
  if (blockIdx.x == gridDim.x - 1) {
    // the last block knows the batch's totals: hits before it + its own; degenerate inputs summed over all blocks
    uint32_t dpart = 0;
    for (uint32_t i = threadIdx.x; i < gridDim.x; i += DEC_THREADS) dpart += blk_cnt[2 * i + 1];
    const uint32_t ndeg = block_sum(dpart, red);
    if (threadIdx.x == 0) {
      const uint32_t H = hbase + nh;
      counts[0] = H;
      counts[1] = B - H;
      stats[ST_SEQ] += B;
      stats[ST_HIT] += H;
      stats[ST_MISS] += B - H;
      stats[ST_DEGEN] += ndeg;
    }
  }
}

// words == nullptr: the bank's own best words; else `words` (of a bank split over several: slot numbers of the
// whole bank of n_total slots, of which this bank holds [slot_base, slot_base + capacity)).
cudaError_t launch_decide(llmcache_bank* bk, uint32_t B, float tau, const float* rq,
                          const llmcache_probe_io* io, cudaStream_t st, uint32_t sim_k, int32_t ham_max,
                          unsigned long long* words, uint32_t slot_base, uint32_t n_total) {
  ProfScope prof(bk, LLMCACHE_K_DECIDE, st);
  const uint32_t tick = (uint32_t)bk->tick, epoch = (uint32_t)(bk->tick / bk->pol.half_life);
  const uint32_t N = bk->desc.capacity;
  unsigned long long* best = words ? words : bk->a.best;
  if (!words) { slot_base = 0; n_total = N; }
  if (B <= DEC_SINGLE_BLOCK_MAX)
    return launch_k(k_decide_compact, dim3(1), dim3(DEC_THREADS), 0, st, best, rq, B, tau,
                    (int)(bk->desc.cmp == LLMCACHE_GE), io->hit, io->slot, io->score, io->hit_idx, io->miss_idx,
                    io->counts, bk->a.hitcnt, bk->a.stats, bk->a.last_use, bk->a.hits, bk->a.rate, bk->a.rate_epoch,
                    tick, epoch, sim_k, ham_max, bk->a.status, N, slot_base, n_total);
  const uint32_t nblk = (B + DEC_THREADS - 1) / DEC_THREADS;
  cudaError_t e = launch_k(k_decide_flags, dim3(nblk), dim3(DEC_THREADS), 0, st, best, rq, B, tau,
                           (int)(bk->desc.cmp == LLMCACHE_GE), io->hit, io->slot, io->score, bk->a.hitcnt,
                           bk->a.blk_cnt, sim_k, ham_max, bk->a.status, N, slot_base, n_total);
  if (e != cudaSuccess) return e;
  bk->n_launches += 1;
  return launch_k(k_compact_touch, dim3(nblk), dim3(DEC_THREADS), 0, st, (const uint8_t*)io->hit,
                  (const int32_t*)io->slot, B, (const uint32_t*)bk->a.blk_cnt, io->hit_idx, io->miss_idx, io->counts,
                  bk->a.hitcnt, bk->a.stats, bk->a.last_use, bk->a.hits, bk->a.rate, bk->a.rate_epoch, tick, epoch,
                  N, slot_base);
}

}  // namespace llmc
