// Threshold decision, hit/miss compaction and metadata refresh (one kernel).
//   Sec. IV-A case equation / Algorithm 1: hit iff sim > tau (">=" selectable, Sec. III-C).
//   Sec. III-E / IV-D: recency, match count and decayed match rate of matched slots.
#include "llmcache_internal.cuh"

namespace llmc {

constexpr int DEC_THREADS = 1024;

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
                 uint32_t sim_k, int32_t ham_max) {
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
      }
      if (!is_hit) sl = -1;
      hit[b] = is_hit ? 1 : 0;
      slot[b] = sl;
      score[b] = sc;
      my_slot = sl;
      if (is_hit) atomicAdd(hitcnt + sl, 1u);
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
    const int32_t j = n_chunks == 1 ? my_slot : slot[b];
    if (j < 0) continue;
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

cudaError_t launch_decide(llmcache_bank* bk, uint32_t B, float tau, const float* rq,
                          const llmcache_probe_io* io, cudaStream_t st, uint32_t sim_k, int32_t ham_max) {
  ProfScope prof(bk, LLMCACHE_K_DECIDE, st);
  return launch_k(k_decide_compact, dim3(1), dim3(DEC_THREADS), 0, st, bk->a.best, rq, B, tau,
                  (int)(bk->desc.cmp == LLMCACHE_GE), io->hit, io->slot, io->score, io->hit_idx, io->miss_idx,
                  io->counts, bk->a.hitcnt, bk->a.stats, bk->a.last_use, bk->a.hits, bk->a.rate, bk->a.rate_epoch,
                  (uint32_t)bk->tick, (uint32_t)(bk->tick / bk->pol.half_life), sim_k, ham_max);
}

}  // namespace llmc
