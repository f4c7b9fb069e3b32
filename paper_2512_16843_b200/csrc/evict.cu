// Replacement controller kernels (Sec. III-E, IV-D): the victim selection for inserts (routine in
// select.cuh) and the explicit flushes (Sec. III-E: entries that have gone unused or unmatched for too long are dropped).
#include "llmcache_internal.cuh"
#include "select.cuh"

namespace llmc {

// Flushes.  mode STALE / IDLE / ALL: one thread per slot.  SLOTS: one thread per listed slot.
__global__ void k_evict(uint8_t* __restrict__ valid, const uint32_t* __restrict__ last_use,
                        const uint32_t* __restrict__ insert_tick, const uint32_t* __restrict__ rate,
                        const uint32_t* __restrict__ rate_epoch, PolicyParams pol, uint32_t N,
                        uint32_t tick, uint32_t epoch, uint32_t mode, const int32_t* __restrict__ slots,
                        uint32_t n_slots, uint32_t* __restrict__ n_evicted, unsigned long long* __restrict__ stats) {
  griddep_sync();
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  bool go = false;
  if (mode == LLMCACHE_EVICT_SLOTS) {
    if (i < n_slots) {
      const int32_t j = slots[i];
      if (j >= 0 && (uint32_t)j < N) {
        // a slot listed twice is counted once: only the thread that flips the flag counts
        const uint32_t word = (uint32_t)j & ~3u, sh = ((uint32_t)j & 3u) * 8;
        const uint32_t old = atomicAnd(reinterpret_cast<uint32_t*>(valid + word), ~(0xFFu << sh));
        go = ((old >> sh) & 0xFFu) != 0;
      }
    }
  } else if (i < N && valid[i]) {
    if (mode == LLMCACHE_EVICT_ALL) go = true;
    else if (mode == LLMCACHE_EVICT_IDLE) go = (tick - last_use[i]) > pol.max_idle;
    else if (mode == LLMCACHE_EVICT_STALE)
      go = pol.policy == LLMCACHE_LRU_STALENESS &&
           rate_now(rate[i], rate_epoch[i], epoch) < pol.stale_floor && (tick - insert_tick[i]) >= pol.min_age;
    if (go) valid[i] = 0;
  }
  const uint32_t bal = __ballot_sync(0xFFFFFFFFu, go);
  if ((threadIdx.x & 31) == 0 && bal) {
    const uint32_t c = __popc(bal);
    if (n_evicted) atomicAdd(n_evicted, c);
    atomicAdd(stats + ST_FLUSH, (unsigned long long)c);
  }
}

// Number of occupied slots (for llmcache_bank_stats): one thread per slot, one atomic per warp.
__global__ void k_count_valid(const uint8_t* __restrict__ valid, uint32_t N, uint32_t* __restrict__ count) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t bal = __ballot_sync(0xFFFFFFFFu, i < N && valid[i] != 0);
  if ((threadIdx.x & 31) == 0 && bal) atomicAdd(count, (uint32_t)__popc(bal));
}

cudaError_t launch_count_valid(llmcache_bank* bk, uint32_t* count_dev, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(count_dev, 0, sizeof(uint32_t), st);
  if (e != cudaSuccess) return e;
  const uint32_t N = bk->desc.capacity;
  k_count_valid<<<(N + 255) / 256, 256, 0, st>>>(bk->a.valid, N, count_dev);
  return cudaGetLastError();
}

constexpr uint32_t SEL_ONE_BLOCK_MAX = 4096;

// One block.  Runs on the bank's side stream, next to the gather of the same probe.
__global__ void __launch_bounds__(SEL_THREADS) k_select_victims(SelectArgs A) { select_victims_block(A); }

cudaError_t launch_select_victims(llmcache_bank* bk, const llmcache_probe_io* io, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  // one block is quickest while the bank's keys and the batch's misses are a few thousand; beyond that the
  // selection runs as a sequence of grids over all SMs
  if (bk->desc.capacity > SEL_ONE_BLOCK_MAX || B > SEL_ONE_BLOCK_MAX) return launch_select_victims_mb(bk, io, B, st);
  SelectArgs sel;
  sel.mv = MetaView{bk->a.valid, bk->a.last_use, bk->a.insert_tick, bk->a.rate, bk->a.rate_epoch};
  sel.pol = bk->pol;
  sel.N = bk->desc.capacity;
  sel.tick = (uint32_t)bk->tick;
  sel.epoch = (uint32_t)(bk->tick / bk->pol.half_life);
  sel.miss_idx = io->miss_idx;
  sel.rq = io->rq;
  sel.counts = io->counts;
  sel.new_slot = bk->a.new_slot;
  sel.victims = bk->a.victims;
  sel.g_key = bk->a.sort_key;
  sel.g_val = bk->a.sort_slot;
  sel.sort_cap = bk->sort_len;
  sel.tally = bk->a.misc;
  sel.status = bk->a.status;
  ProfScope prof(bk, LLMCACHE_K_SELECT, st);
  k_select_victims<<<1, SEL_THREADS, 0, st>>>(sel);
  return cudaGetLastError();
}

cudaError_t launch_evict(llmcache_bank* bk, uint32_t mode, const int32_t* slots, uint32_t n,
                         uint32_t* n_evicted, cudaStream_t st) {
  const uint32_t N = bk->desc.capacity;
  const uint32_t epoch = (uint32_t)(bk->tick / bk->pol.half_life);
  if (n_evicted) {
    cudaError_t e = cudaMemsetAsync(n_evicted, 0, sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
  }
  const uint32_t work = mode == LLMCACHE_EVICT_SLOTS ? n : N;
  if (work == 0) return cudaSuccess;
  ProfScope prof(bk, LLMCACHE_K_EVICT, st);
  return launch_k(k_evict, dim3((work + 255) / 256), dim3(256), 0, st, bk->a.valid, (const uint32_t*)bk->a.last_use,
                  (const uint32_t*)bk->a.insert_tick, (const uint32_t*)bk->a.rate, (const uint32_t*)bk->a.rate_epoch,
                  bk->pol, N, (uint32_t)bk->tick, epoch, mode, slots, n, n_evicted, bk->a.stats);
}

}  // namespace llmc
