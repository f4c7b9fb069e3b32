// Victim selection of the replacement controller (Sec. III-E, Sec. IV-D) for large banks and large
// batches, as a sequence of small grids over all SMs.  Same result as the one-block routine in select.cuh:
// free slots ascending, then occupied slots by ascending eviction key (stale entries ahead, then lower decayed
// match rate, then least recently used), ties to the lower slot; the i-th insertable miss takes the i-th slot.
//
//   k_selmb_keys     taking-order key of every slot; bitwise AND / OR over all keys (which bytes differ at
//                    all); number of insertable misses per block of the miss list
//   k_selmb_hist     one radix-select pass per key byte, most significant first: histogram of the byte over the
//                    keys that match the prefix found so far; the block that finishes last picks the bin that
//                    holds the take-th key.  A byte on which all keys agree costs an empty launch.
//   k_selmb_count    keys below / equal to the threshold key, per block of slots
//   k_selmb_write    chosen slots written in slot order (block offsets = sums over the blocks before)
//   k_selmb_sort_*   bitonic sort of the chosen (key, slot) pairs: pieces of SORT_CAP pairs in shared memory,
//                    the steps with longer strides on global memory
//   k_selmb_assign   slots handed to the insertable misses in miss order
// No block ever waits for another block: every dependency is a grid boundary, and "the block that finishes
// last" is found with a ticket counter.  Integer arithmetic only.
#include "llmcache_internal.cuh"
#include "select.cuh"

namespace llmc {

constexpr int MB_THREADS = 1024;
constexpr uint32_t SORT_CAP = 8192;                   // pairs of one shared-memory piece (96 KB)
constexpr size_t SORT_SMEM = (size_t)SORT_CAP * 12;

// Words of the selection state (zeroed before every selection).
enum { SS_NAND = 0, SS_OR = 2, SS_PREFIX = 4, SS_SKIPPED = 6, SS_NINS = 7, SS_NOCC = 8, SS_TICKET = 16, SS_HIST = 64 };

struct SelMbArgs {
  MetaView mv;
  PolicyParams pol;
  uint32_t N, tick, epoch;
  const int32_t* miss_idx;
  const float* rq;
  const uint32_t* counts;
  int32_t* new_slot;
  unsigned long long* keys;
  uint32_t* state;
  uint32_t* blk;
  uint32_t* mcnt;
  unsigned long long* sort_key;
  uint32_t* sort_slot;
  uint32_t* tally;
  uint32_t* status;
};

__device__ __forceinline__ unsigned long long ld_u64(const uint32_t* state, int word) {
  return *reinterpret_cast<const volatile unsigned long long*>(state + word);
}
__device__ __forceinline__ uint32_t pow2_at_least(uint32_t x) {
  uint32_t p = 1;
  while (p < x) p <<= 1;
  return p;
}
// Exclusive rank of `pred` among the threads of the block (thread order) and the block total.
__device__ __forceinline__ uint32_t mb_rank(bool pred, uint32_t* warp_tot, uint32_t& total) {
  const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const uint32_t bal = __ballot_sync(0xFFFFFFFFu, pred);
  __syncthreads();
  if (lane == 0) warp_tot[w] = __popc(bal);
  __syncthreads();
  uint32_t before = 0, tot = 0;
#pragma unroll
  for (uint32_t i = 0; i < (MB_THREADS >> 5); ++i) {
    const uint32_t c = warp_tot[i];
    if (i < w) before += c;
    tot += c;
  }
  total = tot;
  return before + __popc(bal & ((1u << lane) - 1u));
}
// Sum over the threads of the block of v0 and v1 (every thread receives both).
__device__ __forceinline__ void mb_sum2(uint32_t& v0, uint32_t& v1, uint32_t* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    v0 += __shfl_xor_sync(0xFFFFFFFFu, v0, o);
    v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, o);
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = v0; red[32 + (threadIdx.x >> 5)] = v1; }
  __syncthreads();
  uint32_t a = 0, b = 0;
#pragma unroll
  for (uint32_t i = 0; i < (MB_THREADS >> 5); ++i) { a += red[i]; b += red[32 + i]; }
  v0 = a; v1 = b;
}

__global__ void __launch_bounds__(MB_THREADS) k_selmb_keys(SelMbArgs A) {
  griddep_sync();
  __shared__ unsigned long long s_nand, s_or;
  if (threadIdx.x == 0) { s_nand = 0ull; s_or = 0ull; }
  __syncthreads();
  const uint32_t j = blockIdx.x * MB_THREADS + threadIdx.x;
  unsigned long long na = 0ull, o = 0ull;
  if (j < A.N) {
    unsigned long long key = 0ull;
    if (A.mv.valid[j])
      key = evict_key(A.pol, A.tick, A.epoch, A.mv.rate[j], A.mv.rate_epoch[j], A.mv.insert_tick[j], A.mv.last_use[j]) |
            (1ull << 63);
    A.keys[j] = key;
    na = ~key; o = key;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    na |= __shfl_xor_sync(0xFFFFFFFFu, na, off);
    o |= __shfl_xor_sync(0xFFFFFFFFu, o, off);
  }
  if ((threadIdx.x & 31) == 0) { atomicOr(&s_nand, na); atomicOr(&s_or, o); }
  // insertable misses of this block's part of the miss list
  const uint32_t M = A.counts[1];
  const bool ok = j < M && A.rq[A.miss_idx[j]] > 0.f;
  const uint32_t cnt = (uint32_t)__syncthreads_count(ok);        // also orders the shared atomics above
  if (threadIdx.x == 0) {
    if (s_nand) atomicOr(reinterpret_cast<unsigned long long*>(A.state + SS_NAND), s_nand);
    if (s_or) atomicOr(reinterpret_cast<unsigned long long*>(A.state + SS_OR), s_or);
    if (blockIdx.x * MB_THREADS < M) {
      A.mcnt[blockIdx.x] = cnt;
      if (cnt) atomicAdd(A.state + SS_NINS, cnt);
    }
  }
}

__global__ void __launch_bounds__(MB_THREADS) k_selmb_hist(SelMbArgs A, uint32_t pass) {
  griddep_sync();
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_last;
  const uint32_t take = min(A.state[SS_NINS], A.N);
  if (take == 0) return;
  const unsigned long long k_and = ~ld_u64(A.state, SS_NAND), k_or = ld_u64(A.state, SS_OR);
  const uint32_t shift = 56u - 8u * pass;
  const unsigned long long prefix = ld_u64(A.state, SS_PREFIX);
  if ((((k_and ^ k_or) >> shift) & 0xFFull) == 0ull) {            // every key has the same byte here
    if (blockIdx.x == 0 && threadIdx.x == 0)
      *reinterpret_cast<unsigned long long*>(A.state + SS_PREFIX) = prefix | (k_and & (0xFFull << shift));
    return;
  }
  const uint32_t need = take - A.state[SS_SKIPPED];
  if (threadIdx.x < 256) hist[threadIdx.x] = 0;
  __syncthreads();
  const unsigned long long hi_mask = shift == 56u ? 0ull : (~0ull << (shift + 8u));
  const uint32_t j = blockIdx.x * MB_THREADS + threadIdx.x;
  const unsigned long long key = j < A.N ? A.keys[j] : 0ull;
  const bool in = j < A.N && (key & hi_mask) == prefix;
  const uint32_t digit = (uint32_t)(key >> shift) & 255u;
  // one shared-memory atomic per distinct digit of the warp
  const uint32_t active = __ballot_sync(0xFFFFFFFFu, in);
  if (in) {
    const uint32_t peers = __match_any_sync(active, digit);
    if ((threadIdx.x & 31) == (uint32_t)(__ffs(peers) - 1)) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
  }
  __syncthreads();
  uint32_t* ghist = A.state + SS_HIST + pass * 256;
  if (threadIdx.x < 256 && hist[threadIdx.x]) atomicAdd(ghist + threadIdx.x, hist[threadIdx.x]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(A.state + SS_TICKET + pass, 1u) == gridDim.x - 1 ? 1u : 0u;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (threadIdx.x < 32) {
    // the bin that holds the need-th candidate: each lane sums 8 bins, a scan over the lanes finds the lane,
    // the lane walks its 8 bins
    const uint32_t lane = threadIdx.x;
    uint32_t bins[8], mine = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { bins[i] = __ldcg(ghist + lane * 8 + i); mine += bins[i]; }
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= (uint32_t)o) incl += t;
    }
    const uint32_t excl = incl - mine;
    if (excl < need && need <= incl) {                            // exactly one lane
      uint32_t acc = excl, d = 0;
      for (; d < 7; ++d) {
        if (acc + bins[d] >= need) break;
        acc += bins[d];
      }
      *reinterpret_cast<unsigned long long*>(A.state + SS_PREFIX) = prefix | ((unsigned long long)(lane * 8 + d) << shift);
      A.state[SS_SKIPPED] = take - (need - acc);
    }
  }
}

__global__ void __launch_bounds__(MB_THREADS) k_selmb_count(SelMbArgs A) {
  griddep_sync();
  const uint32_t take = min(A.state[SS_NINS], A.N);
  if (take == 0) return;
  const unsigned long long T = ld_u64(A.state, SS_PREFIX);
  const uint32_t j = blockIdx.x * MB_THREADS + threadIdx.x;
  const unsigned long long key = j < A.N ? A.keys[j] : ~0ull;
  const uint32_t c_less = (uint32_t)__syncthreads_count(j < A.N && key < T);
  const uint32_t c_eq = (uint32_t)__syncthreads_count(j < A.N && key == T);
  if (threadIdx.x == 0) { A.blk[2 * blockIdx.x] = c_less; A.blk[2 * blockIdx.x + 1] = c_eq; }
}

__global__ void __launch_bounds__(MB_THREADS) k_selmb_write(SelMbArgs A) {
  griddep_sync();
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t red[64];
  const uint32_t take = min(A.state[SS_NINS], A.N);
  if (take == 0) return;
  const unsigned long long T = ld_u64(A.state, SS_PREFIX);
  const uint32_t need = take - A.state[SS_SKIPPED];               // keys equal to T that are taken (lowest slots)
  uint32_t less_before = 0, eq_before = 0;
  for (uint32_t i = threadIdx.x; i < blockIdx.x; i += MB_THREADS) { less_before += A.blk[2 * i]; eq_before += A.blk[2 * i + 1]; }
  mb_sum2(less_before, eq_before, red);
  const uint32_t j = blockIdx.x * MB_THREADS + threadIdx.x;
  const unsigned long long key = j < A.N ? A.keys[j] : ~0ull;
  const bool eq = j < A.N && key == T;
  uint32_t tot;
  const uint32_t eq_rank = eq_before + mb_rank(eq, warp_tot, tot);
  const bool chosen = j < A.N && (key < T || (eq && eq_rank < need));
  const uint32_t pos = less_before + min(eq_before, need) + mb_rank(chosen, warp_tot, tot);
  if (chosen) { A.sort_key[pos] = key; A.sort_slot[pos] = j; }
  const uint32_t n_occ = (uint32_t)__syncthreads_count(chosen && (key >> 63));
  if (threadIdx.x == 0 && n_occ) atomicAdd(A.state + SS_NOCC, n_occ);
  // the sort works on a power of two: pad with pairs that sort last
  const uint32_t pad = take + j;
  if (pad < pow2_at_least(take)) { A.sort_key[pad] = ~0ull; A.sort_slot[pad] = 0xFFFFFFFFu; }
}

// The steps with strides below the piece length, for merge sizes size_lo .. size_hi, on one piece per block.
__global__ void __launch_bounds__(MB_THREADS) k_selmb_sort_local(SelMbArgs A, uint32_t size_lo, uint32_t size_hi) {
  griddep_sync();
  extern __shared__ __align__(16) uint8_t sort_sm[];
  unsigned long long* skey = reinterpret_cast<unsigned long long*>(sort_sm);
  uint32_t* sval = reinterpret_cast<uint32_t*>(sort_sm + (size_t)SORT_CAP * 8);
  const uint32_t len = pow2_at_least(min(A.state[SS_NINS], A.N));
  if (len < 2 || size_lo > len) return;
  const uint32_t cap = min(SORT_CAP, len), g0 = blockIdx.x * cap;
  if (g0 >= len) return;
  for (uint32_t i = threadIdx.x; i < cap; i += MB_THREADS) { skey[i] = A.sort_key[g0 + i]; sval[i] = A.sort_slot[g0 + i]; }
  __syncthreads();
  for (uint32_t size = size_lo; size <= size_hi && size <= len; size <<= 1)
    bitonic_steps<MB_THREADS>(skey, sval, cap, g0, size, min(size >> 1, cap >> 1));
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < cap; i += MB_THREADS) { A.sort_key[g0 + i] = skey[i]; A.sort_slot[g0 + i] = sval[i]; }
}

// One compare-exchange step of merge size `size` with a stride of at least the piece length, on global memory.
__global__ void __launch_bounds__(MB_THREADS) k_selmb_sort_global(SelMbArgs A, uint32_t size, uint32_t stride) {
  griddep_sync();
  const uint32_t len = pow2_at_least(min(A.state[SS_NINS], A.N));
  if (size > len) return;
  const uint32_t t = blockIdx.x * MB_THREADS + threadIdx.x;
  if (t >= (len >> 1)) return;
  const uint32_t lg = 31 - __clz(stride);
  const uint32_t i = ((t >> lg) << (lg + 1)) | (t & (stride - 1)), l = i + stride;
  const unsigned long long ka = A.sort_key[i], kb = A.sort_key[l];
  const uint32_t va = A.sort_slot[i], vb = A.sort_slot[l];
  const bool a_gt_b = (ka > kb) || (ka == kb && va > vb);
  const bool ascending = (i & size) == 0;
  if (a_gt_b == ascending) {
    A.sort_key[i] = kb; A.sort_key[l] = ka;
    A.sort_slot[i] = vb; A.sort_slot[l] = va;
  }
}

__global__ void __launch_bounds__(MB_THREADS) k_selmb_assign(SelMbArgs A) {
  griddep_sync();
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t red[64];
  const uint32_t take = min(A.state[SS_NINS], A.N);
  const uint32_t M = A.counts[1];
  uint32_t before = 0, unused = 0;
  for (uint32_t i = threadIdx.x; i < blockIdx.x; i += MB_THREADS) before += A.mcnt[i];
  mb_sum2(before, unused, red);
  const uint32_t m = blockIdx.x * MB_THREADS + threadIdx.x;
  const bool ok = m < M && A.rq[A.miss_idx[m]] > 0.f;
  uint32_t tot;
  const uint32_t r = before + mb_rank(ok, warp_tot, tot);
  if (m < M) {
    int32_t v = -1;
    if (ok && r < take) {
      const uint32_t sv = A.sort_slot[r];
      if (bounds_ok(sv < A.N, A.status, SITE_SELECT)) v = (int32_t)sv;
    }
    A.new_slot[m] = v;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    A.tally[0] = take;
    A.tally[1] = A.state[SS_NOCC];
    A.tally[2] = M - take;
  }
}

cudaError_t setup_select_kernels() {
  return cudaFuncSetAttribute(k_selmb_sort_local, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SORT_SMEM);
}

cudaError_t launch_select_victims_mb(llmcache_bank* bk, const llmcache_probe_io* io, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  SelMbArgs A;
  A.mv = MetaView{bk->a.valid, bk->a.last_use, bk->a.insert_tick, bk->a.rate, bk->a.rate_epoch};
  A.pol = bk->pol;
  A.N = bk->desc.capacity;
  A.tick = (uint32_t)bk->tick;
  A.epoch = (uint32_t)(bk->tick / bk->pol.half_life);
  A.miss_idx = io->miss_idx;
  A.rq = io->rq;
  A.counts = io->counts;
  A.new_slot = bk->a.new_slot;
  A.keys = bk->a.sel_keys;
  A.state = bk->a.sel_state;
  A.blk = bk->a.sel_blk;
  A.mcnt = bk->a.sel_mcnt;
  A.sort_key = bk->a.sort_key;
  A.sort_slot = bk->a.sort_slot;
  A.tally = bk->a.misc;
  A.status = bk->a.status;
  const uint32_t N = A.N;
  const uint32_t nblk_n = (N + MB_THREADS - 1) / MB_THREADS, nblk_b = (B + MB_THREADS - 1) / MB_THREADS;
  ProfScope prof(bk, LLMCACHE_K_SELECT, st);
  uint64_t launches = 0;
  cudaError_t e = cudaMemsetAsync(A.state, 0, (size_t)SEL_STATE_WORDS * 4, st);
  auto go = [&](cudaError_t r) { if (e == cudaSuccess) { e = r; ++launches; } };
  if (e == cudaSuccess) go(launch_k(k_selmb_keys, dim3(nblk_n > nblk_b ? nblk_n : nblk_b), dim3(MB_THREADS), 0, st, A));
  for (uint32_t pass = 0; pass < 8 && e == cudaSuccess; ++pass)
    go(launch_k(k_selmb_hist, dim3(nblk_n), dim3(MB_THREADS), 0, st, A, pass));
  if (e == cudaSuccess) go(launch_k(k_selmb_count, dim3(nblk_n), dim3(MB_THREADS), 0, st, A));
  if (e == cudaSuccess) go(launch_k(k_selmb_write, dim3(nblk_n), dim3(MB_THREADS), 0, st, A));
  // sort of at most min(B, N) pairs (the kernels read the actual length and skip what lies beyond it)
  uint32_t maxlen = 1;
  while (maxlen < (B < N ? B : N)) maxlen <<= 1;
  if (maxlen >= 2) {
    const uint32_t pieces = (maxlen + SORT_CAP - 1) / SORT_CAP;
    if (e == cudaSuccess) go(launch_k(k_selmb_sort_local, dim3(pieces), dim3(MB_THREADS), SORT_SMEM, st, A, 2u, SORT_CAP));
    for (uint32_t size = SORT_CAP << 1; size <= maxlen && size != 0 && e == cudaSuccess; size <<= 1) {
      for (uint32_t stride = size >> 1; stride >= SORT_CAP && e == cudaSuccess; stride >>= 1)
        go(launch_k(k_selmb_sort_global, dim3(((maxlen >> 1) + MB_THREADS - 1) / MB_THREADS), dim3(MB_THREADS), 0, st, A, size, stride));
      if (e == cudaSuccess) go(launch_k(k_selmb_sort_local, dim3(pieces), dim3(MB_THREADS), SORT_SMEM, st, A, size, size));
    }
  }
  if (e == cudaSuccess) go(launch_k(k_selmb_assign, dim3(nblk_b), dim3(MB_THREADS), 0, st, A));
  if (launches) bk->n_launches += launches - 1;                  // the profiling scope has counted one
  return e;
}

}  // namespace llmc
