// Row movers: reuse of cached layer outputs (Algorithm 1 "h_l <- h'"), the
// compaction of miss inputs, and the write-back + insertion of computed layer
// outputs (Algorithm 1 "C_l[f_X] <- h_l").  Rows are n*d elements and are moved
// verbatim with 16-byte accesses.
//
// Work is counted in units of COPY_UNIT bytes of a row.  The units of all rows to
// move form one flat list that is cut into equal spans, one per block, so every
// block moves the same number of bytes whatever the hit / miss counts are (they
// are only known on the device).
#include "llmcache_internal.cuh"

namespace llmc {

constexpr int COPY_THREADS = 256;
constexpr int COPY_UNROLL = 8;                       // 16-byte vectors in flight per thread
constexpr uint32_t COPY_UNIT = 4096;                 // bytes

// Copy `bytes` (multiple of 16) from src to up to two destinations: whole tiles of
// COPY_THREADS * COPY_UNROLL vectors with all loads issued before the stores, then the rest.
__device__ __forceinline__ void copy_bytes(const char* __restrict__ src, char* __restrict__ d0,
                                           char* __restrict__ d1, uint32_t bytes) {
  constexpr uint32_t TILE = COPY_THREADS * COPY_UNROLL * 16;          // 32 KB
  uint32_t done = 0;
  for (; done + TILE <= bytes; done += TILE) {
    const size_t base = (size_t)done + ((size_t)threadIdx.x << 4);
    uint4 v[COPY_UNROLL];
#pragma unroll
    for (int u = 0; u < COPY_UNROLL; ++u) v[u] = ld_stream16(src + base + (size_t)u * (COPY_THREADS * 16));
    if (d0) {
#pragma unroll
      for (int u = 0; u < COPY_UNROLL; ++u) st_stream16(d0 + base + (size_t)u * (COPY_THREADS * 16), v[u]);
    }
    if (d1) {
#pragma unroll
      for (int u = 0; u < COPY_UNROLL; ++u) st_stream16(d1 + base + (size_t)u * (COPY_THREADS * 16), v[u]);
    }
  }
  for (uint32_t off = done + (threadIdx.x << 4); off < bytes; off += COPY_THREADS * 16) {
    const uint4 v = ld_stream16(src + off);
    if (d0) st_stream16(d0 + off, v);
    if (d1) st_stream16(d1 + off, v);
  }
}

__device__ __forceinline__ void block_span(unsigned long long total, uint32_t n_blocks,
                                           unsigned long long& u0, unsigned long long& u1) {
  u0 = total * blockIdx.x / n_blocks;
  u1 = total * (blockIdx.x + 1) / n_blocks;
}

// Units [0, H*upr): hit rows bank.act[slot] -> h_out[b].
// Units after that (only if h_miss): miss inputs h_in[b] -> h_miss[m].
__global__ void __launch_bounds__(COPY_THREADS, 6)
k_gather(const char* __restrict__ act, uint32_t act_rows, char* __restrict__ h_out, size_t row_bytes,
         const char* __restrict__ h_in, char* __restrict__ h_miss, size_t in_row_bytes,
         const int32_t* __restrict__ slot, const int32_t* __restrict__ hit_idx,
         const int32_t* __restrict__ miss_idx, const uint32_t* __restrict__ counts,
         uint32_t* __restrict__ status, uint32_t B, uint32_t N, uint32_t slot_base, uint32_t n_total) {
  griddep_sync();
  const uint32_t H = counts[0], M = counts[1];
  const uint32_t upr = (uint32_t)((row_bytes + COPY_UNIT - 1) / COPY_UNIT);
  const uint32_t upr_in = (uint32_t)((in_row_bytes + COPY_UNIT - 1) / COPY_UNIT);
  const unsigned long long n_hit = (act && h_out) ? (unsigned long long)H * upr : 0ull;
  const unsigned long long total = n_hit + ((h_in && h_miss) ? (unsigned long long)M * upr_in : 0ull);
  unsigned long long u, u1;
  block_span(total, gridDim.x, u, u1);
  while (u < u1) {
    if (u < n_hit) {
      const uint32_t i = (uint32_t)(u / upr), w0 = (uint32_t)(u - (unsigned long long)i * upr);
      const unsigned long long left = (u1 < n_hit ? u1 : n_hit) - u;
      const uint32_t w1 = (uint32_t)min((unsigned long long)upr, w0 + left);
      const int32_t b = hit_idx[i];
      // a bank that holds the slots [slot_base, slot_base + N) of a larger one copies the rows it owns
      if (bounds_ok(i < B && (uint32_t)b < B && (uint32_t)slot[b] < n_total, status, SITE_GATHER_HIT) &&
          (uint32_t)slot[b] - slot_base < N) {
        const uint32_t row = ((uint32_t)slot[b] - slot_base) % act_rows;
        const size_t off = (size_t)w0 * COPY_UNIT;
        const uint32_t bytes = (uint32_t)(min(row_bytes, (size_t)w1 * COPY_UNIT) - off);
        copy_bytes(act + (size_t)row * row_bytes + off, h_out + (size_t)b * row_bytes + off, nullptr, bytes);
      }
      u += w1 - w0;
    } else {
      const unsigned long long jt = u - n_hit;
      const uint32_t m = (uint32_t)(jt / upr_in), w0 = (uint32_t)(jt - (unsigned long long)m * upr_in);
      const uint32_t w1 = (uint32_t)min((unsigned long long)upr_in, w0 + (u1 - u));
      const int32_t b = miss_idx[m];
      if (bounds_ok(m < B && (uint32_t)b < B, status, SITE_GATHER_MISS)) {
        const size_t off = (size_t)w0 * COPY_UNIT;
        const uint32_t bytes = (uint32_t)(min(in_row_bytes, (size_t)w1 * COPY_UNIT) - off);
        copy_bytes(h_in + (size_t)b * in_row_bytes + off, h_miss + (size_t)m * in_row_bytes + off, nullptr, bytes);
      }
      u += w1 - w0;
    }
  }
}

// Units of miss_out[m] -> h_out[miss_idx[m]] and -> act[new_slot[m]].  The block whose span holds
// the first unit of a row also writes the key and the metadata of the new entry.
__global__ void __launch_bounds__(COPY_THREADS, 6)
k_scatter_insert(const char* __restrict__ miss_out, char* __restrict__ h_out, char* __restrict__ act,
                 size_t row_bytes, const int32_t* __restrict__ miss_idx, const int32_t* __restrict__ new_slot,
                 const uint32_t* __restrict__ counts,
                 const uint4* __restrict__ q_fp, const float* __restrict__ rq, uint32_t k,
                 uint4* __restrict__ bank_fp, float* __restrict__ rb, uint8_t* __restrict__ valid,
                 uint32_t* __restrict__ last_use, uint32_t* __restrict__ insert_tick, uint32_t* __restrict__ hits,
                 uint32_t* __restrict__ rate, uint32_t* __restrict__ rate_epoch, uint32_t tick, uint32_t epoch,
                 int32_t* __restrict__ new_slot_out, const uint32_t* __restrict__ tally,
                 unsigned long long* __restrict__ stats, uint32_t* __restrict__ status, uint32_t B, uint32_t N) {
  griddep_sync();
  const uint32_t M = counts[1];
  if (blockIdx.x == 0) {
    if (new_slot_out)
      for (uint32_t m = threadIdx.x; m < M; m += COPY_THREADS) new_slot_out[m] = new_slot[m];
    if (threadIdx.x == 0) {
      stats[ST_INSERT] += tally[0];
      stats[ST_EVICT] += tally[1];
      stats[ST_DROP] += tally[2];
    }
  }
  const uint32_t upr = (uint32_t)((row_bytes + COPY_UNIT - 1) / COPY_UNIT);
  const unsigned long long total = (unsigned long long)M * upr;
  const uint32_t kv = k / 8;                      // 16-byte vectors per fingerprint row
  unsigned long long u, u1;
  block_span(total, gridDim.x, u, u1);
  while (u < u1) {
    const uint32_t m = (uint32_t)(u / upr), w0 = (uint32_t)(u - (unsigned long long)m * upr);
    const uint32_t w1 = (uint32_t)min((unsigned long long)upr, w0 + (u1 - u));
    const int32_t b = miss_idx[m];
    const int32_t v = new_slot[m];
    if (!bounds_ok(m < B && (uint32_t)b < B && (v == -1 || (uint32_t)v < N), status, SITE_SCATTER)) {
      u += w1 - w0;
      continue;
    }
    const size_t off = (size_t)w0 * COPY_UNIT;
    const uint32_t bytes = (uint32_t)(min(row_bytes, (size_t)w1 * COPY_UNIT) - off);
    char* d0 = h_out ? h_out + (size_t)b * row_bytes + off : nullptr;
    char* d1 = (act && v >= 0) ? act + (size_t)v * row_bytes + off : nullptr;
    if (miss_out && (d0 || d1)) copy_bytes(miss_out + (size_t)m * row_bytes + off, d0, d1, bytes);
    if (w0 == 0 && v >= 0) {
      for (uint32_t i = threadIdx.x; i < kv; i += COPY_THREADS)
        bank_fp[(size_t)v * kv + i] = q_fp[(size_t)b * kv + i];
      if (threadIdx.x == 0) {
        rb[v] = rq[b];
        valid[v] = 1;
        last_use[v] = tick;
        insert_tick[v] = tick;
        hits[v] = 0;
        rate[v] = HIT_Q8;
        rate_epoch[v] = epoch;
      }
    }
    u += w1 - w0;
  }
}

static int g_gather_occ = 0, g_scatter_occ = 0;      // resident blocks per SM, from the occupancy calculator

cudaError_t setup_rows_kernels() {
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_gather_occ, k_gather, COPY_THREADS, 0);
  if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&g_scatter_occ, k_scatter_insert, COPY_THREADS, 0);
  if (g_gather_occ < 1) g_gather_occ = 1;
  if (g_scatter_occ < 1) g_scatter_occ = 1;
  return e;
}

// One wave of resident blocks, but never more blocks than there could be units of work.
static uint32_t copy_grid(const llmcache_bank* bk, uint32_t B, size_t row_bytes, int occ) {
  const unsigned long long units = (unsigned long long)B * ((row_bytes + COPY_UNIT - 1) / COPY_UNIT);
  unsigned long long g = (unsigned long long)bk->sm_count * (unsigned long long)occ;
  if (units < g) g = units;
  return g ? (uint32_t)g : 1u;
}

cudaError_t launch_gather(llmcache_bank* bk, const void* h_in, void* h_out,
                          const llmcache_probe_io* io, uint32_t B, cudaStream_t st, uint32_t slot_base, uint32_t n_total) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const size_t row_bytes = (size_t)D.seq_len * D.d_model * 2;
  const size_t in_row_bytes = (size_t)D.seq_len * D.d_model * (D.hidden_dtype == LLMCACHE_BF16 ? 2 : 4);
  const bool want_miss = h_in && io->h_miss;
  const bool want_hit = bk->a.act && h_out;
  if (!want_miss && !want_hit) return cudaSuccess;
  ProfScope prof(bk, LLMCACHE_K_GATHER, st);
  return launch_k(k_gather, dim3(copy_grid(bk, B, in_row_bytes, g_gather_occ)), dim3(COPY_THREADS), 0, st,
                  (const char*)(want_hit ? bk->a.act : nullptr), D.act_rows, (char*)(want_hit ? h_out : nullptr), row_bytes,
                  (const char*)(want_miss ? h_in : nullptr), (char*)(want_miss ? io->h_miss : nullptr), in_row_bytes,
                  (const int32_t*)io->slot, (const int32_t*)io->hit_idx, (const int32_t*)io->miss_idx,
                  (const uint32_t*)io->counts, bk->a.status, B, D.capacity, slot_base, n_total ? n_total : D.capacity);
}

cudaError_t launch_scatter_insert(llmcache_bank* bk, const void* miss_out, const llmcache_probe_io* io,
                                  void* h_out, int32_t* new_slot_out, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const size_t row_bytes = (size_t)D.seq_len * D.d_model * 2;
  const uint32_t epoch = (uint32_t)(bk->tick / bk->pol.half_life);
  ProfScope prof(bk, LLMCACHE_K_SCATTER, st);
  return launch_k(k_scatter_insert, dim3(copy_grid(bk, B, row_bytes, g_scatter_occ)), dim3(COPY_THREADS), 0, st,
                  (const char*)miss_out, (char*)h_out, (char*)bk->a.act, row_bytes, (const int32_t*)io->miss_idx,
                  (const int32_t*)bk->a.new_slot, (const uint32_t*)io->counts, (const uint4*)io->fp,
                  (const float*)io->rq, D.fp_dim, (uint4*)bk->a.fp, bk->a.rb, bk->a.valid, bk->a.last_use,
                  bk->a.insert_tick, bk->a.hits, bk->a.rate, bk->a.rate_epoch, (uint32_t)bk->tick, epoch,
                  new_slot_out, (const uint32_t*)bk->a.misc, bk->a.stats, bk->a.status, B, D.capacity);
}

}  // namespace llmc
