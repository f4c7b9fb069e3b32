// Row movers: reuse of cached layer outputs (Algorithm 1 "h_l <- h'"), the
// compaction of miss inputs, and the write-back + insertion of computed layer
// outputs (Algorithm 1 "C_l[f_X] <- h_l").  Rows are n*d elements and are moved
// verbatim with 16-byte accesses.
#include "llmcache_internal.cuh"

namespace llmc {

constexpr int COPY_THREADS = 256;
constexpr int COPY_UNROLL = COPY_CHUNK / (COPY_THREADS * 16);   // 8 vectors per thread per chunk

// Copy `bytes` (multiple of 16) from src to up to two destinations.
__device__ __forceinline__ void copy_chunk(const char* __restrict__ src, char* __restrict__ d0,
                                           char* __restrict__ d1, uint32_t bytes) {
  const uint32_t nvec = bytes >> 4;
  if (nvec == COPY_THREADS * COPY_UNROLL) {
    uint4 v[COPY_UNROLL];
#pragma unroll
    for (int u = 0; u < COPY_UNROLL; ++u) v[u] = ld_stream16(src + ((size_t)(u * COPY_THREADS + threadIdx.x) << 4));
#pragma unroll
    for (int u = 0; u < COPY_UNROLL; ++u) {
      const size_t off = (size_t)(u * COPY_THREADS + threadIdx.x) << 4;
      if (d0) st_stream16(d0 + off, v[u]);
      if (d1) st_stream16(d1 + off, v[u]);
    }
  } else {
    for (uint32_t i = threadIdx.x; i < nvec; i += COPY_THREADS) {
      const uint4 v = ld_stream16(src + ((size_t)i << 4));
      if (d0) st_stream16(d0 + ((size_t)i << 4), v);
      if (d1) st_stream16(d1 + ((size_t)i << 4), v);
    }
  }
}

// Work items [0, H*cpr_out): hit rows bank.act[slot] -> h_out[b].
// Work items after that (only if h_miss): miss inputs h_in[b] -> h_miss[m].
__global__ void __launch_bounds__(COPY_THREADS)
k_gather(const char* __restrict__ act, uint32_t act_rows, char* __restrict__ h_out, size_t row_bytes,
         const char* __restrict__ h_in, char* __restrict__ h_miss, size_t in_row_bytes,
         const int32_t* __restrict__ slot, const int32_t* __restrict__ hit_idx,
         const int32_t* __restrict__ miss_idx, const uint32_t* __restrict__ counts) {
  const uint32_t H = counts[0], M = counts[1];
  const uint32_t cpr = (uint32_t)((row_bytes + COPY_CHUNK - 1) / COPY_CHUNK);
  const uint32_t cpr_in = (uint32_t)((in_row_bytes + COPY_CHUNK - 1) / COPY_CHUNK);
  const unsigned long long n_hit_items = (act && h_out) ? (unsigned long long)H * cpr : 0ull;
  const unsigned long long n_items = n_hit_items + ((h_in && h_miss) ? (unsigned long long)M * cpr_in : 0ull);
  for (unsigned long long it = blockIdx.x; it < n_items; it += gridDim.x) {
    if (it < n_hit_items) {
      const uint32_t i = (uint32_t)(it / cpr), c = (uint32_t)(it - (unsigned long long)i * cpr);
      const int32_t b = hit_idx[i];
      const uint32_t row = (uint32_t)slot[b] % act_rows;
      const size_t off = (size_t)c * COPY_CHUNK;
      const uint32_t bytes = (uint32_t)min((size_t)COPY_CHUNK, row_bytes - off);
      copy_chunk(act + (size_t)row * row_bytes + off, h_out + (size_t)b * row_bytes + off, nullptr, bytes);
    } else {
      const unsigned long long jt = it - n_hit_items;
      const uint32_t m = (uint32_t)(jt / cpr_in), c = (uint32_t)(jt - (unsigned long long)m * cpr_in);
      const int32_t b = miss_idx[m];
      const size_t off = (size_t)c * COPY_CHUNK;
      const uint32_t bytes = (uint32_t)min((size_t)COPY_CHUNK, in_row_bytes - off);
      copy_chunk(h_in + (size_t)b * in_row_bytes + off, h_miss + (size_t)m * in_row_bytes + off, nullptr, bytes);
    }
  }
}

// Work item (m, c): chunk c of miss_out[m] -> h_out[miss_idx[m]] and -> act[new_slot[m]].
// The block that owns chunk 0 also writes the key and the metadata of the new entry.
__global__ void __launch_bounds__(COPY_THREADS)
k_scatter_insert(const char* __restrict__ miss_out, char* __restrict__ h_out, char* __restrict__ act,
                 size_t row_bytes, const int32_t* __restrict__ miss_idx, const int32_t* __restrict__ new_slot,
                 const uint32_t* __restrict__ counts,
                 const uint4* __restrict__ q_fp, const float* __restrict__ rq, uint32_t k,
                 uint4* __restrict__ bank_fp, float* __restrict__ rb, uint8_t* __restrict__ valid,
                 uint32_t* __restrict__ last_use, uint32_t* __restrict__ insert_tick, uint32_t* __restrict__ hits,
                 uint32_t* __restrict__ rate, uint32_t* __restrict__ rate_epoch, uint32_t tick, uint32_t epoch) {
  const uint32_t M = counts[1];
  const uint32_t cpr = (uint32_t)((row_bytes + COPY_CHUNK - 1) / COPY_CHUNK);
  const unsigned long long n_items = (unsigned long long)M * cpr;
  const uint32_t kv = k / 8;                      // 16-byte vectors per fingerprint row
  for (unsigned long long it = blockIdx.x; it < n_items; it += gridDim.x) {
    const uint32_t m = (uint32_t)(it / cpr), c = (uint32_t)(it - (unsigned long long)m * cpr);
    const int32_t b = miss_idx[m];
    const int32_t v = new_slot[m];
    const size_t off = (size_t)c * COPY_CHUNK;
    const uint32_t bytes = (uint32_t)min((size_t)COPY_CHUNK, row_bytes - off);
    char* d0 = h_out ? h_out + (size_t)b * row_bytes + off : nullptr;
    char* d1 = (act && v >= 0) ? act + (size_t)v * row_bytes + off : nullptr;
    if (miss_out && (d0 || d1)) copy_chunk(miss_out + (size_t)m * row_bytes + off, d0, d1, bytes);
    if (c == 0 && v >= 0) {
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
  }
}

static uint32_t copy_grid(const llmcache_bank* bk, uint32_t B, size_t row_bytes) {
  const unsigned long long items = (unsigned long long)B * ((row_bytes + COPY_CHUNK - 1) / COPY_CHUNK);
  unsigned long long g = (unsigned long long)bk->sm_count * 8;
  if (items < g) g = items;
  return g ? (uint32_t)g : 1u;
}

cudaError_t launch_gather(llmcache_bank* bk, const void* h_in, void* h_out,
                          const llmcache_probe_io* io, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const size_t row_bytes = (size_t)D.seq_len * D.d_model * 2;
  const size_t in_row_bytes = (size_t)D.seq_len * D.d_model * (D.hidden_dtype == LLMCACHE_BF16 ? 2 : 4);
  const bool want_miss = h_in && io->h_miss;
  const bool want_hit = bk->a.act && h_out;
  if (!want_miss && !want_hit) return cudaSuccess;
  ProfScope prof(bk, LLMCACHE_K_GATHER, st);
  k_gather<<<copy_grid(bk, B, in_row_bytes), COPY_THREADS, 0, st>>>(
      (const char*)bk->a.act, D.act_rows, (char*)h_out, row_bytes,
      (const char*)h_in, (char*)io->h_miss, in_row_bytes, io->slot, io->hit_idx, io->miss_idx, io->counts);
  return cudaGetLastError();
}

cudaError_t launch_scatter_insert(llmcache_bank* bk, const void* miss_out, const llmcache_probe_io* io,
                                  void* h_out, const int32_t* new_slot, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const size_t row_bytes = (size_t)D.seq_len * D.d_model * 2;
  const uint32_t epoch = (uint32_t)(bk->tick / bk->pol.half_life);
  ProfScope prof(bk, LLMCACHE_K_SCATTER, st);
  k_scatter_insert<<<copy_grid(bk, B, row_bytes), COPY_THREADS, 0, st>>>(
      (const char*)miss_out, (char*)h_out, (char*)bk->a.act, row_bytes, io->miss_idx, new_slot, io->counts,
      (const uint4*)io->fp, io->rq, D.fp_dim, (uint4*)bk->a.fp, bk->a.rb, bk->a.valid,
      bk->a.last_use, bk->a.insert_tick, bk->a.hits, bk->a.rate, bk->a.rate_epoch, (uint32_t)bk->tick, epoch);
  return cudaGetLastError();
}

}  // namespace llmc
