// Row movers that also aggregate what they move (fingerprint-on-write).
//
// A layer's input is the previous layer's output (Algorithm 1), and the fingerprint of that input
// starts from its mean over the positions (Sec. IV-B, "Embedding Aggregation").  Every row of the
// output passes through the SMs once anyway -- reused rows when they are copied out of the bank
// (Algorithm 1 "h_l <- h'"), computed rows when they are written back and stored (Algorithm 1
// "C_l[f_X] <- h_l") -- so the column sums are taken there and the next layer's probe does not
// have to read the [B, n, d] tensor again.
//
// Layout of the work: the position rows (d elements) of all sequences of the list (hits, or
// misses) are one flat list cut into equal spans, one per block, one block per SM.  A producer
// thread streams a span through a ring of shared-memory stages with bulk asynchronous loads; a
// second thread writes every stage to its one or two destinations with bulk asynchronous stores;
// the consumer warps add the stage's rows into per-thread column sums.  A stage is released to the
// producer when the consumers are done with it and the stores have finished reading it.  One
// vector of partial sums is written per (block, sequence it touches); k_pool_finish adds them in
// a fixed order and divides by n.  All waits are bounded.
#include "llmcache_internal.cuh"
#include "ptx.cuh"

namespace llmc {

__device__ __forceinline__ void bulk_store_1d(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
// all but the latest group have finished reading shared memory
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

struct MoveArgs {
  const char* src;           // gather: the bank's activation store; scatter: miss_out
  char* dst_out;             // h_out (or nullptr)
  char* dst_act;             // scatter: the bank's activation store (or nullptr); gather: nullptr
  const int32_t* idx;        // hit_idx or miss_idx: batch index of the i-th sequence of the list
  const int32_t* slot;       // gather: slot[b] of a hit; scatter: nullptr
  const int32_t* new_slot;   // scatter: slot the i-th miss is stored in (-1: not stored); gather: nullptr
  const uint32_t* count;     // device: length of the list
  float* partial;            // [gridDim.x * Jmax, d]
  uint32_t* status;
  uint32_t act_rows, n, d, V, R, Jmax, stage_rows, stages, cons_threads;
  uint32_t B, N;             // batch size and bank capacity (range checks of a debug build)
  // scatter only: the new entries' keys and metadata (Algorithm 1 "C_l[f_X] <- h_l"), written by the block
  // that moves the first row of a sequence; block 0 also reports the slots and adds up the counters
  const uint4* q_fp; const float* rq; uint32_t kv;                  // query fingerprints, 16-byte vectors per row
  uint4* bank_fp; float* rb; uint8_t* valid;
  uint32_t* last_use; uint32_t* insert_tick; uint32_t* hits; uint32_t* rate; uint32_t* rate_epoch;
  uint32_t tick, epoch;
  int32_t* new_slot_out; const uint32_t* tally; unsigned long long* stats;
};

// Addresses of the i-th sequence of the list.
struct SeqPtrs { const char* src; char* d0; char* d1; };
__device__ __forceinline__ SeqPtrs seq_ptrs(const MoveArgs& a, uint32_t i, size_t seq_bytes) {
  SeqPtrs p;
  const int32_t b = a.idx[i];
  if (!bounds_ok(i < a.B && (uint32_t)b < a.B && (!a.slot || (uint32_t)a.slot[b] < a.N) &&
                 (!a.new_slot || a.new_slot[i] == -1 || (uint32_t)a.new_slot[i] < a.N), a.status, SITE_MOVE)) {
    p.src = a.src;                       // a readable row; nothing is written
    p.d0 = nullptr;
    p.d1 = nullptr;
    return p;
  }
  const size_t src_row = a.slot ? (size_t)((uint32_t)a.slot[b] % a.act_rows) : (size_t)i;
  p.src = a.src + src_row * seq_bytes;
  p.d0 = a.dst_out ? a.dst_out + (size_t)b * seq_bytes : nullptr;
  p.d1 = nullptr;
  if (a.dst_act && a.new_slot) {
    const int32_t v = a.new_slot[i];
    if (v >= 0) p.d1 = a.dst_act + (size_t)v * seq_bytes;
  }
  return p;
}

__global__ void __launch_bounds__(1024, 1)
k_move_pool(const MoveArgs a) {
  griddep_sync();
  extern __shared__ __align__(128) uint8_t sm_raw[];
  const uint32_t n = a.n, d = a.d, V = a.V, R = a.R, stages = a.stages, stage_rows = a.stage_rows;
  const uint32_t cons_threads = a.cons_threads;
  const uint32_t row_bytes = V * 16;
  const size_t seq_bytes = (size_t)n * row_bytes;
  const uint32_t stage_bytes = stage_rows * row_bytes;
  const uint32_t ring = smem_u32(sm_raw);
  float* red = reinterpret_cast<float*>(sm_raw + (size_t)stages * stage_bytes);          // [R][d]
  uint8_t* tail = reinterpret_cast<uint8_t*>(red + (size_t)R * d);
  const uint32_t bar0 = smem_u32(tail);                                                  // full[stages], empty[stages]
  volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(tail + 16 * stages);   // [0] abort, [1] go
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (stages + s); };

  const uint32_t count = *a.count;
  if (blockIdx.x == 0 && a.bank_fp) {
    if (a.new_slot_out)
      for (uint32_t m = threadIdx.x; m < count; m += blockDim.x) a.new_slot_out[m] = a.new_slot[m];
    if (threadIdx.x == 0) {
      a.stats[ST_INSERT] += a.tally[0];
      a.stats[ST_EVICT] += a.tally[1];
      a.stats[ST_DROP] += a.tally[2];
    }
  }
  const unsigned long long total = (unsigned long long)count * n;
  const unsigned long long L = (total + gridDim.x - 1) / gridDim.x;
  unsigned long long r = (unsigned long long)blockIdx.x * L;
  unsigned long long r1 = r + L;
  if (r1 > total) r1 = total;
  if (r >= r1) return;                                                // nothing for this block (uniform)

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), cons_threads / 32 + 1); }
    flags[0] = 0; flags[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  uint32_t i = (uint32_t)(r / n);                                     // sequence of the list
  uint32_t it = 0;
  const unsigned long long lim = wait_limit(a.status);

  if (threadIdx.x == cons_threads) {
    // ------------------------------------------------------------------ producer (one thread)
    bool ok = true;
    if (producer_idle(a.status)) r = r1;
    while (r < r1 && ok) {
      const unsigned long long seg0 = (unsigned long long)i * n;
      unsigned long long seg_end = seg0 + n;
      if (seg_end > r1) seg_end = r1;
      const char* src = seq_ptrs(a, i, seq_bytes).src;
      while (r < seg_end) {
        const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
        const uint32_t s = it % stages, ph = (it / stages) & 1u;
        if (!mbar_wait(empty_bar(s), ph ^ 1u, flags, lim)) { ok = false; break; }
        mbar_expect_tx(full_bar(s), rows * row_bytes);
        bulk_load_1d(ring + s * stage_bytes, src + (size_t)(r - seg0) * row_bytes, rows * row_bytes, full_bar(s));
        r += rows;
        ++it;
      }
      ++i;
    }
    if (!ok) {
      flags[0] = 1;
      atomicExch(a.status, 1u);
      // loads that were started must land before the block's shared memory is released
      const uint32_t back = it < stages ? it : stages;
      volatile uint32_t never = 0;
      for (uint32_t q = 0; q < back; ++q) {
        const uint32_t itx = it - 1 - q;
        mbar_wait(full_bar(itx % stages), (itx / stages) & 1u, &never, 200000000ull);
      }
    }
  } else if (threadIdx.x == cons_threads + 32) {
    // ------------------------------------------------------------------ storer (one thread)
    uint32_t released = 0;                                            // stages handed back so far
    bool ok = true;
    while (r < r1 && ok) {
      const unsigned long long seg0 = (unsigned long long)i * n;
      unsigned long long seg_end = seg0 + n;
      if (seg_end > r1) seg_end = r1;
      const SeqPtrs p = seq_ptrs(a, i, seq_bytes);
      while (r < seg_end) {
        const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
        const uint32_t s = it % stages, ph = (it / stages) & 1u;
        if (!mbar_wait(full_bar(s), ph, flags, lim)) { ok = false; break; }
        const size_t off = (size_t)(r - seg0) * row_bytes;
        if (p.d0) bulk_store_1d(p.d0 + off, ring + s * stage_bytes, rows * row_bytes);
        if (p.d1) bulk_store_1d(p.d1 + off, ring + s * stage_bytes, rows * row_bytes);
        bulk_commit();
        ++it;
        bulk_wait_read_1();                                           // every stage but the latest has been read
        while (released + 1 < it) { mbar_arrive(empty_bar(released % stages)); ++released; }
        r += rows;
      }
      ++i;
    }
    bulk_wait_read_0();
    while (released < it) { mbar_arrive(empty_bar(released % stages)); ++released; }
    bulk_wait_all();                                                  // the writes themselves are complete
    if (!ok) { flags[0] = 1; atomicExch(a.status, 1u); }
  } else if (threadIdx.x < cons_threads) {
    // ------------------------------------------------------------------ consumers: column sums
    const bool active = threadIdx.x < V * R;
    const uint32_t col = threadIdx.x % V, rg = threadIdx.x / V;
    float* out = a.partial + (size_t)blockIdx.x * a.Jmax * d;
    while (r < r1) {
      unsigned long long seg_end = (unsigned long long)(i + 1) * n;
      if (seg_end > r1) seg_end = r1;
      if (a.bank_fp && r == (unsigned long long)i * n) {              // this block moves the sequence's first row
        const int32_t v = a.new_slot[i];
        if (v >= 0) {
          const int32_t b = a.idx[i];
          for (uint32_t c = threadIdx.x; c < a.kv; c += cons_threads)
            a.bank_fp[(size_t)v * a.kv + c] = a.q_fp[(size_t)b * a.kv + c];
          if (threadIdx.x == 0) {
            a.rb[v] = a.rq[b];
            a.valid[v] = 1;
            a.last_use[v] = a.tick;
            a.insert_tick[v] = a.tick;
            a.hits[v] = 0;
            a.rate[v] = HIT_Q8;
            a.rate_epoch[v] = a.epoch;
          }
        }
      }
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
      while (r < seg_end) {
        const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
        const uint32_t s = it % stages, ph = (it / stages) & 1u;
        if (!mbar_wait(full_bar(s), ph, flags, lim)) { flags[0] = 1; atomicExch(a.status, 1u); }
        if (active) {
          const uint32_t src = ring + s * stage_bytes + col * 16;
          for (uint32_t rr = rg; rr < rows; rr += R) {
            const uint4 v = lds16(src + rr * row_bytes);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              acc[2 * q]     += __uint_as_float(w[q] << 16);
              acc[2 * q + 1] += __uint_as_float(w[q] & 0xFFFF0000u);
            }
          }
        }
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(empty_bar(s));       // this warp is done with the stage
        r += rows;
        ++it;
      }
      if (active) {
#pragma unroll
        for (int e = 0; e < 8; ++e) red[(size_t)rg * d + col * 8 + e] = acc[e];
      }
      if (threadIdx.x == 0) flags[1] = flags[0];
      asm volatile("bar.sync 1, %0;" ::"r"(cons_threads) : "memory");
      if (flags[1]) break;                                            // uniform over the consumers
      for (uint32_t c = threadIdx.x; c < d; c += cons_threads) {
        float sum = 0.f;
        for (uint32_t q = 0; q < R; ++q) sum += red[(size_t)q * d + c];
        out[c] = sum;
      }
      asm volatile("bar.sync 1, %0;" ::"r"(cons_threads) : "memory");
      out += d;
      ++i;
    }
  }
  __syncthreads();
}

// pooled[b, :] = (sum of the partial vectors of sequence b, in block order) / n.
// With counts: the items are the hits (partials part0, list idx0) followed by the misses (part1, idx1),
// each list cut as k_move_pool cuts it.  Without: item t is sequence t of a plain pooling pass whose
// spans are L_fixed rows long.
__global__ void __launch_bounds__(128)
k_pool_finish(const float* __restrict__ part0, const float* __restrict__ part1,
              const int32_t* __restrict__ idx0, const int32_t* __restrict__ idx1,
              const uint32_t* __restrict__ counts, uint32_t B, uint32_t n, uint32_t d,
              uint32_t G0, uint32_t G1, uint32_t Jmax, uint32_t L_fixed, float* __restrict__ pooled, uint32_t ld) {
  griddep_sync();
  const uint32_t t = blockIdx.x;
  const float* part = part0;
  uint32_t i = t, b = t, cnt = B, G = G0;
  if (counts) {
    const uint32_t H = counts[0];
    if (t < H) {
      b = (uint32_t)idx0[i];
      cnt = H;
    } else {
      i = t - H;
      cnt = counts[1];
      if (i >= cnt) return;
      b = (uint32_t)idx1[i];
      part = part1;
      G = G1;
    }
  }
  const unsigned long long total = (unsigned long long)cnt * n;
  const unsigned long long L = L_fixed ? (unsigned long long)L_fixed : (total + G - 1) / G;
  const unsigned long long first = (unsigned long long)i * n, last = first + n - 1;
  const uint32_t c_lo = (uint32_t)(first / L), c_hi = (uint32_t)(last / L);
  const uint32_t j_lo = i - (uint32_t)(((unsigned long long)c_lo * L) / n);
  const float fn = (float)n;
  for (uint32_t c = threadIdx.x; c < d; c += blockDim.x) {
    float v = part[((size_t)c_lo * Jmax + j_lo) * d + c];
    for (uint32_t q = c_lo + 1; q <= c_hi; ++q) v += part[(size_t)q * Jmax * d + c];
    pooled[(size_t)b * ld + c] = v / fn;
  }
}

cudaError_t setup_move_kernels() {
  return cudaFuncSetAttribute(k_move_pool, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
}

// which: 0 = hits (bank rows -> h_out), 1 = misses (miss_out -> h_out and the bank)
cudaError_t launch_move_pool(llmcache_bank* bk, int which, const void* miss_out, void* h_out,
                             const llmcache_probe_io* io, int32_t* new_slot_out, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const PoolPlan P = pool_plan(B, D.seq_len, D.d_model, true, bk->sm_count);
  MoveArgs a{};
  a.src = (const char*)(which == 0 ? (const void*)bk->a.act : miss_out);
  a.dst_out = (char*)h_out;
  a.dst_act = which == 0 ? nullptr : (char*)bk->a.act;
  a.idx = (const int32_t*)(which == 0 ? io->hit_idx : io->miss_idx);
  a.slot = which == 0 ? (const int32_t*)io->slot : nullptr;
  a.new_slot = which == 0 ? nullptr : (const int32_t*)bk->a.new_slot;
  a.count = (const uint32_t*)io->counts + which;
  a.partial = bk->a.move_partial + (size_t)which * move_partial_floats(D.max_batch, D.d_model);
  a.status = bk->a.status;
  a.B = B;
  a.N = bk->desc.capacity;
  a.act_rows = D.act_rows;
  a.n = D.seq_len; a.d = D.d_model; a.V = P.V; a.R = P.R; a.Jmax = P.Jmax;
  a.stage_rows = P.stage_rows; a.stages = P.stages; a.cons_threads = P.cons_threads;
  if (which == 1) {
    a.q_fp = (const uint4*)io->fp; a.rq = (const float*)io->rq; a.kv = D.fp_dim / 8;
    a.bank_fp = (uint4*)bk->a.fp; a.rb = bk->a.rb; a.valid = bk->a.valid;
    a.last_use = bk->a.last_use; a.insert_tick = bk->a.insert_tick; a.hits = bk->a.hits;
    a.rate = bk->a.rate; a.rate_epoch = bk->a.rate_epoch;
    a.tick = (uint32_t)bk->tick; a.epoch = (uint32_t)(bk->tick / bk->pol.half_life);
    a.new_slot_out = new_slot_out; a.tally = (const uint32_t*)bk->a.misc; a.stats = bk->a.stats;
  }
  bk->move_grid[which] = P.grid;
  bk->move_jmax = P.Jmax;
  ProfScope prof(bk, which == 0 ? LLMCACHE_K_GATHER : LLMCACHE_K_SCATTER, st);
  return launch_k(k_move_pool, dim3(P.grid), dim3(P.cons_threads + 64), P.smem, st, a);
}

// Position means of the rows moved by the two passes of the current tick -> pooled[b * ld + c].
cudaError_t launch_pool_finish_moved(llmcache_bank* bk, const llmcache_probe_io* io, uint32_t B,
                                     float* pooled, uint32_t ld, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const float* p0 = bk->a.move_partial;
  const float* p1 = p0 + move_partial_floats(D.max_batch, D.d_model);
  ProfScope prof(bk, LLMCACHE_K_POOL_FINISH, st);
  return launch_k(k_pool_finish, dim3(B), dim3(128), 0, st, p0, p1, (const int32_t*)io->hit_idx,
                  (const int32_t*)io->miss_idx, (const uint32_t*)io->counts, B, D.seq_len, D.d_model,
                  bk->move_grid[0], bk->move_grid[1], bk->move_jmax, 0u, pooled, ld);
}

// Position means of a plain pooling pass (partials of k_pool) -> pooled[b * ld + c].
cudaError_t launch_pool_finish_plain(llmcache_bank* bk, const PoolPlan& P, uint32_t B, float* pooled, uint32_t ld,
                                     cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  ProfScope prof(bk, LLMCACHE_K_POOL_FINISH, st);
  return launch_k(k_pool_finish, dim3(B), dim3(128), 0, st, (const float*)bk->a.pool_partial, (const float*)nullptr,
                  (const int32_t*)nullptr, (const int32_t*)nullptr, (const uint32_t*)nullptr, B, D.seq_len, D.d_model,
                  P.grid, P.grid, P.Jmax, P.L, pooled, ld);
}

}  // namespace llmc
