// Fingerprint kernels (Sec. IV-B): pooled reduction over the sequence
// positions, centring + projection, unit-length scaling, bf16 rounding.
#include "llmcache_internal.cuh"
#include "ptx.cuh"

namespace llmc {

// ---------------------------------------------------------------------------
// Pool.  The B*n rows of the batch are one flat list that is cut into equal
// spans, one per block (one block per SM), so every block streams the same
// number of bytes.  A span may cross sequence boundaries: a block writes one
// vector of partial sums per sequence it touches,
//     partial[(block * Jmax + j), :] = sum of its rows of the j-th sequence it touches.
//
// The rows of a span are contiguous in memory.  One producer thread moves them
// into a ring of shared-memory stages with bulk asynchronous copies (completion
// counted on an mbarrier per stage), which keeps well over 100 KB of reads in
// flight per SM without holding them in registers.  The consumer threads form a
// V x R grid: V = 16-byte vectors per row, R = rows taken per pass; every thread
// always owns the same E columns, so the running sums live in registers.  At the
// end of a sequence's rows the R row groups are combined through shared memory
// in a fixed order (deterministic).  A stage never crosses a sequence boundary.
// All waits are bounded; on expiry the status word is set and the block drains
// its copies and leaves.
// ---------------------------------------------------------------------------
template <bool BF16>
__global__ void __launch_bounds__(1024, 1)
k_pool(const uint4* __restrict__ h, float* __restrict__ partial, uint32_t* __restrict__ status,
       uint32_t B, uint32_t n, uint32_t d, uint32_t V, uint32_t R, uint32_t L, uint32_t Jmax,
       uint32_t stage_rows, uint32_t stages, uint32_t cons_threads) {
  griddep_sync();
  constexpr int E = BF16 ? 8 : 4;
  extern __shared__ __align__(128) uint8_t sm_raw[];
  const uint32_t row_bytes = V * 16;
  const uint32_t stage_bytes = stage_rows * row_bytes;
  const uint32_t ring = smem_u32(sm_raw);
  float* red = reinterpret_cast<float*>(sm_raw + (size_t)stages * stage_bytes);          // [R][d]
  uint8_t* tail = reinterpret_cast<uint8_t*>(red + (size_t)R * d);
  const uint32_t bar0 = smem_u32(tail);                                                  // full[stages], empty[stages]
  volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(tail + 16 * stages);   // [0] abort, [1] go
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (stages + s); };

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), cons_threads / 32); }
    flags[0] = 0; flags[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const unsigned long long total = (unsigned long long)B * n;
  unsigned long long r = (unsigned long long)blockIdx.x * L;
  unsigned long long r1 = r + L;
  if (r1 > total) r1 = total;
  uint32_t b = (uint32_t)(r / n);
  uint32_t it = 0;

  if (threadIdx.x >= cons_threads) {
    // ---------------------------------------------------------------- producer (one thread)
    if (threadIdx.x == cons_threads) {
      bool ok = true;
      while (r < r1 && ok) {
        unsigned long long seg_end = (unsigned long long)(b + 1) * n;
        if (seg_end > r1) seg_end = r1;
        while (r < seg_end) {
          const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
          const uint32_t s = it % stages, ph = (it / stages) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, flags)) { ok = false; break; }
          mbar_expect_tx(full_bar(s), rows * row_bytes);
          bulk_load_1d(ring + s * stage_bytes, h + r * V, rows * row_bytes, full_bar(s));
          r += rows;
          ++it;
        }
        ++b;
      }
      if (!ok) {
        flags[0] = 1;
        atomicExch(status, 1u);
        // copies that were started must land before the block's shared memory is released
        const uint32_t back = it < stages ? it : stages;
        volatile uint32_t never = 0;
        for (uint32_t i = 0; i < back; ++i) {
          const uint32_t itx = it - 1 - i;
          mbar_wait(full_bar(itx % stages), (itx / stages) & 1u, &never, 200000000ull);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers
    const bool active = threadIdx.x < V * R;
    const uint32_t col = threadIdx.x % V, rg = threadIdx.x / V;
    float* out = partial + (size_t)blockIdx.x * Jmax * d;
    while (r < r1) {
      unsigned long long seg_end = (unsigned long long)(b + 1) * n;
      if (seg_end > r1) seg_end = r1;
      float acc[E];
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] = 0.f;
      while (r < seg_end) {
        const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
        const uint32_t s = it % stages, ph = (it / stages) & 1u;
        if (!mbar_wait(full_bar(s), ph, flags)) { flags[0] = 1; atomicExch(status, 1u); }
        if (active) {
          const uint32_t src = ring + s * stage_bytes + col * 16;
          for (uint32_t rr = rg; rr < rows; rr += R) {
            const uint4 v = lds16(src + rr * row_bytes);
            if (BF16) {
              const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                acc[2 * i]     += __uint_as_float(w[i] << 16);
                acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
              }
            } else {
              acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
              acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
            }
          }
        }
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(empty_bar(s));      // this warp is done with the stage
        r += rows;
        ++it;
      }
      // combine the row groups of this sequence piece (consumer threads only)
      if (active) {
#pragma unroll
        for (int e = 0; e < E; ++e) red[(size_t)rg * d + col * E + e] = acc[e];
      }
      if (threadIdx.x == 0) flags[1] = flags[0];
      asm volatile("bar.sync 1, %0;" ::"r"(cons_threads) : "memory");
      if (flags[1]) break;                                           // uniform over the consumers
      for (uint32_t i = threadIdx.x; i < d; i += cons_threads) {
        float sum = 0.f;
        for (uint32_t q = 0; q < R; ++q) sum += red[(size_t)q * d + i];
        out[i] = sum;
      }
      asm volatile("bar.sync 1, %0;" ::"r"(cons_threads) : "memory");
      out += d;
      ++b;
    }
  }
  __syncthreads();
}

// ---------------------------------------------------------------------------
// Project + normalise: G sequences per block, 128 threads per sequence in the
// element-wise phases.
//   p = (sum of the sequence's partial vectors) / n - mu ;  g = p . P  (or p when no projection)
//   q = bf16(g / ||g||) ; rq = 1 / ||q||
// P is read with 16-byte loads: a thread owns 8 adjacent output columns and
// every `slices`-th row; the row slices are combined through shared memory in a
// fixed order.
// ---------------------------------------------------------------------------
constexpr int PROJ_G = 2;
constexpr int PROJ_THREADS = 1024;
constexpr int PROJ_TPS = PROJ_THREADS / PROJ_G;      // threads per sequence

// Sum over the TPS threads that serve one sequence (fixed order).  red: [PROJ_THREADS / 32] floats.
__device__ __forceinline__ float group_sum(float v, float* red, int group) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float tot = 0.f;
  constexpr int WPG = PROJ_TPS / 32;
#pragma unroll
  for (int i = 0; i < WPG; ++i) tot += red[group * WPG + i];
  return tot;
}

__global__ void __launch_bounds__(PROJ_THREADS)
k_project(const float* __restrict__ partial, const __nv_bfloat16* __restrict__ proj,
          const float* __restrict__ center, __nv_bfloat16* __restrict__ fp, float* __restrict__ rq,
          uint32_t B, uint32_t n, uint32_t d, uint32_t k, uint32_t L, uint32_t Jmax,
          const float* __restrict__ pooled, uint32_t ld) {
  griddep_sync();
  extern __shared__ float sm[];
  float* p = sm;                               // [G][d]
  float* g = p + (size_t)PROJ_G * d;           // [G][k]            (only with projection)
  float* part = g + (size_t)PROJ_G * k;        // [slices][G][k]    (only with projection)
  __shared__ float red[PROJ_THREADS / 32];
  const uint32_t b0 = blockIdx.x * PROJ_G;
  const float fn = (float)n;
  const int grp = threadIdx.x / PROJ_TPS;      // sequence served in the element-wise phases
  const uint32_t gt = threadIdx.x % PROJ_TPS;
  const uint32_t bq = b0 + grp;

  {
    // pool blocks whose span overlaps rows [b*n, (b+1)*n), in block order
    float* pg = p + (size_t)grp * d;
    if (bq < B && pooled) {
      // the position means were taken elsewhere (while the rows were written)
      for (uint32_t i = gt; i < d; i += PROJ_TPS) {
        float v = pooled[(size_t)bq * ld + i];
        if (center) v -= center[i];
        pg[i] = v;
      }
    } else if (bq < B) {
      const unsigned long long first = (unsigned long long)bq * n, last = first + n - 1;
      const uint32_t c_lo = (uint32_t)(first / L), c_hi = (uint32_t)(last / L);
      const uint32_t j_lo = bq - (uint32_t)(((unsigned long long)c_lo * L) / n);
      for (uint32_t i = gt; i < d; i += PROJ_TPS) {
        // the first block may have touched earlier sequences (index j_lo); later blocks start inside bq
        float v = partial[((size_t)c_lo * Jmax + j_lo) * d + i];
        for (uint32_t c = c_lo + 1; c <= c_hi; ++c) v += partial[(size_t)c * Jmax * d + i];
        v = v / fn;
        if (center) v -= center[i];
        pg[i] = v;
      }
    } else {
      for (uint32_t i = gt; i < d; i += PROJ_TPS) pg[i] = 0.f;
    }
  }
  __syncthreads();

  if (proj) {
    const uint32_t ncg = k >> 3;                                   // groups of 8 columns
    const uint32_t slices = ncg >= blockDim.x ? 1u : blockDim.x / ncg;
    const uint4* P4 = reinterpret_cast<const uint4*>(proj);
    for (uint32_t cg0 = 0; cg0 < ncg; cg0 += blockDim.x) {         // one trip unless k > 8 * threads
      const uint32_t cg = cg0 + (ncg >= blockDim.x ? threadIdx.x : threadIdx.x % ncg);
      const uint32_t sl = ncg >= blockDim.x ? 0u : threadIdx.x / ncg;
      if (cg < ncg && sl < slices) {
        float acc[PROJ_G][8];
#pragma unroll
        for (int gi = 0; gi < PROJ_G; ++gi)
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[gi][e] = 0.f;
        auto fma_row = [&](const uint4& w, uint32_t i) {
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
          float x[PROJ_G];
#pragma unroll
          for (int gi = 0; gi < PROJ_G; ++gi) x[gi] = p[gi * d + i];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float w0 = __uint_as_float(ww[u] << 16), w1 = __uint_as_float(ww[u] & 0xFFFF0000u);
#pragma unroll
            for (int gi = 0; gi < PROJ_G; ++gi) {
              acc[gi][2 * u]     = fmaf(x[gi], w0, acc[gi][2 * u]);
              acc[gi][2 * u + 1] = fmaf(x[gi], w1, acc[gi][2 * u + 1]);
            }
          }
        };
        constexpr int INFL = 8;                                    // rows in flight
        // This thread's rows are sl, sl + slices, ...  Every block reads the same matrix, so each block
        // starts at a different one of them (and wraps): the blocks then ask for different lines at any
        // moment instead of all hitting one L2 line together.
        const uint32_t nrow = sl < d ? (d - sl + slices - 1) / slices : 0u;
        const uint32_t rot = nrow ? (blockIdx.x * 5u) % nrow : 0u;
        auto row_of = [&](uint32_t t) { uint32_t tt = t + rot; if (tt >= nrow) tt -= nrow; return sl + tt * slices; };
        uint32_t t = 0;
        for (; t + INFL <= nrow; t += INFL) {
          uint4 w[INFL];
          uint32_t ri[INFL];
#pragma unroll
          for (int u = 0; u < INFL; ++u) { ri[u] = row_of(t + u); w[u] = ld_nc16(P4 + (size_t)ri[u] * ncg + cg); }
#pragma unroll
          for (int u = 0; u < INFL; ++u) fma_row(w[u], ri[u]);
        }
        for (; t < nrow; ++t) { const uint32_t i = row_of(t); fma_row(ld_nc16(P4 + (size_t)i * ncg + cg), i); }
#pragma unroll
        for (int gi = 0; gi < PROJ_G; ++gi)
#pragma unroll
          for (int e = 0; e < 8; ++e) part[((size_t)sl * PROJ_G + gi) * k + cg * 8 + e] = acc[gi][e];
      }
    }
    __syncthreads();
    for (uint32_t idx = threadIdx.x; idx < PROJ_G * k; idx += blockDim.x) {
      float v = 0.f;
      for (uint32_t sl = 0; sl < slices; ++sl) v += part[(size_t)sl * PROJ_G * k + idx];
      g[idx] = v;
    }
    __syncthreads();
  } else {
    g = p;                                      // identity: k == d
  }

  // unit length + rounding: the G sequences side by side, 128 threads each
  const float* gv = g + (size_t)grp * k;
  float ss = 0.f;
  for (uint32_t c = gt; c < k; c += PROJ_TPS) ss = fmaf(gv[c], gv[c], ss);
  ss = group_sum(ss, red, grp);
  const float nrm = sqrtf(ss);
  const bool ok = isfinite(ss) && nrm >= 1e-20f;
  float qs = 0.f;
  if (bq < B) {
    __nv_bfloat16* dst = fp + (size_t)bq * k;
    for (uint32_t c = gt; c < k; c += PROJ_TPS) {
      __nv_bfloat16 q = __float2bfloat16_rn(ok ? gv[c] / nrm : 0.f);
      dst[c] = q;
      const float qf = __bfloat162float(q);
      qs = fmaf(qf, qf, qs);
    }
  }
  qs = group_sum(qs, red, grp);
  if (gt == 0 && bq < B) rq[bq] = (ok && qs > 0.f) ? 1.0f / sqrtf(qs) : 0.f;
}

// rq[b] = 1/||fp[b]|| for fingerprints supplied by the caller; one warp per row.
__global__ void k_rownorm(const __nv_bfloat16* __restrict__ fp, uint32_t B, uint32_t k, float* __restrict__ rq) {
  griddep_sync();
  const uint32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const uint32_t lane = threadIdx.x & 31;
  if (row >= B) return;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(fp + (size_t)row * k);
  float ss = 0.f;
  for (uint32_t c = lane; c < (k >> 1); c += 32) {
    const uint32_t w = src[c];
    const float a = __uint_as_float(w << 16), b = __uint_as_float(w & 0xFFFF0000u);
    ss = fmaf(a, a, ss);
    ss = fmaf(b, b, ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  if (lane == 0) {
    const float nrm = sqrtf(ss);
    rq[row] = (isfinite(ss) && nrm >= 1e-20f) ? 1.0f / nrm : 0.f;
  }
}

// ---------------------------------------------------------------------------
size_t project_smem_bytes(uint32_t d, uint32_t k, bool has_proj) {
  const uint32_t ncg = k / 8;
  const uint32_t slices = (has_proj && ncg < (uint32_t)PROJ_THREADS) ? PROJ_THREADS / ncg : 1;
  return ((size_t)PROJ_G * d + (has_proj ? (size_t)PROJ_G * k + (size_t)slices * PROJ_G * k : 0)) * sizeof(float);
}

cudaError_t setup_fingerprint_kernels() {
  cudaError_t e = cudaFuncSetAttribute(k_project, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_pool<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_pool<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
  return e;
}

// Launch shape of the pooling pass.  The scratch it needs is grid * Jmax * d floats, which never exceeds
// (B + 3 * POOL_MAX_GRID) * d.
PoolPlan pool_plan(uint32_t B, uint32_t n, uint32_t d, bool bf16, int sm_count) {
  PoolPlan P;
  P.V = bf16 ? d / 8 : d / 4;
  P.R = 512 / P.V; if (P.R < 1) P.R = 1;
  if (P.R > n) P.R = n;
  P.cons_threads = (P.V * P.R + 31) / 32 * 32;
  P.threads = P.cons_threads + 32;                                    // + the producer's warp
  const uint32_t row_bytes = P.V * 16;
  // a stage holds a whole number of passes of R rows, about 16 KB; the ring about 160 KB
  uint32_t passes = 16384 / (P.R * row_bytes); if (passes < 1) passes = 1;
  P.stage_rows = P.R * passes;
  const uint32_t stage_bytes = P.stage_rows * row_bytes;
  P.stages = (160 * 1024) / stage_bytes;
  if (P.stages > 16) P.stages = 16;
  if (P.stages < 2) P.stages = 2;
  const unsigned long long rows = (unsigned long long)B * n;
  unsigned long long grid = (unsigned long long)sm_count;              // one block per SM
  if (grid > POOL_MAX_GRID) grid = POOL_MAX_GRID;
  const unsigned long long min_rows = 2ull * P.stage_rows;             // keep spans long enough to pipeline
  if (grid * min_rows > rows) grid = (rows + min_rows - 1) / min_rows;
  if (grid < 1) grid = 1;
  P.L = (uint32_t)((rows + grid - 1) / grid);
  P.grid = (uint32_t)((rows + P.L - 1) / P.L);
  P.Jmax = (P.L + n - 1) / n + 1;
  P.smem = (size_t)P.stages * stage_bytes + (size_t)P.R * d * sizeof(float) + 16 * P.stages + 16;
  return P;
}

static cudaError_t launch_pool(const PoolPlan& P, bool bf16, const void* h_in, float* partial, uint32_t* status,
                               uint32_t B, uint32_t n, uint32_t d, cudaStream_t st) {
  return launch_k(bf16 ? k_pool<true> : k_pool<false>, dim3(P.grid), dim3(P.threads), P.smem, st,
                  (const uint4*)h_in, partial, status, B, n, d, P.V, P.R, P.L, P.Jmax, P.stage_rows, P.stages,
                  P.cons_threads);
}

static cudaError_t launch_project(const PoolPlan& P, const float* partial, const __nv_bfloat16* proj,
                                  const float* center, __nv_bfloat16* fp, float* rq,
                                  uint32_t B, uint32_t n, uint32_t d, uint32_t k, cudaStream_t st) {
  return launch_k(k_project, dim3((B + PROJ_G - 1) / PROJ_G), dim3(PROJ_THREADS),
                  project_smem_bytes(d, k, proj != nullptr), st, partial, proj, center, fp, rq, B, n, d, k, P.L, P.Jmax,
                  (const float*)nullptr, 0u);
}

cudaError_t launch_fingerprint(llmcache_bank* bk, const void* h_in, uint32_t B,
                               __nv_bfloat16* fp, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const bool bf16 = D.hidden_dtype == LLMCACHE_BF16;
  const PoolPlan P = pool_plan(B, D.seq_len, D.d_model, bf16, bk->sm_count);
  cudaError_t e;
  {
    ProfScope prof(bk, LLMCACHE_K_POOL, st);
    e = launch_pool(P, bf16, h_in, bk->a.pool_partial, bk->a.status, B, D.seq_len, D.d_model, st);
  }
  if (e != cudaSuccess) return e;
  ProfScope prof(bk, LLMCACHE_K_PROJECT, st);
  return launch_project(P, bk->a.pool_partial, bk->a.proj, bk->a.center, fp, rq, B, D.seq_len, D.d_model, D.fp_dim, st);
}

// Step 1a alone: position means of h_in -> pooled[b * ld + c].
cudaError_t launch_pool_only(llmcache_bank* bk, const void* h_in, uint32_t B, float* pooled, uint32_t ld, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const bool bf16 = D.hidden_dtype == LLMCACHE_BF16;
  const PoolPlan P = pool_plan(B, D.seq_len, D.d_model, bf16, bk->sm_count);
  cudaError_t e;
  {
    ProfScope prof(bk, LLMCACHE_K_POOL, st);
    e = launch_pool(P, bf16, h_in, bk->a.pool_partial, bk->a.status, B, D.seq_len, D.d_model, st);
  }
  if (e != cudaSuccess) return e;
  return launch_pool_finish_plain(bk, P, B, pooled, ld, st);
}

// Step 1b alone: fingerprints from given position means pooled[b * ld + c], c < d.
cudaError_t launch_fingerprint_pooled(llmcache_bank* bk, const float* pooled, uint32_t ld, uint32_t B,
                                      __nv_bfloat16* fp, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  ProfScope prof(bk, LLMCACHE_K_PROJECT, st);
  return launch_k(k_project, dim3((B + PROJ_G - 1) / PROJ_G), dim3(PROJ_THREADS),
                  project_smem_bytes(D.d_model, D.fp_dim, bk->a.proj != nullptr), st, (const float*)nullptr,
                  (const __nv_bfloat16*)bk->a.proj, (const float*)bk->a.center, fp, rq, B, D.seq_len, D.d_model,
                  D.fp_dim, 1u, 1u, pooled, ld);
}

cudaError_t launch_rownorm(llmcache_bank* bk, const __nv_bfloat16* fp, uint32_t B, uint32_t k, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  ProfScope prof(bk, LLMCACHE_K_ROWNORM, st);
  return launch_k(k_rownorm, dim3((B + 7) / 8), dim3(256), 0, st, fp, B, k, rq);
}

}  // namespace llmc

// ---------------------------------------------------------------------------
// Fingerprint without any allocation: the pooled partial sums go to a fixed
// array that is part of the loaded library image instead of a bank's scratch.
// ---------------------------------------------------------------------------
#include <mutex>
#include <cstdio>

namespace {

// Partial sums of the pooling pass, [B, splits, d] floats.  8 MiB per GPU that loads the library.
static __device__ __align__(256) float g_fp_static_scratch[LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS];
// Set by the pooling kernel if one of its bounded waits ever expired (stays zero otherwise).
static __device__ uint32_t g_fp_static_status;

constexpr int STATIC_MAX_DEVICES = 64;
struct StaticDev { bool ready = false; float* scratch = nullptr; uint32_t* status = nullptr; int sm_count = 0; };
StaticDev g_static_dev[STATIC_MAX_DEVICES];
std::mutex g_static_mu;
thread_local char g_static_err[192] = "";

// Once per device, with that device current: resolve the device address of the array (its name is
// only a host-side handle) and raise the projection kernel's shared-memory limit.
cudaError_t static_setup(int dev, StaticDev** out) {
  std::lock_guard<std::mutex> lock(g_static_mu);
  StaticDev& sd = g_static_dev[dev];
  if (!sd.ready) {
    float* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_fp_static_scratch);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorInvalidSymbol;
    uint32_t* sptr = nullptr;
    e = cudaGetSymbolAddress((void**)&sptr, g_fp_static_status);
    if (e != cudaSuccess) return e;
    if (!sptr) return cudaErrorInvalidSymbol;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = llmc::setup_fingerprint_kernels();
    if (e != cudaSuccess) return e;
    sd.scratch = ptr;
    sd.status = sptr;
    sd.sm_count = sms;
    sd.ready = true;
  }
  *out = &sd;
  return cudaSuccess;
}

}  // namespace

extern "C" const char* llmcache_fingerprint_static_error(void) { return g_static_err; }

extern "C" int llmcache_fingerprint_static(const void* h_in, uint32_t hidden_dtype, uint32_t B, uint32_t seq_len,
                                           uint32_t d_model, uint32_t fp_dim, const void* proj,
                                           const float* center, void* fp, float* rq, void* stream) {
  using namespace llmc;
  g_static_err[0] = 0;
  auto fail = [&](int rc, const char* msg) { std::snprintf(g_static_err, sizeof(g_static_err), "%s", msg); return rc; };
  if (hidden_dtype != LLMCACHE_F32 && hidden_dtype != LLMCACHE_BF16) return fail(LLMCACHE_ERR_ARG, "unknown hidden_dtype");
  if (B && (!h_in || !fp || !rq)) return fail(LLMCACHE_ERR_ARG, "null input or output pointer");
  if (((uintptr_t)h_in | (uintptr_t)fp | (uintptr_t)proj | (uintptr_t)center) & 15u)
    return fail(LLMCACHE_ERR_ARG, "pointers must be 16-byte aligned");
  const bool bf16 = hidden_dtype == LLMCACHE_BF16;
  const uint32_t d = d_model, n = seq_len, k = fp_dim;
  if (n == 0 || d == 0 || d % 8 != 0 || d > (bf16 ? 7680u : 3840u)) return fail(LLMCACHE_ERR_SHAPE, "d_model not supported");
  if (k == 0 || k % 64 != 0 || k > 2048 || (!proj && k != d)) return fail(LLMCACHE_ERR_SHAPE, "fp_dim not supported");
  if (project_smem_bytes(d, k, proj != nullptr) > 200 * 1024) return fail(LLMCACHE_ERR_UNSUPPORTED, "d_model + fp_dim too large");
  if (B == 0) return LLMCACHE_OK;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
    cudaGetLastError();
    return fail(LLMCACHE_ERR_CUDA, "no current CUDA device");
  }
  StaticDev* sd = nullptr;
  cudaError_t e = static_setup(dev, &sd);
  if (e != cudaSuccess) { cudaGetLastError(); return fail(LLMCACHE_ERR_CUDA, cudaGetErrorString(e)); }

  const PoolPlan P = pool_plan(B, n, d, bf16, sd->sm_count);
  const unsigned long long need = (unsigned long long)P.grid * P.Jmax * d;
  if (need > (unsigned long long)LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS) {
    std::snprintf(g_static_err, sizeof(g_static_err),
                  "batch too large for the fixed scratch: %llu floats of partial sums needed, limit %llu",
                  need, (unsigned long long)LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS);
    return LLMCACHE_ERR_SHAPE;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // every partial sum that the second kernel reads is written by the first one in this call, so
  // nothing in the shared array has to start at zero
  e = launch_pool(P, bf16, h_in, sd->scratch, sd->status, B, n, d, st);
  if (e == cudaSuccess)
    e = launch_project(P, sd->scratch, (const __nv_bfloat16*)proj, center, (__nv_bfloat16*)fp, rq, B, n, d, k, st);
  if (e != cudaSuccess) return fail(LLMCACHE_ERR_CUDA, cudaGetErrorString(e));
  return LLMCACHE_OK;
}
