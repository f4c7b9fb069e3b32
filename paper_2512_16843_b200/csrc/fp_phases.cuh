// Device routines of the fingerprint (Sec. IV-B), written as block-level phases:
//   pool_phase      position sums of a span of rows ("Embedding Aggregation")
//   project_*       centred means times the projection matrix ("Dimensionality Reduction")
//   finish_group    unit length, bf16 rounding, inverse norm of the rounded vector
//   normalise_seq   the same without a projection matrix (k == d)
// Every wait is bounded; a wait that expires sets the status word and the block's abort flag, after
// which all later waits of the block return at once.
#pragma once
#include "llmcache_internal.cuh"
#include "ptx.cuh"

namespace llmc {

// The first SMEM_HEAD bytes of dynamic shared memory hold the mbarriers and flags at fixed places; the data
// areas that follow start on a 1024-byte boundary (what the 128-byte swizzle of the TMA boxes needs).
constexpr uint32_t SMEM_HEAD = 1024;
constexpr uint32_t HEAD_POOL_BARS = 0;       // full[16], empty[16]
constexpr uint32_t HEAD_PROJ_BARS = 256;     // full[8], empty[8]
constexpr uint32_t HEAD_FLAGS = 400;         // u32 [0] abort, [1] consumers' copy of it
constexpr uint32_t HEAD_SEQ_INFO = 704;      // 8 x {c_lo, c_hi, j_lo} of the projection's group

__device__ __forceinline__ volatile uint32_t* head_flags(uint8_t* sm) {
  return reinterpret_cast<volatile uint32_t*>(sm + HEAD_FLAGS);
}

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
// Threads [0, cons_threads) consume, thread cons_threads produces.  Called by all threads of the block.
// ---------------------------------------------------------------------------
// early: the input is not written by the grid that precedes this one in the stream (the caller says so), so the
// producer may start streaming it before that grid has finished; the consumers still wait before they write.
struct PoolShape { uint32_t B, n, d, V, R, L, Jmax, stage_rows, stages, cons_threads, early; };

template <bool BF16>
__device__ __forceinline__ void pool_phase(uint8_t* sm, const uint4* __restrict__ h, float* __restrict__ partial,
                                           uint32_t* __restrict__ status, const PoolShape& S) {
  constexpr int E = BF16 ? 8 : 4;
  const uint32_t n = S.n, d = S.d, V = S.V, R = S.R, stages = S.stages, stage_rows = S.stage_rows;
  const uint32_t cons_threads = S.cons_threads;
  const uint32_t row_bytes = V * 16;
  const uint32_t stage_bytes = stage_rows * row_bytes;
  const uint32_t ring = smem_u32(sm + SMEM_HEAD);
  float* red = reinterpret_cast<float*>(sm + SMEM_HEAD + (size_t)stages * stage_bytes);      // [R][d]
  const uint32_t bar0 = smem_u32(sm + HEAD_POOL_BARS);
  volatile uint32_t* flags = head_flags(sm);
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (16 + s); };
  const unsigned long long lim = wait_limit(status);

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), cons_threads / 32); }
    flags[0] = 0; flags[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const unsigned long long total = (unsigned long long)S.B * n;
  unsigned long long r = (unsigned long long)blockIdx.x * S.L;
  unsigned long long r1 = r + S.L;
  if (r1 > total) r1 = total;
  if (r > total) r = total;
  uint32_t b = (uint32_t)(r / n);
  uint32_t it = 0;

  if (threadIdx.x >= cons_threads) {
    // ---------------------------------------------------------------- producer (one thread)
    if (S.early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == cons_threads && !producer_idle(status)) {
      bool ok = true;
      while (r < r1 && ok) {
        unsigned long long seg_end = (unsigned long long)(b + 1) * n;
        if (seg_end > r1) seg_end = r1;
        while (r < seg_end) {
          const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
          const uint32_t s = it % stages, ph = (it / stages) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, flags, lim)) { ok = false; break; }
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
        // copies that were started must land before the block's shared memory is reused or released
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
    if (S.early) griddep_sync();                       // nothing is written to global memory before this
    const bool active = threadIdx.x < V * R;
    const uint32_t col = threadIdx.x % V, rg = threadIdx.x / V;
    float* out = partial + (size_t)blockIdx.x * S.Jmax * d;
    while (r < r1) {
      unsigned long long seg_end = (unsigned long long)(b + 1) * n;
      if (seg_end > r1) seg_end = r1;
      float acc[E];
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] = 0.f;
      while (r < seg_end) {
        const uint32_t rows = (uint32_t)min((unsigned long long)stage_rows, seg_end - r);
        const uint32_t s = it % stages, ph = (it / stages) & 1u;
        if (!mbar_wait(full_bar(s), ph, flags, lim)) { flags[0] = 1; atomicExch(status, 1u); }
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
// Position means of sequence bq, column i, centred: either given (pooled) or the sum of the pooling
// pass's partial vectors of the blocks whose span overlaps rows [bq*n, (bq+1)*n), in block order.
// The sums were written by the grid before this one; they are read past L1.
// ---------------------------------------------------------------------------
struct MeanSrc { const float* partial; const float* pooled; const float* center; uint32_t ld, n, d, L, Jmax; };

// Which pooling blocks hold rows of sequence bq: blocks c_lo..c_hi; in block c_lo it is the j_lo-th sequence touched
// (that block may have started in an earlier sequence), in the later blocks the first.
struct SeqBlocks { uint32_t c_lo, c_hi, j_lo; };
__device__ __forceinline__ SeqBlocks seq_blocks(const MeanSrc& m, uint32_t bq) {
  SeqBlocks q{0u, 0u, 0u};
  if (!m.pooled) {
    const unsigned long long first = (unsigned long long)bq * m.n, last = first + m.n - 1;
    q.c_lo = (uint32_t)(first / m.L);
    q.c_hi = (uint32_t)(last / m.L);
    q.j_lo = bq - (uint32_t)(((unsigned long long)q.c_lo * m.L) / m.n);
  }
  return q;
}
__device__ __forceinline__ float centred_mean(const MeanSrc& m, const SeqBlocks& q, uint32_t bq, uint32_t i) {
  float v;
  if (m.pooled) {
    v = __ldcg(m.pooled + (size_t)bq * m.ld + i);
  } else {
    v = __ldcg(m.partial + ((size_t)q.c_lo * m.Jmax + q.j_lo) * m.d + i);
    for (uint32_t c = q.c_lo + 1; c <= q.c_hi; ++c) v += __ldcg(m.partial + (size_t)c * m.Jmax * m.d + i);
    v = v / (float)m.n;
  }
  if (m.center) v -= m.center[i];
  return v;
}

// ---------------------------------------------------------------------------
// Project.  A work item is (PROJ_G = 8 sequences starting at b0) x (rows [r0, r0 + nrows) of P).
// The product runs on the tensor cores (mma.sync m16n8k16, bf16 inputs, fp32 accumulate).  An fp32 mean is
// the exact sum of three bf16 numbers (head, middle, tail: 3 x 8 significant bits), so the A operand
// carries the 8 sequences' centred means as three bf16 rows each: head in rows 0..7 and middle in rows
// 8..15 of one mma, tail in rows 0..7 of a second mma into the same accumulator; rows g and g + 8 of the
// accumulator are added at the end.  Nothing of the fp32 means is lost; only the order of the sums
// differs from a plain fp32 dot product.  The item's rows of P are streamed once through a ring of
// shared-memory stages by TMA (issued by thread PROJ_CONS): a stage is k / 64 boxes of stage_rows x 64
// columns with the 128-byte swizzle, so that ldmatrix finds its eight rows in different banks; rows beyond
// the end of P arrive as zeros.  Warp w of the PROJ_CONS / 32 consumer warps owns the output columns
// [w * NT * 8, (w + 1) * NT * 8) over all the item's rows, so nothing has to be combined across warps.
// Shared memory after the head: ring | A [24][a_rows] bf16 (the item's rows are taken a_rows at a time).
// The ring's memory is reused for the group's [8][k] result once the item's rows are consumed.
// ---------------------------------------------------------------------------
constexpr int PROJ_G = 8;                           // sequences per item
constexpr int PROJ_CONS = 512;                      // consumer threads
constexpr int PROJ_THREADS = PROJ_CONS + 32;        // + the producer's warp
constexpr uint32_t PROJ_KSTEP = 16;                 // rows of P per mma

struct ProjShape {
  uint32_t k, stage_rows, stages, ring_bytes;      // stage_rows: a multiple of 16 (rows of the TMA box); ring_bytes >= stages * stage bytes
  uint32_t a_rows;                                  // rows of P per refill of A: a multiple of stage_rows
  uint32_t a_stride;                                // bytes between the rows of A (a multiple of 16, = 16 mod 128)
};
struct ProjSmem {
  uint32_t ring, bar0, a_mat;
  float* part;                                      // the ring's memory seen as floats
  uint8_t* a_ptr;
  uint8_t* seq_info;                                // PROJ_G x SeqBlocks
  volatile uint32_t* flags;
  __device__ __forceinline__ uint32_t full_bar(uint32_t s) const { return bar0 + 8 * s; }
  __device__ __forceinline__ uint32_t empty_bar(uint32_t s) const { return bar0 + 8 * (8 + s); }
};

__device__ __forceinline__ ProjSmem proj_smem(uint8_t* sm, const ProjShape& S) {
  ProjSmem m;
  m.ring = smem_u32(sm + SMEM_HEAD);
  m.part = reinterpret_cast<float*>(sm + SMEM_HEAD);
  m.a_ptr = sm + SMEM_HEAD + S.ring_bytes;
  m.a_mat = smem_u32(m.a_ptr);
  m.bar0 = smem_u32(sm + HEAD_PROJ_BARS);
  m.seq_info = sm + HEAD_SEQ_INFO;
  m.flags = head_flags(sm);
  return m;
}

// One thread, before any other use; followed by a block-level barrier.
__device__ __forceinline__ void proj_init(const ProjSmem& m, const ProjShape& S, bool clear_flags) {
  for (uint32_t s = 0; s < S.stages; ++s) { mbar_init(m.full_bar(s), 1); mbar_init(m.empty_bar(s), PROJ_CONS / 32); }
  if (clear_flags) { m.flags[0] = 0; m.flags[1] = 0; }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Order in which the stages of one refill of A (rows [c0, c0 + crows) of the item) are taken: rotated by an
// amount that differs from item to item.  All items read the same matrix at about the same time; without the
// rotation every SM would ask the same L2 slice for the same lines at the same moment.
__device__ __forceinline__ uint32_t proj_stage_at(uint32_t j, uint32_t nst, uint32_t rot) {
  const uint32_t js = j + rot % nst;
  return js >= nst ? js - nst : js;
}

// Producer thread: the rows [r0, r0 + nrows) of P for one item, whole stages (rows past the item's end are
// loaded too; the A operand is zero there).  `it` counts stages over all items of the block.
__device__ __forceinline__ bool proj_produce(const ProjSmem& m, const ProjShape& S, const CUtensorMap* map,
                                             uint32_t r0, uint32_t nrows, uint32_t rot, uint32_t& it,
                                             unsigned long long lim) {
  const uint32_t box_bytes = S.stage_rows * 128, stage_bytes = (S.k / 64) * box_bytes;
  for (uint32_t c0 = 0; c0 < nrows; c0 += S.a_rows) {
    const uint32_t crows = min(S.a_rows, nrows - c0);
    const uint32_t nst = (crows + S.stage_rows - 1) / S.stage_rows;
    for (uint32_t j = 0; j < nst; ++j, ++it) {
      const uint32_t ra = c0 + proj_stage_at(j, nst, rot) * S.stage_rows;
      const uint32_t s = it % S.stages, ph = (it / S.stages) & 1u;
      if (!mbar_wait(m.empty_bar(s), ph ^ 1u, m.flags, lim)) return false;
      mbar_expect_tx(m.full_bar(s), stage_bytes);
      for (uint32_t b = 0; b < S.k / 64; ++b)
        tma_load_2d(m.ring + s * stage_bytes + b * box_bytes, map, (int)(b * 64), (int)(r0 + ra), m.full_bar(s));
    }
  }
  return true;
}
// After a failed wait: copies that were started must land before the ring is reused or released.
__device__ __forceinline__ void proj_drain(const ProjSmem& m, const ProjShape& S, uint32_t it, uint32_t* status) {
  m.flags[0] = 1;
  atomicExch(status, 1u);
  const uint32_t back = it < S.stages ? it : S.stages;
  volatile uint32_t never = 0;
  for (uint32_t i = 0; i < back; ++i) {
    const uint32_t itx = it - 1 - i;
    mbar_wait(m.full_bar(itx % S.stages), (itx / S.stages) & 1u, &never, 200000000ull);
  }
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t (&r)[2]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];"
               : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// Consumer threads, before proj_consume: where each of the item's sequences lies in the pooling pass's partial
// sums.  Needs nothing that another grid writes, so it can run before the grid dependency is resolved.
__device__ __forceinline__ void proj_prepare(const ProjSmem& m, const MeanSrc& src, uint32_t b0) {
  SeqBlocks* sq = reinterpret_cast<SeqBlocks*>(m.seq_info);
  if (threadIdx.x < PROJ_G) sq[threadIdx.x] = seq_blocks(src, b0 + threadIdx.x);
  asm volatile("bar.sync 1, %0;" ::"n"(PROJ_CONS) : "memory");
}

// Consumer threads (all PROJ_CONS of them): one item.  On return thread (warp w, lane l) holds, for
// t < NT, vals[2t] and vals[2t + 1]: the sums over the item's rows for sequence b0 + l / 4 and columns
// (w * NT + t) * 8 + (l % 4) * 2 and the next one (columns >= k: zero).
template <int NT>
__device__ __forceinline__ void proj_consume(const ProjSmem& m, const ProjShape& S, const MeanSrc& src,
                                             uint32_t B, uint32_t b0, uint32_t r0, uint32_t nrows, uint32_t rot,
                                             uint32_t& it, uint32_t* __restrict__ status, float (&vals)[2 * NT]) {
  const uint32_t k = S.k, box_bytes = S.stage_rows * 128, stage_bytes = (k / 64) * box_bytes;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned long long lim = wait_limit(status);
  const SeqBlocks* sq = reinterpret_cast<const SeqBlocks*>(m.seq_info);
  uint32_t more = 0;                                                 // most pooling blocks per sequence, less one
#pragma unroll
  for (int g = 0; g < PROJ_G; ++g) more = max(more, sq[g].c_hi - sq[g].c_lo);
  float acc[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;
  const uint32_t col0 = warp * NT * 8;                               // first column of this warp
  // ldmatrix row addresses: A matrices (rows 0-7 | 8-15) x (k 0-7 | 8-15), tail matrices (rows 16-23) x (k 0-7 | 8-15);
  // B matrices: rows kk + (lane % 16) of one 8-column tile = one 16-byte chunk of a 128-byte box row, stored at
  // chunk index (chunk ^ (row % 8)) by the swizzle (stages and boxes start on 1024-byte boundaries and kk is a
  // multiple of 16, so row % 8 = lane % 8)
  const uint32_t a_lane = m.a_mat + (lane & 15u) * S.a_stride + (lane >> 4) * 16;
  const uint32_t t_lane = m.a_mat + (16u + (lane & 7u)) * S.a_stride + ((lane >> 3) & 1u) * 16;
  const uint32_t b_row = (lane & 15u) * 128, b_xor = lane & 7u;
  for (uint32_t c0 = 0; c0 < nrows; c0 += S.a_rows) {
    // A: head, middle and tail of the centred means of rows [c0, c0 + crows), padded to a multiple of 16 rows with zeros
    const uint32_t crows = min(S.a_rows, nrows - c0);
    const uint32_t cr16 = (crows + PROJ_KSTEP - 1) / PROJ_KSTEP * PROJ_KSTEP;
    if (c0) asm volatile("bar.sync 1, %0;" ::"n"(PROJ_CONS) : "memory");   // everyone is done with the previous rows of A
    // The threads form `sets` groups of cr16 (or all take every row when there are more rows than threads);
    // set q serves sequences q * GS .. q * GS + GS - 1 of the item.  All loads of a round are independent, so
    // a round costs one L2 round trip; nearly every sequence lies in at most two pooling blocks.
    const uint32_t sets = cr16 * 8 <= PROJ_CONS ? 8u : cr16 * 4 <= PROJ_CONS ? 4u : cr16 * 2 <= PROJ_CONS ? 2u : 1u;
    const uint32_t GS = PROJ_G / sets, set = threadIdx.x / cr16, g0 = set * GS;
    for (uint32_t il = sets > 1 ? threadIdx.x - set * cr16 : threadIdx.x; il < cr16 && set < sets; il += PROJ_CONS) {
      const uint32_t i = r0 + c0 + il;
      const bool live = il < crows;
      float v[PROJ_G];
      const float mu = (live && src.center) ? src.center[i] : 0.f;
      if (src.pooled) {
#pragma unroll
        for (int u = 0; u < PROJ_G; ++u)
          v[u] = (u < GS && live && b0 + g0 + u < B) ? __ldcg(src.pooled + (size_t)(b0 + g0 + u) * src.ld + i) : 0.f;
      } else {
        float w[PROJ_G];
#pragma unroll
        for (int u = 0; u < PROJ_G; ++u) {
          const bool on = u < GS && live && b0 + g0 + u < B;
          const SeqBlocks q = sq[(g0 + u) & (PROJ_G - 1)];
          v[u] = on ? __ldcg(src.partial + ((size_t)q.c_lo * src.Jmax + q.j_lo) * src.d + i) : 0.f;
          w[u] = (on && q.c_lo < q.c_hi) ? __ldcg(src.partial + (size_t)(q.c_lo + 1) * src.Jmax * src.d + i) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < PROJ_G; ++u) v[u] += w[u];
        for (uint32_t e = 2; e <= more; ++e) {
#pragma unroll
          for (int u = 0; u < PROJ_G; ++u) {
            const SeqBlocks q = sq[(g0 + u) & (PROJ_G - 1)];
            w[u] = (u < GS && live && b0 + g0 + u < B && q.c_lo + e <= q.c_hi)
                       ? __ldcg(src.partial + (size_t)(q.c_lo + e) * src.Jmax * src.d + i) : 0.f;
          }
#pragma unroll
          for (int u = 0; u < PROJ_G; ++u) v[u] += w[u];
        }
#pragma unroll
        for (int u = 0; u < PROJ_G; ++u) v[u] = v[u] / (float)src.n;
      }
#pragma unroll
      for (int u = 0; u < PROJ_G; ++u) {
        if (u < GS) {
          const uint32_t g = g0 + u;
          const float x = (live && b0 + g < B) ? v[u] - mu : 0.f;
          const __nv_bfloat16 hi = __float2bfloat16_rn(x);
          const float r1 = x - __bfloat162float(hi);                 // exact
          const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
          const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
          *reinterpret_cast<__nv_bfloat16*>(m.a_ptr + (size_t)g * S.a_stride + il * 2) = hi;
          *reinterpret_cast<__nv_bfloat16*>(m.a_ptr + (size_t)(g + PROJ_G) * S.a_stride + il * 2) = mid;
          *reinterpret_cast<__nv_bfloat16*>(m.a_ptr + (size_t)(g + 2 * PROJ_G) * S.a_stride + il * 2) = lo;
        }
      }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(PROJ_CONS) : "memory");
    const uint32_t nst = (crows + S.stage_rows - 1) / S.stage_rows;
    for (uint32_t j = 0; j < nst; ++j, ++it) {
      const uint32_t ra = proj_stage_at(j, nst, rot) * S.stage_rows;
      const uint32_t rows = min(S.stage_rows, crows - ra);
      const uint32_t s = it % S.stages, ph = (it / S.stages) & 1u;
      if (!mbar_wait(m.full_bar(s), ph, m.flags, lim)) { m.flags[0] = 1; atomicExch(status, 1u); }
      if (col0 < k) {
        const uint32_t stage = m.ring + s * stage_bytes;
        for (uint32_t kk = 0; kk < rows; kk += PROJ_KSTEP) {
          uint32_t a[4], tl[2];
          ldmatrix_x4(a_lane + (ra + kk) * 2, a);
          ldmatrix_x2(t_lane + (ra + kk) * 2, tl);
          const uint32_t a2[4] = {tl[0], 0u, tl[1], 0u};
#pragma unroll
          for (int t = 0; t < NT; ++t) {
            const uint32_t col = col0 + t * 8;
            if (col < k) {
              uint32_t b[2];
              ldmatrix_x2_trans(stage + (col >> 6) * box_bytes + kk * 128 + b_row + ((((col >> 3) & 7u) ^ b_xor) << 4), b);
              mma_bf16_16816(acc[t], a, b);
              mma_bf16_16816(acc[t], a2, b);
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(m.empty_bar(s));
    }
  }
  // head + tail (rows g) and middle (rows g + 8) of the accumulator sit in the same thread
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    vals[2 * t] = acc[t][0] + acc[t][2];
    vals[2 * t + 1] = acc[t][1] + acc[t][3];
  }
}

// Index into an item's [PROJ_G][k] result of vals[2t + e] held by this thread, or 0xFFFFFFFF if beyond k.
template <int NT>
__device__ __forceinline__ uint32_t proj_val_index(uint32_t k, int t, int e) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t col = (warp * NT + t) * 8 + (lane & 3u) * 2 + e;
  return col < k ? (lane >> 2) * k + col : 0xFFFFFFFFu;
}

// Unit length, rounding and inverse norm for the PROJ_G sequences of a group whose projected vectors are in
// gv[g * k + c] (shared memory).  One warp per sequence; called by the PROJ_CONS consumer threads.
__device__ __forceinline__ void finish_group(const float* gv, uint32_t k, uint32_t B, uint32_t b0,
                                             __nv_bfloat16* __restrict__ fp, float* __restrict__ rq) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t g = warp; g < PROJ_G; g += PROJ_CONS / 32) {
    const uint32_t bq = b0 + g;
    if (bq >= B) continue;
    const float* v = gv + (size_t)g * k;
    float ss = 0.f;
    for (uint32_t c = lane; c < k; c += 32) ss = fmaf(v[c], v[c], ss);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    const float nrm = sqrtf(ss);
    const bool ok = isfinite(ss) && nrm >= 1e-20f;
    __nv_bfloat16* dst = fp + (size_t)bq * k;
    float qs = 0.f;
    for (uint32_t c = lane; c < k; c += 32) {
      const __nv_bfloat16 q = __float2bfloat16_rn(ok ? v[c] / nrm : 0.f);
      dst[c] = q;
      const float qf = __bfloat162float(q);
      qs = fmaf(qf, qf, qs);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) qs += __shfl_xor_sync(0xFFFFFFFFu, qs, o);
    if (lane == 0) rq[bq] = (ok && qs > 0.f) ? 1.0f / sqrtf(qs) : 0.f;
  }
}

// ---------------------------------------------------------------------------
// Without a projection matrix (k == d) the fingerprint is the centred mean itself, scaled and rounded.
// One sequence, NRM_THREADS threads (tid = 0..NRM_THREADS-1) that share the named barrier `bar_id`;
// gv: [d] floats and red: [NRM_THREADS / 32] floats of shared memory.
// ---------------------------------------------------------------------------
constexpr int NRM_THREADS = 256;

__device__ __forceinline__ float nrm_block_sum(float v, float* red, uint32_t tid, uint32_t bar_id) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NRM_THREADS) : "memory");
  if ((tid & 31) == 0) red[tid >> 5] = v;
  asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NRM_THREADS) : "memory");
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < NRM_THREADS / 32; ++i) tot += red[i];
  return tot;
}

__device__ __forceinline__ void normalise_seq(const MeanSrc& src, uint32_t bq, float* gv, float* red,
                                              uint32_t tid, uint32_t bar_id,
                                              __nv_bfloat16* __restrict__ fp, float* __restrict__ rq) {
  const uint32_t d = src.d;
  const SeqBlocks sq = seq_blocks(src, bq);
  float ss = 0.f;
  for (uint32_t i = tid; i < d; i += NRM_THREADS) {
    const float v = centred_mean(src, sq, bq, i);
    gv[i] = v;
    ss = fmaf(v, v, ss);
  }
  ss = nrm_block_sum(ss, red, tid, bar_id);
  const float nrm = sqrtf(ss);
  const bool ok = isfinite(ss) && nrm >= 1e-20f;
  __nv_bfloat16* dst = fp + (size_t)bq * d;
  float qs = 0.f;
  for (uint32_t i = tid; i < d; i += NRM_THREADS) {
    const __nv_bfloat16 q = __float2bfloat16_rn(ok ? gv[i] / nrm : 0.f);
    dst[i] = q;
    const float qf = __bfloat162float(q);
    qs = fmaf(qf, qf, qs);
  }
  qs = nrm_block_sum(qs, red, tid, bar_id);
  if (tid == 0) rq[bq] = (ok && qs > 0.f) ? 1.0f / sqrtf(qs) : 0.f;
}

}  // namespace llmc
