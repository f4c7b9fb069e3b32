// Bank scan (Sec. III-C, Sec. IV-A): cosine of every query fingerprint against
// every occupied slot, reduced on the fly to the best slot per query.  The
// B x N score matrix is never written to memory.
//
// The scan is the dense contraction  S[b, j] = sum_c q[b, c] * f[j, c]  over bf16
// fingerprints, both stored with the fingerprint dimension contiguous.  It runs
// on the 5th-generation tensor cores:
//   - one warp streams 128 x 64 query tiles and BN x 64 key tiles into shared
//     memory with TMA (128-byte swizzle), four stages deep;
//   - one thread issues tcgen05.mma (M = 128 queries, N = BN slots, K = 16 per
//     instruction) into one of two BN-column fp32 accumulators in tensor memory;
//   - four warps drain the other accumulator with tcgen05.ld: each thread owns
//     one query row, scales by the slot's inverse norm, masks free slots to -inf
//     and keeps a running (best score, lowest slot) in registers.
// A block walks a run of key tiles for one query tile and publishes its result
// with one 64-bit atomicMax per query (score in orderable form above, inverted
// slot below, so that equal scores resolve to the lowest slot).
// BN is 256 where the scan is a throughput problem; a bank of a few thousand keys
// is cut into tiles of 128 or 64 keys instead, so that its few tiles spread over
// more SMs and an epilogue thread walks fewer columns.
//
// Every wait on an mbarrier is bounded: on expiry the block records
// LLMCACHE_ERR_TIMEOUT in the bank's status word, drains what it has in flight,
// frees its tensor memory and returns.
#include <cuda.h>
#include "llmcache_internal.cuh"
#include "ptx.cuh"

namespace llmc {

constexpr int BM = 128;            // queries per tile (MMA M)
constexpr int BK = 64;             // fingerprint elements per stage (128 bytes: one swizzle span)
constexpr int STAGES = 4;
constexpr int UMMA_K = 16;
constexpr int SCAN_THREADS = 192;  // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..5: epilogue
constexpr uint32_t A_BYTES = BM * BK * 2;   // 16 KB

template <int BN>                  // slots per tile (MMA N): 64, 128 or 256
struct ScanSmem {
  static constexpr uint32_t B_BYTES = BN * BK * 2;              // 8 / 16 / 32 KB
  static constexpr uint32_t TMEM_COLS = 2 * BN;                 // two accumulators of BN columns (a power of two >= 32)
  // offsets from the 1024-byte aligned base of dynamic shared memory
  static constexpr uint32_t A = 0;
  static constexpr uint32_t B = A + STAGES * A_BYTES;
  static constexpr uint32_t SB = B + STAGES * B_BYTES;          // float2 [2][BN]
  static constexpr uint32_t BAR = SB + 2 * BN * 8;              // full[4] empty[4] tfull[2] tempty[2]
  static constexpr uint32_t MISC = BAR + 16 * 8;                // tmem base, abort flag, epilogue go flags
  static constexpr uint32_t TOTAL = MISC + 64;
  static constexpr uint32_t BYTES = TOTAL + 1024;               // slack for manual alignment
  // kind::f16 instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = BN.
  static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
};

// ---------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
k_scan_tc(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_bank,
          const float* __restrict__ rb, const uint8_t* __restrict__ valid,
          unsigned long long* __restrict__ best, uint32_t* __restrict__ status,
          uint32_t B, uint32_t N, uint32_t KB, uint32_t MB, uint32_t NB, uint32_t chunk_len, uint32_t n_units,
          uint32_t slot_base) {
  griddep_sync();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  using SM = ScanSmem<BN>;
  constexpr uint32_t B_BYTES = SM::B_BYTES, TMEM_COLS = SM::TMEM_COLS, IDESC = SM::IDESC;
  const uint32_t sA = base + SM::A, sB = base + SM::B;
  float2* sb = reinterpret_cast<float2*>(gbase + SM::SB);
  const uint32_t bar0 = base + SM::BAR;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (STAGES + s); };
  auto tfull_bar = [&](uint32_t b) { return bar0 + 8 * (2 * STAGES + b); };
  auto tempty_bar = [&](uint32_t b) { return bar0 + 8 * (2 * STAGES + 2 + b); };
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(gbase + SM::MISC);
  volatile uint32_t* tmem_slot = misc + 0;
  volatile uint32_t* abort_flag = misc + 1;
  volatile uint32_t* epi_go = misc + 2;          // [2]

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned long long lim = wait_limit(status);

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (uint32_t b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 128); }
    misc[1] = 0; misc[2] = 0; misc[3] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  uint32_t issued = 0;                            // producer: stages armed so far
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && !producer_idle(status)) {
      bool ok = true;
      for (uint32_t u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const uint32_t mb = u % MB, ch = u / MB;
        const uint32_t nb0 = ch * chunk_len, nb1 = min(NB, nb0 + chunk_len);
        for (uint32_t nb = nb0; nb < nb1 && ok; ++nb) {
          for (uint32_t kb = 0; kb < KB; ++kb) {
            const uint32_t s = issued % STAGES, ph = (issued / STAGES) & 1u;
            if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, lim)) { ok = false; break; }
            mbar_expect_tx(full_bar(s), A_BYTES + B_BYTES);
            tma_load_2d(sA + s * A_BYTES, &map_q, (int)(kb * BK), (int)(mb * BM), full_bar(s));
            tma_load_2d(sB + s * B_BYTES, &map_bank, (int)(kb * BK), (int)(nb * BN), full_bar(s));
            ++issued;
          }
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      uint32_t it = 0, tile = 0;
      for (uint32_t u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
        const uint32_t ch = u / MB;
        const uint32_t nb0 = ch * chunk_len, nb1 = min(NB, nb0 + chunk_len);
        for (uint32_t nb = nb0; nb < nb1 && ok; ++nb, ++tile) {
          const uint32_t buf = tile & 1u, bph = (tile >> 1) & 1u;
          if (!mbar_wait(tempty_bar(buf), bph ^ 1u, abort_flag, lim)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * BN;
          for (uint32_t kb = 0; kb < KB; ++kb, ++it) {
            const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
            if (!mbar_wait(full_bar(s), ph, abort_flag, lim)) { ok = false; break; }
            tc_fence_after();
            const uint64_t da = smem_desc_sw128(sA + s * A_BYTES), db = smem_desc_sw128(sB + s * B_BYTES);
#pragma unroll
            for (uint32_t kk = 0; kk < BK / UMMA_K; ++kk)
              tc_mma_bf16(d_tmem, da + kk * (UMMA_K * 2 / 16), db + kk * (UMMA_K * 2 / 16), IDESC, (kb | kk) != 0u);
            tc_commit(empty_bar(s));              // stage reusable once these MMAs have read it
          }
          if (ok) tc_commit(tfull_bar(buf));      // accumulator complete
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else {
    // ------------------------------------------------------------ epilogue (128 threads)
    const uint32_t et = threadIdx.x - 64;         // 0..127
    const uint32_t quarter = warp & 3u;           // TMEM lanes this warp may read
    const uint32_t row_in_tile = quarter * 32 + lane;
    uint32_t tile = 0;
    bool stop = false;
    for (uint32_t u = blockIdx.x; u < n_units && !stop; u += gridDim.x) {
      const uint32_t mb = u % MB, ch = u / MB;
      const uint32_t nb0 = ch * chunk_len, nb1 = min(NB, nb0 + chunk_len);
      float best_s = -INFINITY;
      uint32_t best_j = 0xFFFFFFFFu;
      for (uint32_t nb = nb0; nb < nb1; ++nb, ++tile) {
        const uint32_t buf = tile & 1u, bph = (tile >> 1) & 1u;
        float2* sbt = sb + buf * BN;
#pragma unroll
        for (uint32_t x = et; x < BN; x += 128) {
          const uint32_t j = nb * BN + x;
          const bool live = j < N && valid[j];
          sbt[x] = live ? make_float2(rb[j], 0.f) : make_float2(0.f, -INFINITY);
        }
        if (et == 0) epi_go[buf] = *abort_flag;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (epi_go[buf]) { stop = true; break; }  // uniform over the 128 threads
        if (!mbar_wait(tfull_bar(buf), bph, abort_flag, lim)) { *abort_flag = 1; atomicExch(status, 1u); }
        tc_fence_after();
        const uint32_t taddr = tmem_base + buf * BN + ((quarter * 32u) << 16);
#pragma unroll 1
        for (uint32_t c = 0; c < BN; c += 32) {
          uint32_t v[32];
          tc_ld_32x32(taddr + c, v);
          tc_wait_ld();
          const uint32_t j0 = nb * BN + c;
#pragma unroll
          for (uint32_t i = 0; i < 32; ++i) {
            const float2 w = sbt[c + i];
            const float s = fmaf(__uint_as_float(v[i]), w.x, w.y);
            if (s > best_s) { best_s = s; best_j = j0 + i; }
          }
        }
        tc_fence_before();
        mbar_arrive(tempty_bar(buf));
      }
      const uint32_t b = mb * BM + row_in_tile;
      // slot_base: where this bank's slots start in a bank that is split over several (0 for a whole bank)
      if (!stop && b < B && best_j != 0xFFFFFFFFu) atomicMax(best + b, pack_best(best_s, best_j + slot_base));
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // loads that were armed but never consumed must land before the block's shared memory is released
    const uint32_t back = issued < (uint32_t)STAGES ? issued : (uint32_t)STAGES;
    volatile uint32_t never = 0;
    for (uint32_t i = 0; i < back; ++i) {
      const uint32_t itx = issued - 1 - i;
      mbar_wait(full_bar(itx % STAGES), (itx / STAGES) & 1u, &never, 200000000ull);
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------
cudaError_t setup_scan_kernels() {
  cudaError_t e = tensor_map_setup();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_scan_tc<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScanSmem<256>::BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_scan_tc<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScanSmem<128>::BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_scan_tc<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, ScanSmem<64>::BYTES);
  return e;
}

template <int BN>
static cudaError_t launch_scan_bn(llmcache_bank* bk, const __nv_bfloat16* q, uint32_t B, cudaStream_t st,
                                  unsigned long long* words, uint32_t slot_base) {
  const uint32_t N = bk->desc.capacity, k = bk->desc.fp_dim;
  alignas(64) CUtensorMap map_q, map_bank;
  if (!make_tensor_map_bf16(&map_q, q, B, k, BM) || !make_tensor_map_bf16(&map_bank, bk->a.fp, N, k, BN))
    return cudaErrorInvalidValue;
  const uint32_t MB = (B + BM - 1) / BM, NB = (N + BN - 1) / BN, KB = k / BK;
  // split the key tiles into runs so that there are a few units of work per SM when the problem allows
  const uint32_t target = 4u * (uint32_t)bk->sm_count;
  uint32_t chunks = (target + MB - 1) / MB;
  if (chunks < 1) chunks = 1;
  if (chunks > NB) chunks = NB;
  const uint32_t chunk_len = (NB + chunks - 1) / chunks;
  chunks = (NB + chunk_len - 1) / chunk_len;
  const uint32_t n_units = MB * chunks;
  const uint32_t grid = n_units < (uint32_t)bk->sm_count ? n_units : (uint32_t)bk->sm_count;
  ProfScope prof(bk, LLMCACHE_K_SCAN, st);
  return launch_k(k_scan_tc<BN>, dim3(grid), dim3(SCAN_THREADS), ScanSmem<BN>::BYTES, st, map_q, map_bank,
                  (const float*)bk->a.rb, (const uint8_t*)bk->a.valid, words ? words : bk->a.best, bk->a.status, B, N,
                  KB, MB, NB, chunk_len, n_units, slot_base);
}

// words == nullptr: best words go to the bank's own array; else to `words` (combined by atomicMax with what is
// there), with slot numbers shifted by slot_base.
cudaError_t launch_scan(llmcache_bank* bk, const __nv_bfloat16* q, uint32_t B, cudaStream_t st,
                        unsigned long long* words, uint32_t slot_base) {
  if (B == 0) return cudaSuccess;
  // the widest key tile that still gives every SM a tile; small banks take narrower tiles
  const unsigned long long MB = (B + BM - 1) / BM, N = bk->desc.capacity, sms = (unsigned long long)bk->sm_count;
  if (MB * ((N + 255) / 256) >= sms) return launch_scan_bn<256>(bk, q, B, st, words, slot_base);
  if (MB * ((N + 127) / 128) >= sms) return launch_scan_bn<128>(bk, q, B, st, words, slot_base);
  return launch_scan_bn<64>(bk, q, B, st, words, slot_base);
}

}  // namespace llmc
