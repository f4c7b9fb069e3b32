// Multi-head scaled dot-product self-attention of the miss-path layer (Sec. IV-A: h_l = f_l(h_{l-1})), head
// size 64, on the 5th-generation tensor cores.
//
// One block per (sequence, head, tile of 128 queries), two blocks resident per SM so that one block's softmax
// overlaps the other's matrix products.  Per tile of 128 keys:
//   S  = Q K^T        tcgen05.mma 128 x 128 x 64 into tensor memory (Q and K tiles come straight out of the
//                     [tokens, 3d] q|k|v matrix by TMA, 128-byte swizzle)
//   P  = softmax step eight warps, two threads per query row: two passes over the row in tensor memory (maximum,
//                     then exponentials and their sum), P written as bf16 into shared memory in the swizzled
//                     K-major layout the next product reads
//   PV = P V          tcgen05.mma 128 x 64 x 128; V is read through its per-head transpose V^T [64, n] (written
//                     by the epilogue of the q|k|v product), so that both operands are K-major
//   O  = O * exp(m_old - m_new) + PV   in registers (running maximum m and sum l per row: on-line softmax)
// causal: position i attends to j <= i; key tiles beyond the diagonal are skipped.
// Warp 0 produces (TMA), warp 1 issues the MMAs and owns the tensor memory, warps 2..9 do the softmax and the
// output.  Two accumulators of 128 columns alternate between key tiles, so that the S of the next tile is computed
// while the softmax works on the current one.  Every wait is bounded (status word, as in scan.cu).
#include <cuda.h>
#include <type_traits>
#include "llmcache_internal.cuh"
#include "ptx.cuh"
#include "layer.cuh"

namespace llmc {

namespace {
constexpr int AT_Q = 128, AT_K = 128, AT_DH = 64;
constexpr int AT_THREADS = 320;                          // warp 0: TMA, warp 1: MMA, warps 2..9: softmax (2 threads per query row)
constexpr int AT_SOFT = 256;
constexpr int AT_SLOTS = 3;                              // ring of 16 KB operand tiles: K_j, V_j, K_j+1, ...
constexpr uint32_t AT_TILE = 16384;                      // bytes of a 128 x 64 (or 2 x 64 x 64) bf16 tile
constexpr uint32_t AT_TMEM_COLS = 256;                   // two accumulators of 128 columns
struct AttSmem {
  static constexpr uint32_t Q = 0;
  static constexpr uint32_t RING = Q + AT_TILE;
  static constexpr uint32_t P = RING + AT_SLOTS * AT_TILE;            // two 128 x 64 sub-tiles
  static constexpr uint32_t BAR = P + 2 * AT_TILE;                    // q_full, full[3], empty[3], s_full[2], p_full, pv_full, pv_read[2]
  static constexpr uint32_t MISC = BAR + 16 * 8;
  static constexpr uint32_t XCH = MISC + 64;                          // float [2 tile parities + 1][2 halves][128 rows]: row maxima; row sums
  static constexpr uint32_t TOTAL = XCH + 3 * 2 * 128 * 4;
};
constexpr uint32_t ATT_SMEM_BYTES = AttSmem::TOTAL + 1024;            // slack for manual alignment
// kind::f16 instruction descriptors: fp32 accumulator, bf16 A and B, both K-major, M = 128
constexpr uint32_t IDESC_S = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(AT_K >> 3) << 17) | ((uint32_t)(AT_Q >> 4) << 24);
constexpr uint32_t IDESC_PV = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(AT_DH >> 3) << 17) | ((uint32_t)(AT_Q >> 4) << 24);

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3f(float a, float b, float c) {       // one instruction on this architecture
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
// named barrier of the two softmax warps that share TMEM lane quarter q (barrier 0 is __syncthreads)
__device__ __forceinline__ void pair_sync(uint32_t q) {
  switch (q) {
    case 0: asm volatile("bar.sync 1, 64;" ::: "memory"); break;
    case 1: asm volatile("bar.sync 2, 64;" ::: "memory"); break;
    case 2: asm volatile("bar.sync 3, 64;" ::: "memory"); break;
    default: asm volatile("bar.sync 4, 64;" ::: "memory"); break;
  }
}
__device__ __forceinline__ void sts16(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
}  // namespace

__global__ void __launch_bounds__(AT_THREADS, 2)
k_attention_tc(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_vt,
               __nv_bfloat16* __restrict__ out, uint32_t* __restrict__ status, uint32_t n, uint32_t d, uint32_t heads,
               uint32_t seq_max, const uint32_t* __restrict__ m_seq_dev, int causal) {
  griddep_sync();
  uint32_t n_seq = seq_max;
  if (m_seq_dev) n_seq = min(seq_max, *m_seq_dev);
  const uint32_t qtiles = (n + AT_Q - 1) / AT_Q;
  const uint32_t seq = blockIdx.x / (heads * qtiles);
  if (seq >= n_seq) return;                                            // uniform over the block; nothing allocated yet
  const uint32_t rem = blockIdx.x % (heads * qtiles);
  const uint32_t h = rem / qtiles, qt = rem % qtiles;
  const uint32_t q0 = qt * AT_Q;
  const uint32_t tok0 = seq * n;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + AttSmem::Q, sRing = base + AttSmem::RING, sP = base + AttSmem::P;
  const uint32_t bar0 = base + AttSmem::BAR;
  const uint32_t q_full = bar0;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * (1 + s); };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (1 + AT_SLOTS + s); };
  // s_full[2]: S of a tile is complete in accumulator 0 / 1; p_full: P of a tile is in shared memory (and its S
  // has been read); pv_full: PV of a tile is complete; pv_read[2]: the PV in accumulator 0 / 1 has been read
  const uint32_t s_full = bar0 + 8 * 7, p_full = bar0 + 8 * 9, pv_full = bar0 + 8 * 10, pv_read = bar0 + 8 * 11;
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(gbase + AttSmem::MISC);
  volatile uint32_t* tmem_slot = misc + 0;
  volatile uint32_t* abort_flag = misc + 1;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned long long lim = wait_limit(status);

  const uint32_t ntiles = (n + AT_K - 1) / AT_K;
  const uint32_t nkv = causal ? min(ntiles, (min(n, q0 + AT_Q) - 1) / AT_K + 1) : ntiles;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (uint32_t s = 0; s < AT_SLOTS; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(s_full, 1); mbar_init(s_full + 8, 1); mbar_init(p_full, AT_SOFT); mbar_init(pv_full, 1);
    mbar_init(pv_read, AT_SOFT); mbar_init(pv_read + 8, AT_SOFT);
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(AT_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  uint32_t issued = 0;                                   // producer: ring tiles armed so far
  bool q_armed = false;
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && !producer_idle(status)) {
      bool ok = true;
      mbar_expect_tx(q_full, AT_TILE);
      tma_load_2d(sQ, &map_qkv, (int)(h * AT_DH), (int)(tok0 + q0), q_full);
      q_armed = true;
      for (uint32_t i = 0; i < 2 * nkv && ok; ++i) {
        const uint32_t s = i % AT_SLOTS, ph = (i / AT_SLOTS) & 1u, j = i >> 1;
        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, lim, 64)) { ok = false; break; }
        mbar_expect_tx(full_bar(s), AT_TILE);
        const uint32_t dst = sRing + s * AT_TILE;
        if ((i & 1u) == 0) {
          tma_load_2d(dst, &map_qkv, (int)(d + h * AT_DH), (int)(tok0 + j * AT_K), full_bar(s));
        } else {
          const int row = (int)((seq * heads + h) * AT_DH);
          tma_load_2d(dst, &map_vt, (int)(j * AT_K), row, full_bar(s));
          tma_load_2d(dst + AT_TILE / 2, &map_vt, (int)(j * AT_K + 64), row, full_bar(s));
        }
        ++issued;
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // Tile j uses accumulator j % 2: first for S_j (128 columns), then, once the softmax has read it, for
    // PV_j (its first 64 columns).  S_(j+1) is issued while the softmax works on tile j, so the softmax never
    // waits for a product that could have run earlier.  Operand tiles are consumed in the order
    // K_0, K_1, V_0, K_2, V_1, ...; item i of the load order K_0, V_0, K_1, V_1, ... sits in ring slot i % 3.
    if (lane == 0) {
      bool ok = mbar_wait(q_full, 0u, abort_flag, lim, 64);
      tc_fence_after();
      const uint64_t dq = smem_desc_sw128(sQ);
      auto issue_s = [&](uint32_t j) -> bool {          // S_j = Q K_j^T into accumulator j % 2
        const uint32_t ik = 2 * j, sk = ik % AT_SLOTS, phk = (ik / AT_SLOTS) & 1u;
        if (!mbar_wait(full_bar(sk), phk, abort_flag, lim, 64)) return false;
        // the accumulator held PV_(j-2): the softmax must have read it
        if (j >= 2 && !mbar_wait(pv_read + 8 * (j & 1u), ((j >> 1) - 1u) & 1u, abort_flag, lim, 64)) return false;
        tc_fence_after();
        const uint64_t dk = smem_desc_sw128(sRing + sk * AT_TILE);
        const uint32_t acc = tmem_base + (j & 1u) * AT_K;
#pragma unroll
        for (uint32_t kk = 0; kk < AT_DH / 16; ++kk)
          tc_mma_bf16(acc, dq + kk * 2, dk + kk * 2, IDESC_S, kk != 0u);
        tc_commit(empty_bar(sk));
        tc_commit(s_full + 8 * (j & 1u));                // the (j / 2)-th completion of this barrier
        return true;
      };
      if (ok && nkv) ok = issue_s(0);
      for (uint32_t j = 0; j < nkv && ok; ++j) {
        if (j + 1 < nkv && !issue_s(j + 1)) { ok = false; break; }
        // PV_j = P_j V_j into the first 64 columns of accumulator j % 2 (S_j has been read: p_full says so)
        const uint32_t iv = 2 * j + 1, sv = iv % AT_SLOTS, phv = (iv / AT_SLOTS) & 1u;
        if (!mbar_wait(full_bar(sv), phv, abort_flag, lim, 64)) { ok = false; break; }
        if (!mbar_wait(p_full, j & 1u, abort_flag, lim, 64)) { ok = false; break; }
        tc_fence_after();
        const uint32_t acc = tmem_base + (j & 1u) * AT_K;
#pragma unroll
        for (uint32_t kk = 0; kk < AT_K / 16; ++kk) {
          const uint64_t dp = smem_desc_sw128(sP + (kk >> 2) * AT_TILE) + (kk & 3u) * 2;
          const uint64_t dv = smem_desc_sw128(sRing + sv * AT_TILE + (kk >> 2) * (AT_TILE / 2)) + (kk & 3u) * 2;
          tc_mma_bf16(acc, dp, dv, IDESC_PV, kk != 0u);
        }
        tc_commit(empty_bar(sv));
        tc_commit(pv_full);
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else {
    // ------------------------------------------------------------ softmax + output
    // 256 threads, two per query row: warps w and w + 4 read the same 32 lanes of tensor memory; the first takes
    // key columns 0..63 of a tile and output columns 0..31, the second key columns 64..127 and output columns
    // 32..63.  The two exchange their row maxima through shared memory once per tile; the row sums are kept
    // apart until the end (both threads scale by the same factors).
    const uint32_t quarter = warp & 3u;                  // TMEM lanes this warp may read
    const uint32_t hf = (warp - 2u) >> 2;                // which half of the columns
    const uint32_t r = quarter * 32 + lane;              // row of the tile
    const uint32_t qrow = q0 + r;
    const uint32_t lane_addr = (quarter * 32u) << 16;
    const float sc = 0.125f * 1.4426950408889634f;       // 1 / sqrt(64), in base-2 exponent units
    float* xch = reinterpret_cast<float*>(gbase + AttSmem::XCH);
    unsigned long long o2[16];                           // 32 output columns as packed pairs
#pragma unroll
    for (int c = 0; c < 16; ++c) o2[c] = 0ull;
    float m_run = -INFINITY, l_run = 0.f, corr_prev = 1.f;
    bool ok = true;
    // O = O * corr + PV of tile j (its product sits in the first 64 columns of accumulator j % 2)
    auto accumulate = [&](uint32_t j, float corr) -> bool {
      if (!mbar_wait(pv_full, j & 1u, abort_flag, lim, 32)) return false;
      tc_fence_after();
      uint32_t v[32];
      tc_ld_32x32(tmem_base + (j & 1u) * AT_K + lane_addr + hf * 32, v);
      tc_wait_ld();
      const unsigned long long c2 = f2_pack(corr, corr);
#pragma unroll
      for (uint32_t i = 0; i < 16; ++i)
        o2[i] = f2_fma(o2[i], c2, f2_pack(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])));
      tc_fence_before();
      mbar_arrive(pv_read + 8 * (j & 1u));
      return true;
    };
    for (uint32_t j = 0; j < nkv; ++j) {
      const uint32_t k0 = j * AT_K + hf * 64;            // first key of this thread's columns
      const uint32_t acc = tmem_base + (j & 1u) * AT_K + lane_addr + hf * 64;
      // masking is needed only in the tile that holds the end of the sequence and, if causal, on the diagonal
      const bool masked = (j * AT_K + AT_K > n) || (causal && j * AT_K + AT_K > q0 + 1);
      if (!mbar_wait(s_full + 8 * (j & 1u), (j >> 1) & 1u, abort_flag, lim, 32)) { ok = false; break; }
      tc_fence_after();
      // pass 1: maximum of the raw products over this thread's 64 columns (the scale is positive)
      float mx = -INFINITY;
#pragma unroll 1
      for (uint32_t c = 0; c < 64; c += 32) {
        uint32_t v[32];
        tc_ld_32x32(acc + c, v);
        tc_wait_ld();
        if (masked) {
#pragma unroll
          for (uint32_t i = 0; i < 32; ++i) {
            const uint32_t key = k0 + c + i;
            if (key < n && (!causal || key <= qrow)) mx = fmaxf(mx, __uint_as_float(v[i]));
          }
        } else {
          // four independent chains, joined at the end
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (uint32_t i = 0; i < 32; i += 8) {
#pragma unroll
            for (uint32_t u = 0; u < 4; ++u)
              m4[u] = max3f(m4[u], __uint_as_float(v[i + 2 * u]), __uint_as_float(v[i + 2 * u + 1]));
          }
          mx = fmaxf(max3f(mx, m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        }
      }
      float* xm = xch + (j & 1u) * 256;
      xm[hf * 128 + r] = mx;
      pair_sync(quarter);                                // the two warps that share these rows
      const float m_new = fmaxf(m_run, fmaxf(mx, xm[(hf ^ 1u) * 128 + r]) * sc);
      // the product of the previous tile, while the tensor cores are free to start the next S
      if (j > 0 && !accumulate(j - 1, corr_prev)) { ok = false; break; }
      const bool dead = m_new == -INFINITY;              // no key of any tile so far is visible to this row
      const float corr = dead ? 1.f : ex2f(m_run - m_new);
      const unsigned long long sc2 = f2_pack(sc, sc), nm2 = f2_pack(dead ? 0.f : -m_new, dead ? 0.f : -m_new);
      // pass 2: exponentials, their sum, P as bf16 into shared memory (16-byte chunk c of row r at chunk c ^ (r % 8))
      float psa = 0.f, psb = 0.f;                        // two running sums (even and odd columns)
      const uint32_t sub = sP + hf * AT_TILE + r * 128u;
      // two copies of the loop: only the tile that holds the sequence's end or the diagonal tests every key
      auto pass2 = [&](auto with_mask) {
        constexpr bool MASKED = decltype(with_mask)::value;
#pragma unroll 1
        for (uint32_t c = 0; c < 64; c += 32) {
          uint32_t v[32];
          tc_ld_32x32(acc + c, v);
          tc_wait_ld();
#pragma unroll
          for (uint32_t q4 = 0; q4 < 4; ++q4) {
            uint32_t pk[4];
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) {
              const uint32_t i = q4 * 8 + 2 * e;
              const unsigned long long t2 = f2_fma(f2_pack(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), sc2, nm2);
              float pa = ex2f(f2_lo(t2)), pb = ex2f(f2_hi(t2));
              if constexpr (MASKED) {
                const uint32_t key = k0 + c + i;
                if (dead || !(key < n && (!causal || key <= qrow))) pa = 0.f;
                if (dead || !(key + 1 < n && (!causal || key + 1 <= qrow))) pb = 0.f;
              }
              psa += pa;
              psb += pb;
              pk[e] = pack2(pa, pb);
            }
            const uint32_t chunk = (c >> 3) + q4;
            sts16(sub + ((chunk ^ (r & 7u)) << 4), pk[0], pk[1], pk[2], pk[3]);
          }
        }
      };
      if (masked) pass2(std::true_type{}); else pass2(std::false_type{});
      tc_fence_before();                                              // S_j has been read ...
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // ... and P_j is visible to the tensor cores
      mbar_arrive(p_full);
      l_run = l_run * corr + (psa + psb);
      m_run = m_new;
      corr_prev = corr;
    }
    if (ok && nkv) ok = accumulate(nkv - 1, corr_prev);
    if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    // the row's sum is the sum of the two threads' sums
    xch[512 + hf * 128 + r] = l_run;
    pair_sync(quarter);
    const float l_tot = l_run + xch[512 + (hf ^ 1u) * 128 + r];
    if (ok && qrow < n) {
      const float inv = 1.0f / l_tot;
      uint4* op = reinterpret_cast<uint4*>(out + ((size_t)tok0 + qrow) * d + h * AT_DH + hf * 32);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4)
        op[q4] = make_uint4(pack2(f2_lo(o2[q4 * 4]) * inv, f2_hi(o2[q4 * 4]) * inv),
                            pack2(f2_lo(o2[q4 * 4 + 1]) * inv, f2_hi(o2[q4 * 4 + 1]) * inv),
                            pack2(f2_lo(o2[q4 * 4 + 2]) * inv, f2_hi(o2[q4 * 4 + 2]) * inv),
                            pack2(f2_lo(o2[q4 * 4 + 3]) * inv, f2_hi(o2[q4 * 4 + 3]) * inv));
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    // loads that were armed but never consumed must land before the block's shared memory is released
    volatile uint32_t never = 0;
    if (q_armed) mbar_wait(q_full, 0u, &never, 200000000ull);
    const uint32_t back = issued < (uint32_t)AT_SLOTS ? issued : (uint32_t)AT_SLOTS;
    for (uint32_t i = 0; i < back; ++i) {
      const uint32_t itx = issued - 1 - i;
      mbar_wait(full_bar(itx % AT_SLOTS), (itx / AT_SLOTS) & 1u, &never, 200000000ull);
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(AT_TMEM_COLS) : "memory");
  }
}

cudaError_t setup_attention_kernel() {
  cudaError_t e = tensor_map_setup();
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_attention_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM_BYTES);
}

// Positions between the rows of V^T: a multiple of 8 (16 bytes), so that every row can start a TMA box.
uint32_t attention_vt_pitch(uint32_t n) { return (n + 7u) / 8u * 8u; }

cudaError_t launch_attention_tc(const __nv_bfloat16* qkv, const __nv_bfloat16* vt, __nv_bfloat16* out, uint32_t* status,
                                uint32_t n, uint32_t d, uint32_t heads, uint32_t seq_max, const uint32_t* m_seq_dev,
                                int causal, cudaStream_t st) {
  if (seq_max == 0) return cudaSuccess;
  const uint32_t pitch = attention_vt_pitch(n);
  alignas(64) CUtensorMap map_qkv, map_vt;
  if (!make_tensor_map_bf16(&map_qkv, qkv, (uint64_t)seq_max * n, 3ull * d, AT_Q) ||
      !make_tensor_map_bf16_pitch(&map_vt, vt, (uint64_t)seq_max * heads * AT_DH, n, pitch, AT_DH))
    return cudaErrorInvalidValue;
  const uint32_t qtiles = (n + AT_Q - 1) / AT_Q;
  return launch_k(k_attention_tc, dim3(seq_max * heads * qtiles), dim3(AT_THREADS), ATT_SMEM_BYTES, st, map_qkv, map_vt,
                  out, status, n, d, heads, seq_max, m_seq_dev, causal);
}

}  // namespace llmc
