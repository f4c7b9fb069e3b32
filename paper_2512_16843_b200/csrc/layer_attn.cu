// Multi-head scaled dot-product self-attention of the miss-path layer (Sec. IV-A: h_l = f_l(h_{l-1})), head
// size 64, on the 5th-generation tensor cores.
//
// One block per (sequence, head, tile of 128 queries), two blocks resident per SM so that one block's softmax
// overlaps the other's matrix products.  Per tile of 128 keys:
//   S  = Q K^T        tcgen05.mma 128 x 128 x 64 into tensor memory (Q and K tiles come straight out of the
//                     [tokens, 3d] q|k|v matrix by TMA, 128-byte swizzle)
//   P  = softmax step four warps, one thread per query row: two passes over the row in tensor memory (maximum, then
//                     exponentials and their sum), P written as bf16 into shared memory in the swizzled K-major
//                     layout the next product reads
//   PV = P V          tcgen05.mma 128 x 64 x 128 into a second accumulator; V is read through its per-head
//                     transpose V^T [64, n] (written by k_transpose_v), so that both operands are K-major
//   O  = O * exp(m_old - m_new) + PV   in registers (running maximum m and sum l per row: on-line softmax)
// causal: position i attends to j <= i; key tiles beyond the diagonal are skipped.
// Warp 0 produces (TMA), warp 1 issues the MMAs and owns the tensor memory, warps 2..5 do the softmax and the
// output.  Every wait is bounded (status word, as in scan.cu).
#include <cuda.h>
#include "llmcache_internal.cuh"
#include "ptx.cuh"
#include "layer.cuh"

namespace llmc {

namespace {
constexpr int AT_Q = 128, AT_K = 128, AT_DH = 64;
constexpr int AT_THREADS = 192;
constexpr int AT_SLOTS = 3;                              // ring of 16 KB operand tiles: K_j, V_j, K_j+1, ...
constexpr uint32_t AT_TILE = 16384;                      // bytes of a 128 x 64 (or 2 x 64 x 64) bf16 tile
constexpr uint32_t AT_TMEM_COLS = 256;                   // S: columns 0..127, PV: columns 128..191
struct AttSmem {
  static constexpr uint32_t Q = 0;
  static constexpr uint32_t RING = Q + AT_TILE;
  static constexpr uint32_t P = RING + AT_SLOTS * AT_TILE;            // two 128 x 64 sub-tiles
  static constexpr uint32_t BAR = P + 2 * AT_TILE;                    // q_full, full[3], empty[3], s_full, s_empty, p_full, pv_full, pv_empty
  static constexpr uint32_t MISC = BAR + 16 * 8;
  static constexpr uint32_t TOTAL = MISC + 64;
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
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ void sts16(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
}  // namespace

// V^T per (sequence, head): vt[((seq * heads + h) * 64 + c) * pitch + pos] = v[seq, pos, h * 64 + c].
// One block per (sequence * heads + h, tile of 64 positions).
__global__ void __launch_bounds__(256)
k_transpose_v(const __nv_bfloat16* __restrict__ qkv, __nv_bfloat16* __restrict__ vt, uint32_t n, uint32_t d,
              uint32_t heads, uint32_t pitch, uint32_t seq_max, const uint32_t* __restrict__ m_seq_dev) {
  griddep_sync();
  __shared__ __nv_bfloat16 tile[64][AT_DH + 2];
  uint32_t n_seq = seq_max;
  if (m_seq_dev) n_seq = min(seq_max, *m_seq_dev);
  const uint32_t sh = blockIdx.x, seq = sh / heads, h = sh % heads;
  if (seq >= n_seq) return;
  const uint32_t p0 = blockIdx.y * 64;
  for (uint32_t idx = threadIdx.x; idx < 64 * 32; idx += 256) {        // 64 positions x 32 pairs of head dims
    const uint32_t r = idx >> 5, c2 = idx & 31u;
    uint32_t w = 0;
    if (p0 + r < n)
      w = *reinterpret_cast<const uint32_t*>(qkv + ((size_t)seq * n + p0 + r) * 3 * d + 2 * d + h * AT_DH + c2 * 2);
    *reinterpret_cast<uint32_t*>(&tile[r][c2 * 2]) = w;
  }
  __syncthreads();
  for (uint32_t idx = threadIdx.x; idx < 64 * 64; idx += 256) {
    const uint32_t c = idx >> 6, r = idx & 63u;
    if (p0 + r < n) vt[((size_t)sh * AT_DH + c) * pitch + p0 + r] = tile[r][c];
  }
}

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
  const uint32_t s_full = bar0 + 8 * 7, s_empty = bar0 + 8 * 8, p_full = bar0 + 8 * 9, pv_full = bar0 + 8 * 10,
                 pv_empty = bar0 + 8 * 11;
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
    mbar_init(s_full, 1); mbar_init(s_empty, 128); mbar_init(p_full, 128); mbar_init(pv_full, 1); mbar_init(pv_empty, 128);
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
  const uint32_t tmem_s = tmem_base, tmem_pv = tmem_base + AT_K;

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
        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, lim)) { ok = false; break; }
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
    if (lane == 0) {
      bool ok = mbar_wait(q_full, 0u, abort_flag, lim);
      tc_fence_after();
      const uint64_t dq = smem_desc_sw128(sQ);
      for (uint32_t j = 0; j < nkv && ok; ++j) {
        const uint32_t jp = j & 1u;
        // S = Q K_j^T
        const uint32_t ik = 2 * j, sk = ik % AT_SLOTS, phk = (ik / AT_SLOTS) & 1u;
        if (!mbar_wait(full_bar(sk), phk, abort_flag, lim)) { ok = false; break; }
        if (!mbar_wait(s_empty, jp ^ 1u, abort_flag, lim)) { ok = false; break; }      // softmax is done with S_(j-1)
        tc_fence_after();
        const uint64_t dk = smem_desc_sw128(sRing + sk * AT_TILE);
#pragma unroll
        for (uint32_t kk = 0; kk < AT_DH / 16; ++kk)
          tc_mma_bf16(tmem_s, dq + kk * 2, dk + kk * 2, IDESC_S, kk != 0u);
        tc_commit(empty_bar(sk));
        tc_commit(s_full);
        // PV = P_j V_j
        const uint32_t iv = 2 * j + 1, sv = iv % AT_SLOTS, phv = (iv / AT_SLOTS) & 1u;
        if (!mbar_wait(full_bar(sv), phv, abort_flag, lim)) { ok = false; break; }
        if (!mbar_wait(p_full, jp, abort_flag, lim)) { ok = false; break; }
        if (!mbar_wait(pv_empty, jp ^ 1u, abort_flag, lim)) { ok = false; break; }     // PV_(j-1) has been read
        tc_fence_after();
#pragma unroll
        for (uint32_t kk = 0; kk < AT_K / 16; ++kk) {
          const uint64_t dp = smem_desc_sw128(sP + (kk >> 2) * AT_TILE) + (kk & 3u) * 2;
          const uint64_t dv = smem_desc_sw128(sRing + sv * AT_TILE + (kk >> 2) * (AT_TILE / 2)) + (kk & 3u) * 2;
          tc_mma_bf16(tmem_pv, dp, dv, IDESC_PV, kk != 0u);
        }
        tc_commit(empty_bar(sv));
        tc_commit(pv_full);
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else {
    // ------------------------------------------------------------ softmax + output (128 threads, one query row each)
    const uint32_t quarter = warp & 3u;                  // TMEM lanes this warp may read
    const uint32_t r = quarter * 32 + lane;              // row of the tile
    const uint32_t qrow = q0 + r;
    const uint32_t lane_addr = (quarter * 32u) << 16;
    const float sc = 0.125f * 1.4426950408889634f;       // 1 / sqrt(64), in base-2 exponent units
    float o[AT_DH];
#pragma unroll
    for (int c = 0; c < AT_DH; ++c) o[c] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (uint32_t j = 0; j < nkv; ++j) {
      const uint32_t jp = j & 1u, k0 = j * AT_K;
      if (!mbar_wait(s_full, jp, abort_flag, lim)) { *abort_flag = 1; atomicExch(status, 1u); ok = false; break; }
      tc_fence_after();
      // pass 1: row maximum
      float m_new = m_run;
#pragma unroll 1
      for (uint32_t c = 0; c < AT_K; c += 32) {
        uint32_t v[32];
        tc_ld_32x32(tmem_s + lane_addr + c, v);
        tc_wait_ld();
#pragma unroll
        for (uint32_t i = 0; i < 32; ++i) {
          const uint32_t key = k0 + c + i;
          const bool live = key < n && (!causal || key <= qrow);
          m_new = fmaxf(m_new, live ? __uint_as_float(v[i]) * sc : -INFINITY);
        }
      }
      const float corr = (m_new == -INFINITY) ? 1.f : ex2f(m_run - m_new);
      // pass 2: exponentials, their sum, P as bf16 into shared memory (16-byte chunk c of row r at chunk c ^ (r % 8))
      float psum = 0.f;
#pragma unroll 1
      for (uint32_t c = 0; c < AT_K; c += 32) {
        uint32_t v[32];
        tc_ld_32x32(tmem_s + lane_addr + c, v);
        tc_wait_ld();
        float p[32];
#pragma unroll
        for (uint32_t i = 0; i < 32; ++i) {
          const uint32_t key = k0 + c + i;
          const bool live = key < n && (!causal || key <= qrow) && m_new != -INFINITY;
          p[i] = live ? ex2f(__uint_as_float(v[i]) * sc - m_new) : 0.f;
          psum += p[i];
        }
        const uint32_t sub = sP + (c >> 6) * AT_TILE + r * 128u;
#pragma unroll
        for (uint32_t q4 = 0; q4 < 4; ++q4) {
          const uint32_t chunk = ((c & 63u) >> 3) + q4;
          sts16(sub + ((chunk ^ (r & 7u)) << 4), pack2(p[q4 * 8], p[q4 * 8 + 1]), pack2(p[q4 * 8 + 2], p[q4 * 8 + 3]),
                pack2(p[q4 * 8 + 4], p[q4 * 8 + 5]), pack2(p[q4 * 8 + 6], p[q4 * 8 + 7]));
        }
      }
      tc_fence_before();
      mbar_arrive(s_empty);                                           // S_j has been read
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // P visible to the tensor cores
      mbar_arrive(p_full);
      l_run = l_run * corr + psum;
      m_run = m_new;
      // O = O * corr + P_j V_j
      if (!mbar_wait(pv_full, jp, abort_flag, lim)) { *abort_flag = 1; atomicExch(status, 1u); ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (uint32_t c = 0; c < AT_DH; c += 32) {
        uint32_t v[32];
        tc_ld_32x32(tmem_pv + lane_addr + c, v);
        tc_wait_ld();
#pragma unroll
        for (uint32_t i = 0; i < 32; ++i) o[c + i] = fmaf(o[c + i], corr, __uint_as_float(v[i]));
      }
      tc_fence_before();
      mbar_arrive(pv_empty);
    }
    if (ok && qrow < n) {
      const float inv = 1.0f / l_run;
      uint4* op = reinterpret_cast<uint4*>(out + ((size_t)tok0 + qrow) * d + h * AT_DH);
#pragma unroll
      for (int q4 = 0; q4 < 8; ++q4)
        op[q4] = make_uint4(pack2(o[q4 * 8] * inv, o[q4 * 8 + 1] * inv), pack2(o[q4 * 8 + 2] * inv, o[q4 * 8 + 3] * inv),
                            pack2(o[q4 * 8 + 4] * inv, o[q4 * 8 + 5] * inv), pack2(o[q4 * 8 + 6] * inv, o[q4 * 8 + 7] * inv));
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

cudaError_t launch_attention_tc(const __nv_bfloat16* qkv, __nv_bfloat16* vt, __nv_bfloat16* out, uint32_t* status,
                                uint32_t n, uint32_t d, uint32_t heads, uint32_t seq_max, const uint32_t* m_seq_dev,
                                int causal, cudaStream_t st) {
  if (seq_max == 0) return cudaSuccess;
  const uint32_t pitch = attention_vt_pitch(n);
  alignas(64) CUtensorMap map_qkv, map_vt;
  if (!make_tensor_map_bf16(&map_qkv, qkv, (uint64_t)seq_max * n, 3ull * d, AT_Q) ||
      !make_tensor_map_bf16_pitch(&map_vt, vt, (uint64_t)seq_max * heads * AT_DH, n, pitch, AT_DH))
    return cudaErrorInvalidValue;
  cudaError_t e = launch_k(k_transpose_v, dim3(seq_max * heads, (n + 63) / 64), dim3(256), 0, st, qkv, vt, n, d, heads,
                           pitch, seq_max, m_seq_dev);
  if (e != cudaSuccess) return e;
  const uint32_t qtiles = (n + AT_Q - 1) / AT_Q;
  return launch_k(k_attention_tc, dim3(seq_max * heads * qtiles), dim3(AT_THREADS), ATT_SMEM_BYTES, st, map_qkv, map_vt,
                  out, status, n, d, heads, seq_max, m_seq_dev, causal);
}

}  // namespace llmc
