// Dense layer of the miss path: C[M, N] = act(A[M, K] . W[N, K]^T + bias) (+ residual), bf16 in and
// out, fp32 accumulation.  The transformer layer f_l that runs on the misses (Algorithm 1,
// "h_l <- f_l(h_{l-1})") is made of four of these.  Same machinery as the bank scan: TMA (128-byte
// swizzle) into a 4-stage ring, tcgen05.mma 128 x 256 x 16 into two TMEM accumulators, eight epilogue warps
// that drain one accumulator while the next tile's MMAs run and hand their output to the bulk-copy engine
// through shared memory.  The number of valid rows may come from device memory (the miss count of the probe
// that precedes it), so no host sync is needed.
// All mbarrier waits are bounded (status word, see scan.cu).
#include <cuda.h>
#include "llmcache_internal.cuh"
#include "ptx.cuh"
#include "layer.cuh"

namespace llmc {

namespace {
constexpr int GM = 128, GN = 256, GK = 64, GSTAGES = 4, G_UMMA_K = 16;
constexpr int GEMM_THREADS = 320;                   // warp 0: TMA, warp 1: MMA, warps 2..9: epilogue (two sets of four)
constexpr int GEMM_EPI = 256;
constexpr uint32_t GA_BYTES = GM * GK * 2, GB_BYTES = GN * GK * 2;
constexpr uint32_t G_TMEM_COLS = 512;
constexpr uint32_t G_BOX_BYTES = GM * 32 * 2;       // one 32-column group of a tile: 128 rows of 64 bytes
struct GemmSmem {
  static constexpr uint32_t A = 0;
  static constexpr uint32_t B = A + GSTAGES * GA_BYTES;
  static constexpr uint32_t STG = B + GSTAGES * GB_BYTES;        // per epilogue set one box (four warps x 32 rows) on its way out
  static constexpr uint32_t RES = STG + 2 * G_BOX_BYTES;         // the same for the residual on its way in
  static constexpr uint32_t BIAS = RES + 2 * G_BOX_BYTES;        // float [GN]
  static constexpr uint32_t BAR = BIAS + GN * 4;
  static constexpr uint32_t MISC = BAR + 24 * 8;
  static constexpr uint32_t TOTAL = MISC + 64;
};
constexpr uint32_t GEMM_SMEM_BYTES = GemmSmem::TOTAL + 1024;
static_assert(GEMM_SMEM_BYTES <= 232448, "shared memory of one block");
constexpr uint32_t G_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(GN >> 3) << 17) | ((uint32_t)(GM >> 4) << 24);

// GELU with the error function, x/2 + |x|/2 x erf(|x| / sqrt 2), for two values at once with packed fp32
// arithmetic and no special-function instruction: on u = min(|x|, 3.3 sqrt 2) an odd polynomial u Q(u^2) with nine
// coefficients stands for erf(u / sqrt 2) (beyond the clamp erf is within 3.1e-6 of its value there).  The
// coefficients minimise the largest error of GELU itself (gelu_erf_fit.py, beside this file): 8.2e-5 absolute
// with the float32 evaluation included, below the bf16 rounding of the result.  (The rational approximation with
// a reciprocal and an exponential used before cost two special-function instructions per element, and those
// bounded the epilogue of the first feed-forward product.)
__device__ __forceinline__ unsigned long long f2_dup(float x) { return f2_pack(x, x); }
// eight pairs at a time, stage by stage: the nine-term Horner chain of one pair is serial, eight of them side by
// side keep the pipeline fed with two epilogue warps per scheduler
__device__ __forceinline__ void gelu_erf2_x8(unsigned long long (&y)[8]) {
  unsigned long long u[8], s[8], q[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    u[j] = f2_pack(fminf(fabsf(f2_lo(y[j])), 4.666905f), fminf(fabsf(f2_hi(y[j])), 4.666905f));
    s[j] = f2_mul(u[j], u[j]);
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) q[j] = f2_fma(f2_dup(4.615854921e-11f), s[j], f2_dup(-5.357377653e-09f));
  const float k[7] = {2.722534873e-07f, -8.016299034e-06f, 1.529819274e-04f, -2.011742676e-03f,
                      1.894705929e-02f, -1.315938234e-01f, 7.972128987e-01f};
#pragma unroll
  for (int t = 0; t < 7; ++t) {
#pragma unroll
    for (int j = 0; j < 8; ++j) q[j] = f2_fma(q[j], s[j], f2_dup(k[t]));
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const unsigned long long erf_abs = f2_mul(u[j], q[j]);
    const unsigned long long h = f2_pack(0.5f * fabsf(f2_lo(y[j])), 0.5f * fabsf(f2_hi(y[j])));
    y[j] = f2_fma(h, erf_abs, f2_mul(y[j], f2_dup(0.5f)));
  }
}
__device__ __forceinline__ float gelu_tanh_f(float x) {
  return 0.5f * x * (1.0f + tanhf(0.7978845608028654f * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
}  // namespace

// ACT, RES, VT: the activation, whether a residual is added and whether the V columns go out transposed are fixed
// per instantiation, so that each epilogue carries only its own code
template <uint32_t ACT, bool RES, bool VT>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
          const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_res,
          const float* __restrict__ bias, const __nv_bfloat16* __restrict__ residual,
          __nv_bfloat16* __restrict__ out, uint32_t* __restrict__ status,
          uint32_t M_max, uint32_t N, uint32_t KB, const uint32_t* __restrict__ m_seq_dev, uint32_t rows_per_seq,
          VtOut vt) {
  constexpr uint32_t act = ACT;
  griddep_sync();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sA = base + GemmSmem::A, sB = base + GemmSmem::B;
  const uint32_t sSTG = base + GemmSmem::STG, sRES = base + GemmSmem::RES;
  float* sbias = reinterpret_cast<float*>(gbase + GemmSmem::BIAS);
  const uint32_t bar0 = base + GemmSmem::BAR;
  auto full_bar = [&](uint32_t s) { return bar0 + 8 * s; };
  auto empty_bar = [&](uint32_t s) { return bar0 + 8 * (GSTAGES + s); };
  auto tfull_bar = [&](uint32_t b) { return bar0 + 8 * (2 * GSTAGES + b); };
  auto tempty_bar = [&](uint32_t b) { return bar0 + 8 * (2 * GSTAGES + 2 + b); };
  auto res_bar = [&](uint32_t w) { return bar0 + 8 * (2 * GSTAGES + 4 + w); };      // one per epilogue warp
  volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(gbase + GemmSmem::MISC);
  volatile uint32_t* tmem_slot = misc + 0;
  volatile uint32_t* abort_flag = misc + 1;
  volatile uint32_t* epi_go = misc + 2;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned long long lim = wait_limit(status);

  // rows that hold data: all of them, or (sequences counted on the device) x (rows per sequence)
  uint32_t M = M_max;
  if (m_seq_dev) {
    const unsigned long long m = (unsigned long long)(*m_seq_dev) * rows_per_seq;
    M = m < M_max ? (uint32_t)m : M_max;
  }
  const uint32_t MB = (M + GM - 1) / GM, NB = (N + GN - 1) / GN;
  const uint32_t n_tiles = MB * NB;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < GSTAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (uint32_t b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), GEMM_EPI);
    }
    for (uint32_t w = 0; w < GEMM_EPI / 32; ++w) mbar_init(res_bar(w), 1);
    misc[1] = 0; misc[2] = 0; misc[3] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32((const void*)tmem_slot)), "r"(G_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  uint32_t issued = 0, r_issued = 0;
  if (warp == 0) {
    if (lane == 0 && !producer_idle(status)) {         // ---- TMA producer
      bool ok = true;
      for (uint32_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        const uint32_t mb = t / NB, nb = t % NB;       // consecutive blocks share the A tile in L2
        for (uint32_t kb = 0; kb < KB; ++kb) {
          const uint32_t s = issued % GSTAGES, ph = (issued / GSTAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, lim)) { ok = false; break; }
          mbar_expect_tx(full_bar(s), GA_BYTES + GB_BYTES);
          tma_load_2d(sA + s * GA_BYTES, &map_a, (int)(kb * GK), (int)(mb * GM), full_bar(s));
          tma_load_2d(sB + s * GB_BYTES, &map_w, (int)(kb * GK), (int)(nb * GN), full_bar(s));
          ++issued;
        }
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else if (warp == 1) {
    if (lane == 0) {                                   // ---- MMA issuer
      bool ok = true;
      uint32_t it = 0, tile = 0;
      for (uint32_t t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tile) {
        const uint32_t buf = tile & 1u, bph = (tile >> 1) & 1u;
        if (!mbar_wait(tempty_bar(buf), bph ^ 1u, abort_flag, lim)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * GN;
        for (uint32_t kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % GSTAGES, ph = (it / GSTAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, lim)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = smem_desc_sw128(sA + s * GA_BYTES), db = smem_desc_sw128(sB + s * GB_BYTES);
#pragma unroll
          for (uint32_t kk = 0; kk < GK / G_UMMA_K; ++kk)
            tc_mma_bf16(d_tmem, da + kk * (G_UMMA_K * 2 / 16), db + kk * (G_UMMA_K * 2 / 16), G_IDESC, (kb | kk) != 0u);
          tc_commit(empty_bar(s));
        }
        if (ok) tc_commit(tfull_bar(buf));
      }
      if (!ok) { *abort_flag = 1; atomicExch(status, 1u); }
    }
  } else {
    // ---- epilogue: bias, activation, residual, bf16 output; thread = one output row of the tile, 32 columns at
    // a time.  Full tiles leave through shared memory: every thread puts its 64 bytes of a 32-column group into
    // its warp's 32-row staging box (64-byte swizzle, so that the 16-byte stores of a warp spread over all banks)
    // and lane 0 hands the box to the bulk-copy engine, which writes whole lines; the residual rows arrive the same
    // way, one group ahead.  (With one 16-byte store per thread and row the product ran at 0.6-0.75 of the rate of
    // its own main loop: a warp's store touched 32 lines, and more epilogue warps changed nothing.)  The last,
    // partial row block of a device-counted M and the transposed V columns use plain stores.
    // Two sets of four warps share a tile: set 0 takes the even groups, set 1 the odd ones.  Every warp has its own
    // boxes, residual barrier and bulk groups and meets the others only at the tile's ends, so that one warp's
    // arithmetic (the GELU is a chain of dependent instructions) covers another's waits.
    const uint32_t et = threadIdx.x - 64, set = et >> 7, quarter = warp & 3u;
    const uint32_t ew = et >> 5;                        // epilogue warp 0..7
    const uint32_t sub = set * G_BOX_BYTES + quarter * (G_BOX_BYTES / 4);     // this warp's 32 rows of its set's box
    const uint32_t row_in_tile = quarter * 32 + lane;
    const uint32_t my_off = row_in_tile * 64u, sw = (row_in_tile >> 1) & 3u;
    constexpr bool use_res = RES;
    auto tile_full = [&](uint32_t t) { return (t / NB + 1) * GM <= M; };
    uint32_t r_used = 0;
    uint32_t ct = blockIdx.x, cg = set;                // next residual rows to request (lane 0 of every warp)
    auto res_issue = [&]() {
      while (ct < n_tiles && !tile_full(ct)) ct += gridDim.x;
      if (ct >= n_tiles) return;
      const uint32_t cmb = ct / NB, cnb = ct % NB;
      mbar_expect_tx(res_bar(ew), G_BOX_BYTES / 4);
      tma_load_2d(sRES + sub, &map_res, (int)(cnb * GN + cg * 32), (int)(cmb * GM + quarter * 32), res_bar(ew));
      ++r_issued;
      cg += 2;
      if (cg >= GN / 32 || cnb * GN + cg * 32 >= N) { cg = set; ct += gridDim.x; }
    };
    if (use_res && lane == 0) res_issue();
    uint32_t tile = 0;
    for (uint32_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile) {
      const uint32_t mb = t / NB, nb = t % NB;
      const uint32_t buf = tile & 1u, bph = (tile >> 1) & 1u;
      for (uint32_t x = et; x < GN; x += GEMM_EPI) {
        const uint32_t c = nb * GN + x;
        sbias[x] = (bias && c < N) ? bias[c] : 0.f;
      }
      if (et == 0) *epi_go = *abort_flag;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (*epi_go) break;
      if (!mbar_wait(tfull_bar(buf), bph, abort_flag, lim)) { *abort_flag = 1; atomicExch(status, 1u); }
      tc_fence_after();
      const uint32_t taddr = tmem_base + buf * GN + ((quarter * 32u) << 16);
      const uint32_t row = mb * GM + row_in_tile;
      const bool row_ok = row < M, staged = tile_full(t);
#pragma unroll 1
      for (uint32_t c = set * 32; c < GN; c += 64) {
        const uint32_t col0 = nb * GN + c;
        if (col0 >= N) break;                           // N is a multiple of 64: a 32-column group is all in or all out
        uint32_t v[32];
        tc_ld_32x32(taddr + c, v);
        // the residual of this group goes to registers first and its box is refilled at once, so that the next
        // group's residual has this whole group's time to arrive
        uint4 rr[4];
        const bool res_here = staged && use_res;
        if (res_here) {
          if (!mbar_wait(res_bar(ew), r_used & 1u, abort_flag, lim)) { *abort_flag = 1; atomicExch(status, 1u); }
          ++r_used;
          const uint8_t* rb = gbase + GemmSmem::RES + set * G_BOX_BYTES + my_off;
#pragma unroll
          for (uint32_t q = 0; q < 4; ++q) rr[q] = *reinterpret_cast<const uint4*>(rb + ((q ^ sw) << 4));
          __syncwarp();
          if (lane == 0) res_issue();
        }
        tc_wait_ld();
        float f[32];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const float2* b2 = reinterpret_cast<const float2*>(sbias + c) + half * 8;
          unsigned long long y[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float2 b = b2[j];
            y[j] = f2_add(f2_pack(__uint_as_float(v[half * 16 + 2 * j]), __uint_as_float(v[half * 16 + 2 * j + 1])),
                          f2_pack(b.x, b.y));
          }
          if (act == LAYER_ACT_GELU_ERF) gelu_erf2_x8(y);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            f[half * 16 + 2 * j] = f2_lo(y[j]);
            f[half * 16 + 2 * j + 1] = f2_hi(y[j]);
          }
        }
        if (act == LAYER_ACT_GELU_TANH) {
#pragma unroll
          for (int i = 0; i < 32; ++i) f[i] = gelu_tanh_f(f[i]);
        }
        if (VT && col0 >= vt.col0) {
          // the V third of a q|k|v product goes out transposed per head, for the attention kernel:
          // vt[((seq * heads + h) * 64 + c) * pitch + pos]; the lanes of a warp are consecutive positions
          if (row_ok) {
            const uint32_t seq = row / rows_per_seq, pos = row - seq * rows_per_seq;
            const uint32_t hc = col0 - vt.col0;                       // h * 64 + c of the first column
            __nv_bfloat16* dst = vt.ptr + ((size_t)seq * vt.heads * 64 + hc) * vt.pitch + pos;
#pragma unroll
            for (int i = 0; i < 32; ++i) dst[(size_t)i * vt.pitch] = __float2bfloat16_rn(f[i]);
          }
          continue;
        }
        if (staged) {
          if (use_res) {
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q) {
              const uint32_t w[4] = {rr[q].x, rr[q].y, rr[q].z, rr[q].w};
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                f[q * 8 + 2 * u]     += __uint_as_float(w[u] << 16);
                f[q * 8 + 2 * u + 1] += __uint_as_float(w[u] & 0xFFFF0000u);
              }
            }
          }
          if (lane == 0) bulk_wait_read<0>();           // the warp's previous rows have been read out
          __syncwarp();
          uint8_t* ob = gbase + GemmSmem::STG + set * G_BOX_BYTES + my_off;
#pragma unroll
          for (uint32_t q = 0; q < 4; ++q)
            *reinterpret_cast<uint4*>(ob + ((q ^ sw) << 4)) =
                make_uint4(pack_bf16(f[q * 8], f[q * 8 + 1]), pack_bf16(f[q * 8 + 2], f[q * 8 + 3]),
                           pack_bf16(f[q * 8 + 4], f[q * 8 + 5]), pack_bf16(f[q * 8 + 6], f[q * 8 + 7]));
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&map_out, (int)col0, (int)(mb * GM + quarter * 32), sSTG + sub);
            bulk_commit();
          }
          continue;
        }
        if (row_ok) {
          const size_t off = (size_t)row * N + col0;
          if (RES) {
            const uint4* r4 = reinterpret_cast<const uint4*>(residual + off);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 r = r4[q];
              const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                f[q * 8 + 2 * u]     += __uint_as_float(w[u] << 16);
                f[q * 8 + 2 * u + 1] += __uint_as_float(w[u] & 0xFFFF0000u);
              }
            }
          }
          uint4* o4 = reinterpret_cast<uint4*>(out + off);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            o4[q] = make_uint4(pack_bf16(f[q * 8], f[q * 8 + 1]), pack_bf16(f[q * 8 + 2], f[q * 8 + 3]),
                               pack_bf16(f[q * 8 + 4], f[q * 8 + 5]), pack_bf16(f[q * 8 + 6], f[q * 8 + 7]));
        }
      }
      tc_fence_before();
      mbar_arrive(tempty_bar(buf));
      asm volatile("bar.sync 1, 256;" ::: "memory");   // the bias of the next tile overwrites this one's
    }
    if (lane == 0) {
      bulk_wait_all();
      // residual boxes still on their way (only after a wait ran out): they must land before the block ends
      volatile uint32_t never = 0;
      for (; r_used < r_issued; ++r_used) mbar_wait(res_bar(ew), r_used & 1u, &never, 200000000ull);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    const uint32_t back = issued < (uint32_t)GSTAGES ? issued : (uint32_t)GSTAGES;
    volatile uint32_t never = 0;
    for (uint32_t i = 0; i < back; ++i) {
      const uint32_t itx = issued - 1 - i;
      mbar_wait(full_bar(itx % GSTAGES), (itx / GSTAGES) & 1u, &never, 200000000ull);
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(G_TMEM_COLS) : "memory");
  }
}

namespace {
// the instantiation for (act, residual, transposed V columns), or null
using GemmKernel = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const float*,
                            const __nv_bfloat16*, __nv_bfloat16*, uint32_t*, uint32_t, uint32_t, uint32_t, const uint32_t*,
                            uint32_t, VtOut);
GemmKernel gemm_kernel(uint32_t act, bool res, bool vt) {
  if (vt) return (!res && act == LAYER_ACT_NONE) ? k_gemm_tc<LAYER_ACT_NONE, false, true> : nullptr;
  switch (act) {
    case LAYER_ACT_NONE: return res ? k_gemm_tc<LAYER_ACT_NONE, true, false> : k_gemm_tc<LAYER_ACT_NONE, false, false>;
    case LAYER_ACT_GELU_ERF: return res ? k_gemm_tc<LAYER_ACT_GELU_ERF, true, false> : k_gemm_tc<LAYER_ACT_GELU_ERF, false, false>;
    case LAYER_ACT_GELU_TANH: return res ? k_gemm_tc<LAYER_ACT_GELU_TANH, true, false> : k_gemm_tc<LAYER_ACT_GELU_TANH, false, false>;
    default: return nullptr;
  }
}
}  // namespace

cudaError_t setup_gemm_kernel() {
  cudaError_t e = tensor_map_setup();
  if (e != cudaSuccess) return e;
  const uint32_t acts[3] = {LAYER_ACT_NONE, LAYER_ACT_GELU_ERF, LAYER_ACT_GELU_TANH};
  for (uint32_t act : acts)
    for (int res = 0; res < 2; ++res) {
      e = cudaFuncSetAttribute(gemm_kernel(act, res != 0, false), cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
      if (e != cudaSuccess) return e;
    }
  return cudaFuncSetAttribute(gemm_kernel(LAYER_ACT_NONE, false, true), cudaFuncAttributeMaxDynamicSharedMemorySize,
                              GEMM_SMEM_BYTES);
}

// out[M, N] = act(a[M, K] . w[N, K]^T + bias) (+ residual).  K, N multiples of 64.
cudaError_t launch_gemm(const __nv_bfloat16* a, const __nv_bfloat16* w, const float* bias,
                        const __nv_bfloat16* residual, __nv_bfloat16* out, uint32_t* status, uint32_t M_max,
                        uint32_t N, uint32_t K, const uint32_t* m_seq_dev, uint32_t rows_per_seq, uint32_t act,
                        int sm_count, cudaStream_t st, VtOut vt) {
  if (M_max == 0) return cudaSuccess;
  const GemmKernel kern = gemm_kernel(act, residual != nullptr, vt.ptr != nullptr);
  if (!kern) return cudaErrorInvalidValue;                   // e.g. the transposed columns take no residual or activation
  alignas(64) CUtensorMap map_a, map_w, map_out, map_res;
  if (!make_tensor_map_bf16(&map_a, a, M_max, K, GM) || !make_tensor_map_bf16(&map_w, w, N, K, GN) ||
      !make_tensor_map_bf16_box32(&map_out, out, M_max, N) ||
      !make_tensor_map_bf16_box32(&map_res, residual ? residual : out, M_max, N))
    return cudaErrorInvalidValue;
  const uint32_t tiles = ((M_max + GM - 1) / GM) * ((N + GN - 1) / GN);
  const uint32_t grid = tiles < (uint32_t)sm_count ? tiles : (uint32_t)sm_count;
  return launch_k(kern, dim3(grid), dim3(GEMM_THREADS), GEMM_SMEM_BYTES, st, map_a, map_w, map_out, map_res, bias,
                  residual, out, status, M_max, N, K / GK, m_seq_dev, rows_per_seq, vt);
}

}  // namespace llmc
