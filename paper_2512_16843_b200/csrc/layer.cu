// The transformer layer f_l that runs on the misses (Sec. IV-A: h_l = f_l(h_{l-1}); Algorithm 1
// else-branch).  Plain layer kernels: the four dense layers are layer_gemm.cu; here are layer
// normalisation, multi-head self-attention, and the layer object of the C ABI.
//   post-norm, bidirectional, GELU(erf)   : BERT-style encoder layer
//   pre-norm,  causal,        GELU(tanh)  : GPT-2-style decoder layer
// Activations are bf16 in memory, arithmetic is fp32.  The number of sequences to process can be
// read from device memory (the miss count of the preceding probe), so the caller needs no host sync.
#include <cmath>
#include <new>
#include "layer.cuh"

namespace llmc {
__device__ __forceinline__ uint32_t smem_u32_of(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
}

namespace llmc {

// ---------------------------------------------------------------------------
// Layer normalisation over the last dimension, one warp per row; biased variance, eps inside the root.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_layernorm(const __nv_bfloat16* __restrict__ x, const float* __restrict__ g, const float* __restrict__ b,
            __nv_bfloat16* __restrict__ y, uint32_t M_max, uint32_t d, const uint32_t* __restrict__ m_seq_dev,
            uint32_t rows_per_seq, float eps) {
  griddep_sync();
  uint32_t M = M_max;
  if (m_seq_dev) {
    const unsigned long long m = (unsigned long long)(*m_seq_dev) * rows_per_seq;
    M = m < M_max ? (uint32_t)m : M_max;
  }
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
  for (uint32_t row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < M; row += warps) {
    const uint32_t* xr = reinterpret_cast<const uint32_t*>(x + (size_t)row * d);
    float s = 0.f;
    for (uint32_t c = lane; c < d / 2; c += 32) {
      const uint32_t w = xr[c];
      s += __uint_as_float(w << 16) + __uint_as_float(w & 0xFFFF0000u);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    const float mu = s / (float)d;
    float v = 0.f;
    for (uint32_t c = lane; c < d / 2; c += 32) {
      const uint32_t w = xr[c];
      const float a0 = __uint_as_float(w << 16) - mu, a1 = __uint_as_float(w & 0xFFFF0000u) - mu;
      v = fmaf(a0, a0, v);
      v = fmaf(a1, a1, v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const float rstd = 1.0f / sqrtf(v / (float)d + eps);
    uint32_t* yr = reinterpret_cast<uint32_t*>(y + (size_t)row * d);
    for (uint32_t c = lane; c < d / 2; c += 32) {
      const uint32_t w = xr[c];
      const float a0 = (__uint_as_float(w << 16) - mu) * rstd * g[2 * c] + b[2 * c];
      const float a1 = (__uint_as_float(w & 0xFFFF0000u) - mu) * rstd * g[2 * c + 1] + b[2 * c + 1];
      const __nv_bfloat162 o2 = __floats2bfloat162_rn(a0, a1);
      yr[c] = *reinterpret_cast<const uint32_t*>(&o2);
    }
  }
}

// ---------------------------------------------------------------------------
// Multi-head scaled dot-product self-attention, head size 64, on tensor cores (mma.sync m16n8k16,
// bf16 inputs, fp32 accumulation).  One block of 4 warps per (sequence, head, tile of 64 queries);
// a warp owns 16 query rows.  Keys and values pass through shared memory in tiles of 64 positions
// (cp.async, double-buffered; 16-byte chunks XOR-swizzled by row so that ldmatrix is conflict-free); S = Q K^T stays in
// registers, softmax is computed on line (running maximum and sum per row), P is re-used as the A
// operand of P V straight from the accumulator layout.  causal: position i attends to j <= i.
// qkv: [tokens, 3d] (q | k | v per token); out: [tokens, d].
// ---------------------------------------------------------------------------
constexpr int ATT_DH = 64, ATT_Q = 64, ATT_KT = 64, ATT_THREADS = 128;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
// byte offset of 16-byte chunk `c` (0..7) of row `r` in a [64][64] bf16 tile
__device__ __forceinline__ uint32_t tile_off(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }

__global__ void __launch_bounds__(ATT_THREADS, 4)
k_attention(const __nv_bfloat16* __restrict__ qkv, __nv_bfloat16* __restrict__ out, uint32_t n, uint32_t d,
            uint32_t heads, uint32_t seq_max, const uint32_t* __restrict__ m_seq_dev, int causal) {
  griddep_sync();
  __shared__ __align__(128) uint8_t sq[ATT_Q * 128], sk[2][ATT_KT * 128], sv[2][ATT_KT * 128];   // K/V double-buffered
  uint32_t n_seq = seq_max;
  if (m_seq_dev) n_seq = min(seq_max, *m_seq_dev);
  const uint32_t qtiles = (n + ATT_Q - 1) / ATT_Q;
  const uint32_t seq = blockIdx.x / (heads * qtiles);
  if (seq >= n_seq) return;                                       // uniform over the block
  const uint32_t rem = blockIdx.x % (heads * qtiles);
  const uint32_t h = rem / qtiles, qt = rem % qtiles;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  const size_t tok0 = (size_t)seq * n;
  const uint32_t q0 = qt * ATT_Q;

  // stage a [64 rows][64] bf16 tile (rows of `which` = 0: q, 1: k, 2: v, starting at position p0)
  auto stage = [&](uint8_t* dst, uint32_t which, uint32_t p0) {
    for (uint32_t idx = threadIdx.x; idx < 64 * 8; idx += ATT_THREADS) {
      const uint32_t r = idx >> 3, c = idx & 7u;
      uint4 w = make_uint4(0, 0, 0, 0);
      if (p0 + r < n) w = *reinterpret_cast<const uint4*>(qkv + (tok0 + p0 + r) * 3 * d + which * d + h * ATT_DH + c * 8);
      *reinterpret_cast<uint4*>(dst + tile_off(r, c)) = w;
    }
  };
  // same, asynchronously (cp.async, 16 bytes per copy); rows beyond the sequence are zero-filled
  auto stage_async = [&](uint8_t* dst, uint32_t which, uint32_t p0) {
    for (uint32_t idx = threadIdx.x; idx < 64 * 8; idx += ATT_THREADS) {
      const uint32_t r = idx >> 3, c = idx & 7u;
      const uint32_t sa = smem_u32_of(dst) + tile_off(r, c);
      if (p0 + r < n) {
        const __nv_bfloat16* src = qkv + (tok0 + p0 + r) * 3 * d + which * d + h * ATT_DH + c * 8;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(src) : "memory");
      } else {
        *reinterpret_cast<uint4*>(dst + tile_off(r, c)) = make_uint4(0, 0, 0, 0);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  stage(sq, 0, q0);
  __syncthreads();
  // Q fragments of this warp's 16 rows: 4 k-steps of 16 head dims
  uint32_t qa[4][4];
  {
    const uint32_t row = warp * 16 + (lane & 7u) + ((lane >> 3) & 1u) * 8;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) ldsm_x4(smem_u32_of(sq) + tile_off(row, ks * 2 + (lane >> 4)), qa[ks]);
  }
  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const uint32_t row_g[2] = {q0 + warp * 16 + g, q0 + warp * 16 + g + 8};          // the two query rows of this thread
  const uint32_t last_q = min(n, q0 + ATT_Q) - 1;
  const uint32_t j_end = causal ? last_q + 1 : n;
  const float scale = 0.125f;                                                       // 1 / sqrt(64)

  stage_async(sk[0], 1, 0);
  stage_async(sv[0], 2, 0);
  uint32_t cur = 0;
  for (uint32_t j0 = 0; j0 < j_end; j0 += ATT_KT, cur ^= 1u) {
    // fetch the next tile into the other buffer while this one is used
    if (j0 + ATT_KT < j_end) {
      stage_async(sk[cur ^ 1u], 1, j0 + ATT_KT);
      stage_async(sv[cur ^ 1u], 2, j0 + ATT_KT);
      asm volatile("cp.async.wait_group 2;" ::: "memory");          // the two groups of the current tile are done
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const uint8_t* skc = sk[cur];
    const uint8_t* svc = sv[cur];
    // S = Q K^T for 16 rows x 64 keys
    float sacc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {                                              // pairs of 8-key tiles
        uint32_t kb[4];
        const uint32_t mi = lane >> 3;
        const uint32_t krow = np * 16 + (mi >> 1) * 8 + (lane & 7u);
        ldsm_x4(smem_u32_of(skc) + tile_off(krow, ks * 2 + (mi & 1u)), kb);
        mma_bf16_16816(sacc[np * 2], qa[ks], kb[0], kb[1]);
        mma_bf16_16816(sacc[np * 2 + 1], qa[ks], kb[2], kb[3]);
      }
    }
    // scale, mask, on-line softmax (rows g and g + 8; a row is spread over the 4 threads of a quad)
    float m_new[2] = {m_run[0], m_run[1]};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t key = j0 + i * 8 + t4 * 2 + (e & 1);
        const uint32_t qrow = row_g[e >> 1];
        const bool ok = key < n && (!causal || key <= qrow);
        const float v = ok ? sacc[i][e] * scale : -INFINITY;
        sacc[i][e] = v;
        m_new[e >> 1] = fmaxf(m_new[e >> 1], v);
      }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      m_new[r] = fmaxf(m_new[r], __shfl_xor_sync(0xFFFFFFFFu, m_new[r], 1));
      m_new[r] = fmaxf(m_new[r], __shfl_xor_sync(0xFFFFFFFFu, m_new[r], 2));
    }
    float corr[2], psum[2] = {0.f, 0.f};
#pragma unroll
    for (int r = 0; r < 2; ++r) corr[r] = (m_new[r] == -INFINITY) ? 1.f : __expf(m_run[r] - m_new[r]);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = e >> 1;
        const float p = (m_new[r] == -INFINITY) ? 0.f : __expf(sacc[i][e] - m_new[r]);
        sacc[i][e] = p;
        psum[r] += p;
      }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      psum[r] += __shfl_xor_sync(0xFFFFFFFFu, psum[r], 1);
      psum[r] += __shfl_xor_sync(0xFFFFFFFFu, psum[r], 2);
      l_run[r] = l_run[r] * corr[r] + psum[r];
      m_run[r] = m_new[r];
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) { o[i][0] *= corr[0]; o[i][1] *= corr[0]; o[i][2] *= corr[1]; o[i][3] *= corr[1]; }
    // O += P V : P from the accumulator layout, V through transposed ldmatrix
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {                                                // 16 keys per step
      uint32_t pa[4];
      pa[0] = pack2_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
      pa[1] = pack2_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
      pa[2] = pack2_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
      pa[3] = pack2_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
      for (int np = 0; np < 4; ++np) {                                              // pairs of 8-wide head-dim tiles
        uint32_t vb[4];
        const uint32_t mi = lane >> 3;
        const uint32_t vrow = kk * 16 + (mi & 1u) * 8 + (lane & 7u);
        ldsm_x4_t(smem_u32_of(svc) + tile_off(vrow, np * 2 + (mi >> 1)), vb);
        mma_bf16_16816(o[np * 2], pa, vb[0], vb[1]);
        mma_bf16_16816(o[np * 2 + 1], pa, vb[2], vb[3]);
      }
    }
    __syncthreads();                                                 // all warps are done with this buffer
  }
  // normalise and store: thread holds rows g, g+8, columns i*8 + 2*t4 .. +1
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    if (row_g[r] < n) {
      const float inv = 1.0f / l_run[r];
      uint32_t* op = reinterpret_cast<uint32_t*>(out + (tok0 + row_g[r]) * d + h * ATT_DH);
#pragma unroll
      for (int i = 0; i < 8; ++i) op[i * 4 + t4] = pack2_bf16(o[i][2 * r] * inv, o[i][2 * r + 1] * inv);
    }
  }
}

cudaError_t launch_layernorm(const __nv_bfloat16* x, const float* g, const float* b, __nv_bfloat16* y, uint32_t M_max,
                             uint32_t d, const uint32_t* m_seq_dev, uint32_t rows_per_seq, float eps, int sm_count,
                             cudaStream_t st) {
  if (M_max == 0) return cudaSuccess;
  unsigned long long blocks = ((unsigned long long)M_max + 7) / 8;           // 8 warps (rows) per block
  const unsigned long long cap = (unsigned long long)sm_count * 8;
  if (blocks > cap) blocks = cap;
  return launch_k(k_layernorm, dim3((uint32_t)blocks), dim3(256), 0, st, x, g, b, y, M_max, d, m_seq_dev,
                  rows_per_seq, eps);
}

cudaError_t launch_attention(const __nv_bfloat16* qkv, __nv_bfloat16* out, uint32_t n, uint32_t d, uint32_t heads,
                             uint32_t seq_max, const uint32_t* m_seq_dev, int causal, cudaStream_t st) {
  if (seq_max == 0) return cudaSuccess;
  const uint32_t qtiles = (n + ATT_Q - 1) / ATT_Q;
  return launch_k(k_attention, dim3(seq_max * heads * qtiles), dim3(ATT_THREADS), 0, st, qkv, out, n, d, heads, seq_max,
                  m_seq_dev, causal);
}

}  // namespace llmc
