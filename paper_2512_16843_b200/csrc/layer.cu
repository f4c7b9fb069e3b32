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
// Multi-head scaled dot-product self-attention, head size 64.  One block per (sequence, head, tile of
// 128 queries); a thread owns one query row (q and the output accumulator in registers); keys and
// values pass through shared memory in tiles of 64 positions as fp32; softmax is computed on line
// (running maximum and sum).  causal: position i attends to j <= i.
// qkv: [tokens, 3d] (q | k | v per token); out: [tokens, d].
// ---------------------------------------------------------------------------
constexpr int ATT_DH = 64, ATT_Q = 128, ATT_KT = 64;

__global__ void __launch_bounds__(ATT_Q)
k_attention(const __nv_bfloat16* __restrict__ qkv, __nv_bfloat16* __restrict__ out, uint32_t n, uint32_t d,
            uint32_t heads, uint32_t seq_max, const uint32_t* __restrict__ m_seq_dev, int causal) {
  griddep_sync();
  __shared__ __align__(16) float sk[ATT_KT][ATT_DH];
  __shared__ __align__(16) float sv[ATT_KT][ATT_DH];
  uint32_t n_seq = seq_max;
  if (m_seq_dev) n_seq = min(seq_max, *m_seq_dev);
  const uint32_t qtiles = (n + ATT_Q - 1) / ATT_Q;
  const uint32_t seq = blockIdx.x / (heads * qtiles);
  if (seq >= n_seq) return;                                       // uniform over the block
  const uint32_t rem = blockIdx.x % (heads * qtiles);
  const uint32_t h = rem / qtiles, qt = rem % qtiles;
  const uint32_t i = qt * ATT_Q + threadIdx.x;                    // query position
  const bool live = i < n;
  const size_t tok0 = (size_t)seq * n;
  const float scale = 0.125f;                                     // 1 / sqrt(64)

  float q[ATT_DH], acc[ATT_DH];
#pragma unroll
  for (int c = 0; c < ATT_DH; ++c) { q[c] = 0.f; acc[c] = 0.f; }
  if (live) {
    const uint4* qp = reinterpret_cast<const uint4*>(qkv + (tok0 + i) * 3 * d + h * ATT_DH);
#pragma unroll
    for (int u = 0; u < ATT_DH / 8; ++u) {
      const uint4 w = qp[u];
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        q[u * 8 + 2 * t]     = __uint_as_float(ww[t] << 16) * scale;
        q[u * 8 + 2 * t + 1] = __uint_as_float(ww[t] & 0xFFFF0000u) * scale;
      }
    }
  }
  float m_run = -INFINITY, l_run = 0.f;
  const uint32_t last_q = min(n, (qt + 1) * ATT_Q) - 1;
  const uint32_t j_end = causal ? last_q + 1 : n;                 // keys any query of this tile can see
  for (uint32_t j0 = 0; j0 < j_end; j0 += ATT_KT) {
    __syncthreads();
    // stage K and V rows j0 .. j0+63 of this head as fp32 (zero beyond the sequence)
    for (uint32_t idx = threadIdx.x; idx < ATT_KT * (ATT_DH / 8); idx += ATT_Q) {
      const uint32_t r = idx / (ATT_DH / 8), u = idx % (ATT_DH / 8);
      const uint32_t j = j0 + r;
      uint4 kw = make_uint4(0, 0, 0, 0), vw = make_uint4(0, 0, 0, 0);
      if (j < n) {
        const __nv_bfloat16* base = qkv + (tok0 + j) * 3 * d + h * ATT_DH + u * 8;
        kw = *reinterpret_cast<const uint4*>(base + d);
        vw = *reinterpret_cast<const uint4*>(base + 2 * d);
      }
      const uint32_t k4[4] = {kw.x, kw.y, kw.z, kw.w}, v4[4] = {vw.x, vw.y, vw.z, vw.w};
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        sk[r][u * 8 + 2 * t] = __uint_as_float(k4[t] << 16);
        sk[r][u * 8 + 2 * t + 1] = __uint_as_float(k4[t] & 0xFFFF0000u);
        sv[r][u * 8 + 2 * t] = __uint_as_float(v4[t] << 16);
        sv[r][u * 8 + 2 * t + 1] = __uint_as_float(v4[t] & 0xFFFF0000u);
      }
    }
    __syncthreads();
    if (!live) continue;
    const uint32_t jmax = min((uint32_t)ATT_KT, (causal ? min(n, i + 1) : n) - min(j0, causal ? min(n, i + 1) : n));
    for (uint32_t r = 0; r < jmax; ++r) {
      float s = 0.f;
      const float4* kr = reinterpret_cast<const float4*>(sk[r]);
#pragma unroll
      for (int u = 0; u < ATT_DH / 4; ++u) {
        const float4 k4 = kr[u];
        s = fmaf(q[4 * u], k4.x, s); s = fmaf(q[4 * u + 1], k4.y, s);
        s = fmaf(q[4 * u + 2], k4.z, s); s = fmaf(q[4 * u + 3], k4.w, s);
      }
      const float m_new = fmaxf(m_run, s);
      const float corr = __expf(m_run - m_new);                  // 0 on the first key (m_run = -inf)
      const float p = __expf(s - m_new);
      l_run = l_run * corr + p;
      const float4* vr = reinterpret_cast<const float4*>(sv[r]);
#pragma unroll
      for (int u = 0; u < ATT_DH / 4; ++u) {
        const float4 v4 = vr[u];
        acc[4 * u]     = fmaf(p, v4.x, acc[4 * u] * corr);
        acc[4 * u + 1] = fmaf(p, v4.y, acc[4 * u + 1] * corr);
        acc[4 * u + 2] = fmaf(p, v4.z, acc[4 * u + 2] * corr);
        acc[4 * u + 3] = fmaf(p, v4.w, acc[4 * u + 3] * corr);
      }
      m_run = m_new;
    }
  }
  if (live) {
    const float inv = 1.0f / l_run;
    uint4* op = reinterpret_cast<uint4*>(out + (tok0 + i) * d + h * ATT_DH);
#pragma unroll
    for (int u = 0; u < ATT_DH / 8; ++u) {
      uint32_t w[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const __nv_bfloat162 o2 = __floats2bfloat162_rn(acc[u * 8 + 2 * t] * inv, acc[u * 8 + 2 * t + 1] * inv);
        w[t] = *reinterpret_cast<const uint32_t*>(&o2);
      }
      op[u] = make_uint4(w[0], w[1], w[2], w[3]);
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
  return launch_k(k_attention, dim3(seq_max * heads * qtiles), dim3(ATT_Q), 0, st, qkv, out, n, d, heads, seq_max,
                  m_seq_dev, causal);
}

}  // namespace llmc
