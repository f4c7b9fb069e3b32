// The transformer layer f_l that runs on the misses (Sec. IV-A: h_l = f_l(h_{l-1}); Algorithm 1
// else-branch).  Plain layer kernels: the four dense layers are layer_gemm.cu, multi-head self-attention is
// layer_attn.cu; here is layer normalisation.
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
// WPL > 0: the row (at most 64 * WPL elements) is read once, with 16-byte loads, and kept in registers for the
// mean, the variance and the output; WPL == 0: any width, the row is read three times (from L1/L2).
// ---------------------------------------------------------------------------
template <int WPL>
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
    if constexpr (WPL > 0) {
      // lane l holds the 16-byte chunks l, l + 32, ... of the row (d is a multiple of 8)
      constexpr int CH = WPL / 4;                                   // chunks per lane
      const uint32_t nch = d / 8;
      const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * d);
      uint4 w[CH];
#pragma unroll
      for (int i = 0; i < CH; ++i) w[i] = (lane + 32u * i < nch) ? ld_nc16(xr + lane + 32u * i) : make_uint4(0, 0, 0, 0);
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const uint32_t q[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) s += __uint_as_float(q[u] << 16) + __uint_as_float(q[u] & 0xFFFF0000u);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
      const float mu = s / (float)d;
      float v = 0.f;
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        if (lane + 32u * i < nch) {
          const uint32_t q[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float a0 = __uint_as_float(q[u] << 16) - mu, a1 = __uint_as_float(q[u] & 0xFFFF0000u) - mu;
            v = fmaf(a0, a0, v);
            v = fmaf(a1, a1, v);
          }
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      const float rstd = 1.0f / sqrtf(v / (float)d + eps);
      uint4* yr = reinterpret_cast<uint4*>(y + (size_t)row * d);
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        const uint32_t c8 = lane + 32u * i;
        if (c8 < nch) {
          const uint32_t q[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
          const float4 g0 = *reinterpret_cast<const float4*>(g + c8 * 8), g1 = *reinterpret_cast<const float4*>(g + c8 * 8 + 4);
          const float4 b0 = *reinterpret_cast<const float4*>(b + c8 * 8), b1 = *reinterpret_cast<const float4*>(b + c8 * 8 + 4);
          const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
          const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
          uint32_t o4[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float a0 = (__uint_as_float(q[u] << 16) - mu) * rstd * gg[2 * u] + bb[2 * u];
            const float a1 = (__uint_as_float(q[u] & 0xFFFF0000u) - mu) * rstd * gg[2 * u + 1] + bb[2 * u + 1];
            const __nv_bfloat162 o2 = __floats2bfloat162_rn(a0, a1);
            o4[u] = *reinterpret_cast<const uint32_t*>(&o2);
          }
          yr[c8] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
        }
      }
    } else {
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
}

cudaError_t launch_layernorm(const __nv_bfloat16* x, const float* g, const float* b, __nv_bfloat16* y, uint32_t M_max,
                             uint32_t d, const uint32_t* m_seq_dev, uint32_t rows_per_seq, float eps, int sm_count,
                             cudaStream_t st) {
  if (M_max == 0) return cudaSuccess;
  unsigned long long blocks = ((unsigned long long)M_max + 7) / 8;           // 8 warps (rows) per block
  const unsigned long long cap = (unsigned long long)sm_count * 8;
  if (blocks > cap) blocks = cap;
  // rows up to 1,024 (2,048) elements stay in registers: 16 (32) words per lane
  auto kern = d <= 1024 ? k_layernorm<16> : d <= 2048 ? k_layernorm<32> : k_layernorm<0>;
  return launch_k(kern, dim3((uint32_t)blocks), dim3(256), 0, st, x, g, b, y, M_max, d, m_seq_dev,
                  rows_per_seq, eps);
}

}  // namespace llmc
