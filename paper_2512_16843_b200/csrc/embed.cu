// h_0 <- E(X), the first assignment of Algorithm 1 after the fingerprint: the hidden states that enter layer 1 are
// the token embeddings of the sequence plus the position embeddings, followed (BERT-style models) by a layer
// norm over the model width.  One warp per token: the two table rows are read once (16-byte loads), summed in
// fp32 and kept in registers for the mean, the variance and the output; HBM-bound (per token d * 2 bytes read
// from each table, d * 2 written).
#include "llmcache.h"
#include "llmcache_internal.cuh"
#include "ptx.cuh"
#include "layer.cuh"

namespace llmc {

namespace {

// CH: 16-byte chunks of a row per lane (the row stays in registers); 0: any width, the sum is formed three times
template <int CH>
__global__ void __launch_bounds__(256)
k_embed(const long long* __restrict__ tokens, const __nv_bfloat16* __restrict__ tok_emb,
        const __nv_bfloat16* __restrict__ pos_emb, const float* __restrict__ gain, const float* __restrict__ bias,
        __nv_bfloat16* __restrict__ h0, uint32_t* __restrict__ bad_ids, unsigned long long rows, uint32_t n, uint32_t d,
        long long vocab, int layer_norm, float eps) {
  griddep_sync();
  const uint32_t lane = threadIdx.x & 31;
  const unsigned long long warps = ((unsigned long long)gridDim.x * blockDim.x) >> 5;
  const uint32_t nch = d / 8;
  for (unsigned long long row = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; row < rows; row += warps) {
    const long long id = tokens[row];
    uint4* out = reinterpret_cast<uint4*>(h0 + row * d);
    if (id < 0 || id >= vocab) {                          // not a token of the table: a row of zeros, counted
      for (uint32_t c = lane; c < nch; c += 32) out[c] = make_uint4(0, 0, 0, 0);
      if (lane == 0 && bad_ids) atomicAdd(bad_ids, 1u);
      continue;
    }
    const uint4* er = reinterpret_cast<const uint4*>(tok_emb + (size_t)id * d);
    const uint4* pr = pos_emb ? reinterpret_cast<const uint4*>(pos_emb + (size_t)(row % n) * d) : nullptr;
    // the eight sums of chunk c
    auto chunk = [&](uint32_t c, float (&x)[8]) {
      const uint4 e = ld_nc16(er + c);
      const uint4 p = pr ? ld_nc16(pr + c) : make_uint4(0, 0, 0, 0);
      const uint32_t ew[4] = {e.x, e.y, e.z, e.w}, pw[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        x[2 * u] = __uint_as_float(ew[u] << 16) + __uint_as_float(pw[u] << 16);
        x[2 * u + 1] = __uint_as_float(ew[u] & 0xFFFF0000u) + __uint_as_float(pw[u] & 0xFFFF0000u);
      }
    };
    auto emit = [&](uint32_t c, const float (&x)[8], float mu, float rstd) {
      float y[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        y[u] = (x[u] - mu) * rstd;
        if (layer_norm) {
          if (gain) y[u] *= gain[c * 8 + u];
          if (bias) y[u] += bias[c * 8 + u];
        }
      }
      uint32_t o[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const __nv_bfloat162 t = __floats2bfloat162_rn(y[2 * u], y[2 * u + 1]);
        o[u] = *reinterpret_cast<const uint32_t*>(&t);
      }
      out[c] = make_uint4(o[0], o[1], o[2], o[3]);
    };
    if constexpr (CH > 0) {
      float x[CH][8];
#pragma unroll
      for (int i = 0; i < CH; ++i) {
        if (lane + 32u * i < nch) chunk(lane + 32u * i, x[i]);
        else {
#pragma unroll
          for (int u = 0; u < 8; ++u) x[i][u] = 0.f;
        }
      }
      float mu = 0.f, rstd = 1.f;
      if (layer_norm) {
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < CH; ++i)
#pragma unroll
          for (int u = 0; u < 8; ++u) s += x[i][u];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        mu = s / (float)d;
        float v = 0.f;
#pragma unroll
        for (int i = 0; i < CH; ++i)
          if (lane + 32u * i < nch) {
#pragma unroll
            for (int u = 0; u < 8; ++u) v = fmaf(x[i][u] - mu, x[i][u] - mu, v);
          }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        rstd = 1.0f / sqrtf(v / (float)d + eps);
      }
#pragma unroll
      for (int i = 0; i < CH; ++i)
        if (lane + 32u * i < nch) emit(lane + 32u * i, x[i], mu, rstd);
    } else {
      float mu = 0.f, rstd = 1.f;
      if (layer_norm) {
        float s = 0.f;
        for (uint32_t c = lane; c < nch; c += 32) {
          float x[8];
          chunk(c, x);
#pragma unroll
          for (int u = 0; u < 8; ++u) s += x[u];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        mu = s / (float)d;
        float v = 0.f;
        for (uint32_t c = lane; c < nch; c += 32) {
          float x[8];
          chunk(c, x);
#pragma unroll
          for (int u = 0; u < 8; ++u) v = fmaf(x[u] - mu, x[u] - mu, v);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        rstd = 1.0f / sqrtf(v / (float)d + eps);
      }
      for (uint32_t c = lane; c < nch; c += 32) {
        float x[8];
        chunk(c, x);
        emit(c, x, mu, rstd);
      }
    }
  }
}

}  // namespace

cudaError_t launch_embed(const long long* tokens, const __nv_bfloat16* tok_emb, const __nv_bfloat16* pos_emb,
                         const float* gain, const float* bias, __nv_bfloat16* h0, uint32_t* bad_ids,
                         unsigned long long rows, uint32_t n, uint32_t d, long long vocab, int layer_norm, float eps,
                         int sm_count, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  unsigned long long blocks = (rows + 7) / 8;                                  // 8 warps (tokens) per block
  const unsigned long long cap = (unsigned long long)sm_count * 8;
  if (blocks > cap) blocks = cap;
  auto kern = d <= 1024 ? k_embed<4> : d <= 2048 ? k_embed<8> : k_embed<0>;
  return launch_k(kern, dim3((uint32_t)blocks), dim3(256), 0, st, tokens, tok_emb, pos_emb, gain, bias, h0, bad_ids, rows,
                  n, d, vocab, layer_norm, eps);
}

}  // namespace llmc

extern "C" int llmcache_embed(const int64_t* tokens, uint64_t n_seqs, uint32_t seq_len, uint32_t d_model, int64_t vocab,
                              const void* tok_emb, const void* pos_emb, int32_t layer_norm, const float* ln_gain,
                              const float* ln_bias, float ln_eps, void* h0, uint32_t* bad_ids, void* stream) {
  if (vocab <= 0 || seq_len == 0) return LLMCACHE_ERR_ARG;
  if (d_model == 0 || d_model % 8 != 0 || d_model > 16384) return LLMCACHE_ERR_SHAPE;
  if (n_seqs == 0) return LLMCACHE_OK;                     // an empty batch has no buffers to check
  if (!tokens || !tok_emb || !h0) return LLMCACHE_ERR_ARG;
  const uintptr_t al = (uintptr_t)tok_emb | (uintptr_t)pos_emb | (uintptr_t)h0 | (uintptr_t)ln_gain | (uintptr_t)ln_bias;
  if ((al & 15u) || ((uintptr_t)tokens & 7u) || ((uintptr_t)bad_ids & 3u)) return LLMCACHE_ERR_ARG;
  if (layer_norm && !(ln_eps >= 0.f)) return LLMCACHE_ERR_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return LLMCACHE_ERR_CUDA;
  const cudaError_t e = llmc::launch_embed(
      reinterpret_cast<const long long*>(tokens), static_cast<const __nv_bfloat16*>(tok_emb),
      static_cast<const __nv_bfloat16*>(pos_emb), ln_gain, ln_bias, static_cast<__nv_bfloat16*>(h0), bad_ids,
      (unsigned long long)n_seqs * seq_len, seq_len, d_model, (long long)vocab, layer_norm ? 1 : 0, ln_eps, sms,
      static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? LLMCACHE_OK : LLMCACHE_ERR_CUDA;
}

