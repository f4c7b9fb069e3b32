// Divergence monitor (Sec. III-E, divergence tracking of the outputs stored under a fingerprint;
// Sec. IV-D, the monitor that re-checks stored entries): for every stride-th hit of the last probe the layer is run
// again on that sequence's input and compared with the stored output it was served; entries whose
// relative L2 difference exceeds a bound are invalidated.
#include "llmcache_internal.cuh"

struct llmcache_layer;
extern "C" int llmcache_layer_forward(llmcache_layer* layer, const void* x, uint32_t n_seqs,
                                      const uint32_t* n_seqs_dev, void* out, void* stream);

namespace llmc {

// sample i <- input row of the (i * stride)-th hit; also publishes the sample count.
__global__ void __launch_bounds__(256)
k_div_gather(const uint4* __restrict__ h_in, uint4* __restrict__ h_sample, const int32_t* __restrict__ hit_idx,
             const uint32_t* __restrict__ counts, uint32_t stride, uint32_t row_vecs, uint32_t* __restrict__ n_samples) {
  griddep_sync();
  const uint32_t H = counts[0];
  const uint32_t S = (H + stride - 1) / stride;
  if (blockIdx.x == 0 && threadIdx.x == 0) *n_samples = S;
  const unsigned long long total = (unsigned long long)S * row_vecs;
  for (unsigned long long v = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; v < total;
       v += (unsigned long long)gridDim.x * blockDim.x) {
    const uint32_t i = (uint32_t)(v / row_vecs), c = (uint32_t)(v % row_vecs);
    const int32_t b = hit_idx[i * stride];
    h_sample[v] = ld_stream16(h_in + (size_t)b * row_vecs + c);
  }
}

// One block per sample: rel = ||fresh - stored|| / ||fresh||; invalidate the slot when rel > bound
// (unless the slot was re-inserted during the current tick).
__global__ void __launch_bounds__(256)
k_div_compare(const uint4* __restrict__ fresh, const uint4* __restrict__ act, uint32_t act_rows,
              const int32_t* __restrict__ hit_idx, const int32_t* __restrict__ slot, const uint32_t* __restrict__ n_samples,
              uint32_t stride, uint32_t row_vecs, float bound, float* __restrict__ rel_out, uint8_t* __restrict__ valid,
              const uint32_t* __restrict__ insert_tick, uint32_t tick, uint32_t* __restrict__ n_invalid,
              unsigned long long* __restrict__ stats) {
  griddep_sync();
  __shared__ float red[2][8];
  const uint32_t S = *n_samples;
  for (uint32_t i = blockIdx.x; i < S; i += gridDim.x) {
    const int32_t b = hit_idx[i * stride];
    const int32_t j = slot[b];
    const uint4* f = fresh + (size_t)i * row_vecs;
    const uint4* s = act + (size_t)((uint32_t)j % act_rows) * row_vecs;
    float num = 0.f, den = 0.f;
    for (uint32_t c = threadIdx.x; c < row_vecs; c += blockDim.x) {
      const uint4 a = f[c], q = s[c];
      const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, qw[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float a0 = __uint_as_float(aw[u] << 16), a1 = __uint_as_float(aw[u] & 0xFFFF0000u);
        const float d0 = a0 - __uint_as_float(qw[u] << 16), d1 = a1 - __uint_as_float(qw[u] & 0xFFFF0000u);
        num = fmaf(d0, d0, num); num = fmaf(d1, d1, num);
        den = fmaf(a0, a0, den); den = fmaf(a1, a1, den);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      num += __shfl_xor_sync(0xFFFFFFFFu, num, o);
      den += __shfl_xor_sync(0xFFFFFFFFu, den, o);
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = num; red[1][threadIdx.x >> 5] = den; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float tn = 0.f, td = 0.f;
      for (int w = 0; w < 8; ++w) { tn += red[0][w]; td += red[1][w]; }
      const float rel = td > 0.f ? sqrtf(tn) / sqrtf(td) : 0.f;
      rel_out[i] = rel;
      if (rel > bound && insert_tick[j] != tick) {
        // several samples may point at one slot: only the one that flips the flag counts
        const uint32_t word = (uint32_t)j & ~3u, sh = ((uint32_t)j & 3u) * 8;
        const uint32_t old = atomicAnd(reinterpret_cast<uint32_t*>(valid + word), ~(0xFFu << sh));
        if ((old >> sh) & 0xFFu) { atomicAdd(n_invalid, 1u); atomicAdd(stats + ST_FLUSH, 1ull); }
      }
    }
  }
}

}  // namespace llmc

extern "C" int llmcache_divergence_check(llmcache_bank_t* bk, llmcache_layer* layer, const void* h_in,
                                         const llmcache_probe_io* io, uint32_t stride, float bound, void* h_sample,
                                         void* out_sample, float* rel_out, uint32_t* counters_dev, void* stream) {
  using namespace llmc;
  if (!bk || !layer || !h_in || !io || !h_sample || !out_sample || !rel_out || !counters_dev || stride == 0)
    return LLMCACHE_ERR_ARG;
  if (!bk->a.act || bk->desc.hidden_dtype != LLMCACHE_BF16) return LLMCACHE_ERR_UNSUPPORTED;
  if (bk->probe_open && bk->last_B) return LLMCACHE_ERR_STATE;        // run it after the commit
  if (!(bound >= 0.f)) return LLMCACHE_ERR_ARG;
  const uint32_t B = bk->last_B;
  if (B == 0) return LLMCACHE_OK;
  cudaStream_t st = (cudaStream_t)stream;
  const uint32_t row_vecs = (uint32_t)(((size_t)bk->desc.seq_len * bk->desc.d_model * 2) / 16);
  const uint32_t S_max = (B + stride - 1) / stride;
  cudaError_t e = cudaMemsetAsync(counters_dev, 0, 2 * sizeof(uint32_t), st);
  if (e == cudaSuccess)
    e = launch_k(k_div_gather, dim3((uint32_t)bk->sm_count * 4), dim3(256), 0, st, (const uint4*)h_in, (uint4*)h_sample,
                 (const int32_t*)io->hit_idx, (const uint32_t*)io->counts, stride, row_vecs, counters_dev);
  if (e != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  int rc = llmcache_layer_forward(layer, h_sample, S_max, counters_dev, out_sample, stream);
  if (rc != LLMCACHE_OK) return rc;
  e = launch_k(k_div_compare, dim3(S_max < 592u ? S_max : 592u), dim3(256), 0, st, (const uint4*)out_sample,
               (const uint4*)bk->a.act, bk->desc.act_rows, (const int32_t*)io->hit_idx, (const int32_t*)io->slot,
               (const uint32_t*)counters_dev, stride, row_vecs, bound, rel_out, bk->a.valid,
               (const uint32_t*)bk->a.insert_tick, (uint32_t)bk->tick, counters_dev + 1, bk->a.stats);
  if (e != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  return LLMCACHE_OK;
}
