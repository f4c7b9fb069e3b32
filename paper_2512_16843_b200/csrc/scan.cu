// Bank scan (Sec. III-C, Sec. IV-A): cosine of every query fingerprint against
// every occupied slot, reduced on the fly to the best slot per query.  The
// B x N score matrix is never written to memory.
#include "llmcache_internal.cuh"

namespace llmc {

// Straightforward CUDA-core version: a block holds QT queries in shared memory
// (as fp32) and each thread walks one bank row.
constexpr int SCAN_QT = 16;
constexpr int SCAN_THREADS = 128;

__global__ void __launch_bounds__(SCAN_THREADS)
k_scan_simt(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ bank_fp,
            const float* __restrict__ rb, const uint8_t* __restrict__ valid,
            unsigned long long* __restrict__ best, uint32_t B, uint32_t N, uint32_t k) {
  extern __shared__ float sq[];                       // [QT][k]
  const uint32_t b0 = blockIdx.y * SCAN_QT;
  for (uint32_t idx = threadIdx.x; idx < SCAN_QT * k; idx += blockDim.x) {
    const uint32_t qi = idx / k, c = idx - qi * k;
    sq[idx] = (b0 + qi < B) ? __bfloat162float(q[(size_t)(b0 + qi) * k + c]) : 0.f;
  }
  __syncthreads();
  const uint32_t j = blockIdx.x * SCAN_THREADS + threadIdx.x;
  float acc[SCAN_QT];
#pragma unroll
  for (int i = 0; i < SCAN_QT; ++i) acc[i] = 0.f;
  const bool live = (j < N) && valid[j];
  if (live) {
    const uint4* row = reinterpret_cast<const uint4*>(bank_fp + (size_t)j * k);
    for (uint32_t c8 = 0; c8 < k / 8; ++c8) {
      const uint4 v = __ldg(row + c8);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float f0 = __uint_as_float(w[u] << 16), f1 = __uint_as_float(w[u] & 0xFFFF0000u);
        const uint32_t c = c8 * 8 + 2 * u;
#pragma unroll
        for (int i = 0; i < SCAN_QT; ++i) {
          acc[i] = fmaf(sq[i * k + c], f0, acc[i]);
          acc[i] = fmaf(sq[i * k + c + 1], f1, acc[i]);
        }
      }
    }
  }
  const float scale = live ? rb[j] : 0.f;
#pragma unroll
  for (int i = 0; i < SCAN_QT; ++i) {
    unsigned long long pk = live ? pack_best(acc[i] * scale, j) : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, pk, o);
      pk = other > pk ? other : pk;
    }
    if ((threadIdx.x & 31) == 0 && pk != 0ull && b0 + i < B) atomicMax(best + b0 + i, pk);
  }
}

cudaError_t setup_scan_kernels() {
  return cudaFuncSetAttribute(k_scan_simt, cudaFuncAttributeMaxDynamicSharedMemorySize, SCAN_QT * 2048 * 4);
}

cudaError_t launch_scan(llmcache_bank* bk, const __nv_bfloat16* q, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const uint32_t N = bk->desc.capacity, k = bk->desc.fp_dim;
  dim3 grid((N + SCAN_THREADS - 1) / SCAN_THREADS, (B + SCAN_QT - 1) / SCAN_QT);
  ProfScope prof(bk, LLMCACHE_K_SCAN, st);
  k_scan_simt<<<grid, SCAN_THREADS, (size_t)SCAN_QT * k * sizeof(float), st>>>(
      q, bk->a.fp, bk->a.rb, bk->a.valid, bk->a.best, B, N, k);
  return cudaGetLastError();
}

}  // namespace llmc
