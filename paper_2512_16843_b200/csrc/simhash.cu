// SimHash lookup (Sec. III-A, IV-B): k-bit sign codes of the fingerprints, nearest key in Hamming
// distance by XOR + population count.  Integer arithmetic only.
#include "llmcache_internal.cuh"

namespace llmc {

// code word w of row r = sign bits of elements 32w .. 32w+31 of the bf16 row (bit i = element 32w + i)
__global__ void __launch_bounds__(256)
k_pack_signs(const __nv_bfloat16* __restrict__ fp, uint32_t* __restrict__ bits, uint32_t rows, uint32_t k) {
  griddep_sync();
  const uint32_t lane = threadIdx.x & 31;
  const uint32_t words = k >> 5;
  const unsigned long long total = (unsigned long long)rows * words;
  const unsigned long long warps = ((unsigned long long)gridDim.x * blockDim.x) >> 5;
  const unsigned short* raw = reinterpret_cast<const unsigned short*>(fp);
  for (unsigned long long w = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < total; w += warps) {
    const unsigned short v = raw[w * 32 + lane];
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, (v >> 15) & 1u);
    if (lane == 0) bits[w] = word;
  }
}

// A block holds QT query codes in shared memory; a thread owns one slot.  The best (smallest distance,
// then lowest slot) per query is published with a 64-bit atomicMax on (~distance, ~slot).
constexpr int SH_QT = 32, SH_THREADS = 128;

__global__ void __launch_bounds__(SH_THREADS)
k_scan_simhash(const uint32_t* __restrict__ qbits, const uint32_t* __restrict__ bits, const uint8_t* __restrict__ valid,
               unsigned long long* __restrict__ best, uint32_t B, uint32_t N, uint32_t words) {
  griddep_sync();
  extern __shared__ uint32_t sq[];                     // [QT][words]
  const uint32_t b0 = blockIdx.y * SH_QT;
  for (uint32_t i = threadIdx.x; i < SH_QT * words; i += SH_THREADS) {
    const uint32_t qi = i / words;
    sq[i] = (b0 + qi < B) ? qbits[(size_t)(b0 + qi) * words + (i - qi * words)] : 0u;
  }
  __syncthreads();
  const uint32_t j = blockIdx.x * SH_THREADS + threadIdx.x;
  const bool live = j < N && valid[j];
  uint32_t dist[SH_QT];
#pragma unroll
  for (int q = 0; q < SH_QT; ++q) dist[q] = 0;
  if (live) {
    const uint32_t* row = bits + (size_t)j * words;
    for (uint32_t w = 0; w < words; ++w) {
      const uint32_t x = __ldg(row + w);
#pragma unroll
      for (int q = 0; q < SH_QT; ++q) dist[q] += __popc(x ^ sq[q * words + w]);
    }
  }
#pragma unroll
  for (int q = 0; q < SH_QT; ++q) {
    unsigned long long pk = live ? (((unsigned long long)(0xFFFFFFFFu - dist[q]) << 32) | (0xFFFFFFFFu - j)) : 0ull;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, pk, o);
      pk = other > pk ? other : pk;
    }
    if ((threadIdx.x & 31) == 0 && pk != 0ull && b0 + q < B) atomicMax(best + b0 + q, pk);
  }
}

cudaError_t launch_simhash_scan(llmcache_bank* bk, const __nv_bfloat16* q, uint32_t B, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const uint32_t N = bk->desc.capacity, k = bk->desc.fp_dim, words = k / 32;
  cudaError_t e = cudaSuccess;
  const uint32_t cap = (uint32_t)bk->sm_count * 8;
  if (bk->bits_dirty) {
    const unsigned long long blocks = ((unsigned long long)N * words + 7) / 8;
    e = launch_k(k_pack_signs, dim3((uint32_t)(blocks < cap ? blocks : cap)), dim3(256), 0, st,
                 (const __nv_bfloat16*)bk->a.fp, bk->a.bits, N, k);
    if (e != cudaSuccess) return e;
    bk->bits_dirty = false;
    bk->n_launches += 1;
  }
  const unsigned long long qblocks = ((unsigned long long)B * words + 7) / 8;
  e = launch_k(k_pack_signs, dim3((uint32_t)(qblocks < cap ? qblocks : cap)), dim3(256), 0, st, q, bk->a.qbits, B, k);
  if (e != cudaSuccess) return e;
  bk->n_launches += 1;
  ProfScope prof(bk, LLMCACHE_K_SCAN, st);
  dim3 grid((N + SH_THREADS - 1) / SH_THREADS, (B + SH_QT - 1) / SH_QT);
  return launch_k(k_scan_simhash, grid, dim3(SH_THREADS), (size_t)SH_QT * words * 4, st, (const uint32_t*)bk->a.qbits,
                  (const uint32_t*)bk->a.bits, (const uint8_t*)bk->a.valid, bk->a.best, B, N, words);
}

}  // namespace llmc
