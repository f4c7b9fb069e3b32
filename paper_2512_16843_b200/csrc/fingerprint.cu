// Fingerprint kernels (Sec. IV-B): pooled reduction over the sequence
// positions, centring + projection, unit-length scaling, bf16 rounding.
#include "llmcache_internal.cuh"

namespace llmc {

// ---------------------------------------------------------------------------
// Pool: partial[b, s, :] = sum over the s-th slice of positions of h[b, t, :].
// grid (S, B).  A block is V x R threads: V = 16-byte vectors per row, R = rows
// taken per pass.  Every thread always owns the same E columns, so the running
// sums live in registers; the R row groups are combined through shared memory
// in a fixed order (deterministic).
// ---------------------------------------------------------------------------
template <bool BF16>
__global__ void __launch_bounds__(1024)
k_pool(const uint4* __restrict__ h, float* __restrict__ partial,
       uint32_t n, uint32_t d, uint32_t V, uint32_t R, uint32_t S, uint32_t rows_per_slice) {
  constexpr int E = BF16 ? 8 : 4;
  extern __shared__ float sm_pool[];           // [R][d]
  const uint32_t b = blockIdx.y, s = blockIdx.x;
  const uint32_t col = threadIdx.x % V, rg = threadIdx.x / V;
  const uint32_t t0 = s * rows_per_slice;
  const uint32_t t1 = min(n, t0 + rows_per_slice);
  float acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;

  const uint4* base = h + (size_t)b * n * V + col;
  auto add = [&](const uint4& v) {
    if (BF16) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[2 * i]     += __uint_as_float(w[i] << 16);
        acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
      }
    } else {
      acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
      acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
    }
  };
  uint32_t t = t0 + rg;
  // four rows in flight per thread
  for (; t + 3 * R < t1; t += 4 * R) {
    uint4 v0 = ld_stream16(base + (size_t)t * V);
    uint4 v1 = ld_stream16(base + (size_t)(t + R) * V);
    uint4 v2 = ld_stream16(base + (size_t)(t + 2 * R) * V);
    uint4 v3 = ld_stream16(base + (size_t)(t + 3 * R) * V);
    add(v0); add(v1); add(v2); add(v3);
  }
  for (; t < t1; t += R) add(ld_stream16(base + (size_t)t * V));

#pragma unroll
  for (int e = 0; e < E; ++e) sm_pool[(size_t)rg * d + col * E + e] = acc[e];
  __syncthreads();
  float* out = partial + ((size_t)b * S + s) * d;
  for (uint32_t i = threadIdx.x; i < d; i += blockDim.x) {
    float sum = 0.f;
    for (uint32_t r = 0; r < R; ++r) sum += sm_pool[(size_t)r * d + i];
    out[i] = sum;
  }
}

// ---------------------------------------------------------------------------
// Project + normalise: G sequences per block.
//   p = (sum_s partial) / n - mu ;  g = p . P  (or p when no projection)
//   q = bf16(g / ||g||) ; rq = 1 / ||q||
// ---------------------------------------------------------------------------
constexpr int PROJ_G = 4;
constexpr int PROJ_THREADS = 512;

__device__ __forceinline__ float block_sum(float v, float* red /*[32]*/) {
  // fixed-order tree: lanes by shuffle, then warps serially by thread 0
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float tot = 0.f;
  const int nw = (blockDim.x + 31) >> 5;
  for (int i = 0; i < nw; ++i) tot += red[i];
  return tot;
}

__global__ void __launch_bounds__(PROJ_THREADS)
k_project(const float* __restrict__ partial, const __nv_bfloat16* __restrict__ proj,
          const float* __restrict__ center, __nv_bfloat16* __restrict__ fp, float* __restrict__ rq,
          uint32_t B, uint32_t n, uint32_t d, uint32_t k, uint32_t S) {
  extern __shared__ float sm[];
  float* p = sm;                               // [G][d]
  float* g = p + (size_t)PROJ_G * d;           // [G][k]
  float* part = g + (size_t)PROJ_G * k;        // [slices][G][k]  (only with projection)
  __shared__ float red[32];
  const uint32_t b0 = blockIdx.x * PROJ_G;
  const float fn = (float)n;

  for (uint32_t idx = threadIdx.x; idx < PROJ_G * d; idx += blockDim.x) {
    const uint32_t gi = idx / d, i = idx - gi * d;
    const uint32_t b = b0 + gi;
    float v = 0.f;
    if (b < B) {
      const float* src = partial + (size_t)b * S * d + i;
      for (uint32_t s = 0; s < S; ++s) v += src[(size_t)s * d];
      v = v / fn;
      if (center) v -= center[i];
    }
    p[idx] = v;
  }
  __syncthreads();

  if (proj) {
    const uint32_t ncol2 = k >> 1;
    const uint32_t slices = ncol2 >= blockDim.x ? 1u : blockDim.x / ncol2;
    const uint32_t active = ncol2 >= blockDim.x ? blockDim.x : slices * ncol2;
    if (threadIdx.x < active) {
      const uint32_t sl = ncol2 >= blockDim.x ? 0u : threadIdx.x / ncol2;
      const uint32_t c2_0 = ncol2 >= blockDim.x ? threadIdx.x : threadIdx.x % ncol2;
      const uint32_t dper = (d + slices - 1) / slices;
      const uint32_t i0 = sl * dper, i1 = min(d, i0 + dper);
      for (uint32_t c2 = c2_0; c2 < ncol2; c2 += (ncol2 >= blockDim.x ? blockDim.x : ncol2)) {
        float a0[PROJ_G], a1[PROJ_G];
#pragma unroll
        for (int gi = 0; gi < PROJ_G; ++gi) { a0[gi] = 0.f; a1[gi] = 0.f; }
        const uint32_t* col = reinterpret_cast<const uint32_t*>(proj) + c2;
#pragma unroll 8
        for (uint32_t i = i0; i < i1; ++i) {
          const uint32_t w = __ldg(col + (size_t)i * ncol2);
          const float w0 = __uint_as_float(w << 16), w1 = __uint_as_float(w & 0xFFFF0000u);
#pragma unroll
          for (int gi = 0; gi < PROJ_G; ++gi) {
            const float x = p[gi * d + i];
            a0[gi] = fmaf(x, w0, a0[gi]);
            a1[gi] = fmaf(x, w1, a1[gi]);
          }
        }
#pragma unroll
        for (int gi = 0; gi < PROJ_G; ++gi) {
          part[((size_t)sl * PROJ_G + gi) * k + 2 * c2]     = a0[gi];
          part[((size_t)sl * PROJ_G + gi) * k + 2 * c2 + 1] = a1[gi];
        }
      }
    }
    __syncthreads();
    for (uint32_t idx = threadIdx.x; idx < PROJ_G * k; idx += blockDim.x) {
      float v = 0.f;
      for (uint32_t sl = 0; sl < slices; ++sl) v += part[(size_t)sl * PROJ_G * k + idx];
      g[idx] = v;
    }
    __syncthreads();
  } else {
    g = p;                                      // identity: k == d
  }

  for (int gi = 0; gi < PROJ_G; ++gi) {
    const uint32_t b = b0 + gi;
    if (b >= B) break;                          // uniform across the block
    const float* gv = g + (size_t)gi * k;
    float ss = 0.f;
    for (uint32_t c = threadIdx.x; c < k; c += blockDim.x) ss = fmaf(gv[c], gv[c], ss);
    ss = block_sum(ss, red);
    const float nrm = sqrtf(ss);
    const bool ok = isfinite(ss) && nrm >= 1e-20f;
    float qs = 0.f;
    __nv_bfloat16* dst = fp + (size_t)b * k;
    for (uint32_t c = threadIdx.x; c < k; c += blockDim.x) {
      __nv_bfloat16 q = __float2bfloat16_rn(ok ? gv[c] / nrm : 0.f);
      dst[c] = q;
      const float qf = __bfloat162float(q);
      qs = fmaf(qf, qf, qs);
    }
    qs = block_sum(qs, red);
    if (threadIdx.x == 0) rq[b] = (ok && qs > 0.f) ? 1.0f / sqrtf(qs) : 0.f;
  }
}

// rq[b] = 1/||fp[b]|| for fingerprints supplied by the caller; one warp per row.
__global__ void k_rownorm(const __nv_bfloat16* __restrict__ fp, uint32_t B, uint32_t k, float* __restrict__ rq) {
  const uint32_t row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const uint32_t lane = threadIdx.x & 31;
  if (row >= B) return;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(fp + (size_t)row * k);
  float ss = 0.f;
  for (uint32_t c = lane; c < (k >> 1); c += 32) {
    const uint32_t w = src[c];
    const float a = __uint_as_float(w << 16), b = __uint_as_float(w & 0xFFFF0000u);
    ss = fmaf(a, a, ss);
    ss = fmaf(b, b, ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  if (lane == 0) {
    const float nrm = sqrtf(ss);
    rq[row] = (isfinite(ss) && nrm >= 1e-20f) ? 1.0f / nrm : 0.f;
  }
}

// ---------------------------------------------------------------------------
size_t project_smem_bytes(uint32_t d, uint32_t k, bool has_proj) {
  uint32_t slices = 1;
  if (has_proj && (k / 2) < (uint32_t)PROJ_THREADS) slices = PROJ_THREADS / (k / 2);
  return ((size_t)PROJ_G * d + (has_proj ? (size_t)PROJ_G * k + (size_t)slices * PROJ_G * k : 0)) * sizeof(float);
}

cudaError_t setup_fingerprint_kernels() {
  return cudaFuncSetAttribute(k_project, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

uint32_t pool_split_for(uint32_t B, uint32_t n, int sm_count, uint32_t R) {
  // aim for >= 4 blocks per SM, never slices shorter than 4 passes of R rows
  uint32_t want = (uint32_t)((4 * sm_count + B - 1) / (B ? B : 1));
  uint32_t max_by_len = n / (4 * R) ? n / (4 * R) : 1;
  uint32_t S = want < 1 ? 1 : want;
  if (S > max_by_len) S = max_by_len;
  if (S > (uint32_t)POOL_MAX_SPLIT) S = POOL_MAX_SPLIT;
  return S;
}

cudaError_t launch_fingerprint(llmcache_bank* bk, const void* h_in, uint32_t B,
                               __nv_bfloat16* fp, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const bool bf16 = D.hidden_dtype == LLMCACHE_BF16;
  const uint32_t d = D.d_model, n = D.seq_len, k = D.fp_dim;
  const uint32_t V = bf16 ? d / 8 : d / 4;
  uint32_t R = 512 / V; if (R < 1) R = 1;
  if (R > n) R = n;
  const uint32_t S = pool_split_for(B, n, bk->sm_count, R);
  const uint32_t rows_per_slice = (n + S - 1) / S;
  const uint32_t S_eff = (n + rows_per_slice - 1) / rows_per_slice;
  dim3 grid(S_eff, B);
  const size_t smem = (size_t)R * d * sizeof(float);
  {
  ProfScope prof(bk, LLMCACHE_K_POOL, st);
  if (bf16)
    k_pool<true><<<grid, V * R, smem, st>>>((const uint4*)h_in, bk->a.pool_partial, n, d, V, R, S_eff, rows_per_slice);
  else
    k_pool<false><<<grid, V * R, smem, st>>>((const uint4*)h_in, bk->a.pool_partial, n, d, V, R, S_eff, rows_per_slice);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  const size_t smem2 = project_smem_bytes(d, k, bk->a.proj != nullptr);
  ProfScope prof(bk, LLMCACHE_K_PROJECT, st);
  k_project<<<(B + PROJ_G - 1) / PROJ_G, PROJ_THREADS, smem2, st>>>(
      bk->a.pool_partial, bk->a.proj, bk->a.center, fp, rq, B, n, d, k, S_eff);
  return cudaGetLastError();
}

cudaError_t launch_rownorm(llmcache_bank* bk, const __nv_bfloat16* fp, uint32_t B, uint32_t k, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  ProfScope prof(bk, LLMCACHE_K_ROWNORM, st);
  k_rownorm<<<(B + 7) / 8, 256, 0, st>>>(fp, B, k, rq);
  return cudaGetLastError();
}

}  // namespace llmc

// ---------------------------------------------------------------------------
// Fingerprint without any allocation: the pooled partial sums go to a fixed
// array that is part of the loaded library image instead of a bank's scratch.
// ---------------------------------------------------------------------------
#include <mutex>
#include <cstdio>

namespace {

// Partial sums of the pooling pass, [B, splits, d] floats.  8 MiB per GPU that loads the library.
static __device__ __align__(256) float g_fp_static_scratch[LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS];

constexpr int STATIC_MAX_DEVICES = 64;
struct StaticDev { bool ready = false; float* scratch = nullptr; int sm_count = 0; };
StaticDev g_static_dev[STATIC_MAX_DEVICES];
std::mutex g_static_mu;
thread_local char g_static_err[192] = "";

// Once per device, with that device current: resolve the device address of the array (its name is
// only a host-side handle) and raise the projection kernel's shared-memory limit.
cudaError_t static_setup(int dev, StaticDev** out) {
  std::lock_guard<std::mutex> lock(g_static_mu);
  StaticDev& sd = g_static_dev[dev];
  if (!sd.ready) {
    float* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_fp_static_scratch);
    if (e != cudaSuccess) return e;
    if (!ptr) return cudaErrorInvalidSymbol;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = llmc::setup_fingerprint_kernels();
    if (e != cudaSuccess) return e;
    sd.scratch = ptr;
    sd.sm_count = sms;
    sd.ready = true;
  }
  *out = &sd;
  return cudaSuccess;
}

}  // namespace

extern "C" const char* llmcache_fingerprint_static_error(void) { return g_static_err; }

extern "C" int llmcache_fingerprint_static(const void* h_in, uint32_t hidden_dtype, uint32_t B, uint32_t seq_len,
                                           uint32_t d_model, uint32_t fp_dim, const void* proj,
                                           const float* center, void* fp, float* rq, void* stream) {
  using namespace llmc;
  g_static_err[0] = 0;
  auto fail = [&](int rc, const char* msg) { std::snprintf(g_static_err, sizeof(g_static_err), "%s", msg); return rc; };
  if (hidden_dtype != LLMCACHE_F32 && hidden_dtype != LLMCACHE_BF16) return fail(LLMCACHE_ERR_ARG, "unknown hidden_dtype");
  if (B && (!h_in || !fp || !rq)) return fail(LLMCACHE_ERR_ARG, "null input or output pointer");
  if (((uintptr_t)h_in | (uintptr_t)fp | (uintptr_t)proj | (uintptr_t)center) & 15u)
    return fail(LLMCACHE_ERR_ARG, "pointers must be 16-byte aligned");
  const bool bf16 = hidden_dtype == LLMCACHE_BF16;
  const uint32_t d = d_model, n = seq_len, k = fp_dim;
  if (n == 0 || d == 0 || d % 8 != 0 || d > (bf16 ? 8192u : 4096u)) return fail(LLMCACHE_ERR_SHAPE, "d_model not supported");
  if (k == 0 || k % 64 != 0 || k > 2048 || (!proj && k != d)) return fail(LLMCACHE_ERR_SHAPE, "fp_dim not supported");
  if (project_smem_bytes(d, k, proj != nullptr) > 200 * 1024) return fail(LLMCACHE_ERR_UNSUPPORTED, "d_model + fp_dim too large");
  if (B == 0) return LLMCACHE_OK;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) {
    cudaGetLastError();
    return fail(LLMCACHE_ERR_CUDA, "no current CUDA device");
  }
  StaticDev* sd = nullptr;
  cudaError_t e = static_setup(dev, &sd);
  if (e != cudaSuccess) { cudaGetLastError(); return fail(LLMCACHE_ERR_CUDA, cudaGetErrorString(e)); }

  const uint32_t V = bf16 ? d / 8 : d / 4;
  uint32_t R = 512 / V; if (R < 1) R = 1;
  if (R > n) R = n;
  const uint32_t S = pool_split_for(B, n, sd->sm_count, R);
  const uint32_t rows_per_slice = (n + S - 1) / S;
  const uint32_t S_eff = (n + rows_per_slice - 1) / rows_per_slice;
  if ((unsigned long long)B * S_eff * d > (unsigned long long)LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS) {
    std::snprintf(g_static_err, sizeof(g_static_err),
                  "batch too large for the fixed scratch: B * splits * d_model = %llu floats, limit %llu",
                  (unsigned long long)B * S_eff * d, (unsigned long long)LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS);
    return LLMCACHE_ERR_SHAPE;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // every partial sum that the second kernel reads is written by the first one in this call, so
  // nothing in the shared array has to start at zero
  dim3 grid(S_eff, B);
  const size_t smem = (size_t)R * d * sizeof(float);
  if (bf16)
    k_pool<true><<<grid, V * R, smem, st>>>((const uint4*)h_in, sd->scratch, n, d, V, R, S_eff, rows_per_slice);
  else
    k_pool<false><<<grid, V * R, smem, st>>>((const uint4*)h_in, sd->scratch, n, d, V, R, S_eff, rows_per_slice);
  e = cudaGetLastError();
  if (e == cudaSuccess) {
    k_project<<<(B + PROJ_G - 1) / PROJ_G, PROJ_THREADS, project_smem_bytes(d, k, proj != nullptr), st>>>(
        sd->scratch, (const __nv_bfloat16*)proj, center, (__nv_bfloat16*)fp, rq, B, n, d, k, S_eff);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) return fail(LLMCACHE_ERR_CUDA, cudaGetErrorString(e));
  return LLMCACHE_OK;
}
