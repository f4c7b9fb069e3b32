// Fingerprint kernels (Sec. IV-B): pooled reduction over the sequence
// positions, centring + projection, unit-length scaling, bf16 rounding.
//
//   k_pool          the pooling pass
//   k_project       projection + rounding (from the pooling pass's partial sums or from given position
//                   means) on the tensor cores, one thread-block cluster per group of 8 sequences
//   k_normalise     the same without a projection matrix
//   k_rownorm       inverse norms of caller-supplied fingerprints
#include "llmcache_internal.cuh"
#include "ptx.cuh"
#include "fp_phases.cuh"

namespace llmc {

template <bool BF16>
__global__ void __launch_bounds__(1024, 1)
k_pool(const uint4* __restrict__ h, float* __restrict__ partial, uint32_t* __restrict__ status, PoolShape S) {
  if (!S.early) griddep_sync();
  extern __shared__ __align__(128) uint8_t sm_raw[];
  pool_phase<BF16>(sm_raw, h, partial, status, S);
}

// ---------------------------------------------------------------------------
// Projection + rounding as a kernel of its own.  One thread-block cluster of S blocks serves G
// sequences: the d rows of P are split over the S blocks, the S partial results meet in block 0's
// shared memory (distributed shared memory) and are added there in block order.  The producer thread
// starts before the preceding grid has finished: P never changes.  Every block of a cluster reaches
// both cluster barriers whatever happens.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in block `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

template <int NT>
__global__ void __launch_bounds__(PROJ_THREADS, 1)
k_project(const __grid_constant__ CUtensorMap map_p, MeanSrc src, __nv_bfloat16* __restrict__ fp, float* __restrict__ rq,
          uint32_t* __restrict__ status, uint32_t B, ProjShape S, uint32_t rows_per) {
  extern __shared__ __align__(128) uint8_t sm_raw[];
  const uint32_t CS = cluster_size(), rank = cluster_rank();
  const uint32_t b0 = (blockIdx.x / CS) * PROJ_G, k = S.k, d = src.d;
  const uint32_t r0 = min(d, rank * rows_per), nrows = min(d, r0 + rows_per) - r0;
  const ProjSmem m = proj_smem(sm_raw, S);
  if (threadIdx.x == 0) proj_init(m, S, true);
  __syncthreads();

  float vals[2 * NT];
#pragma unroll
  for (int i = 0; i < 2 * NT; ++i) vals[i] = 0.f;
  if (threadIdx.x >= PROJ_CONS) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == PROJ_CONS && !producer_idle(status)) {
      uint32_t it = 0;
      if (!proj_produce(m, S, &map_p, r0, nrows, blockIdx.x * 5u, it, wait_limit(status))) proj_drain(m, S, it, status);
    }
    __syncwarp();
  } else {
    proj_prepare(m, src, b0);
    griddep_sync();
    uint32_t it = 0;
    proj_consume<NT>(m, S, src, B, b0, r0, nrows, blockIdx.x * 5u, it, status, vals);
  }
  // every block of the cluster is done with its own ring: block 0's may now receive the CS partial results
  cluster_sync_all();
  if (threadIdx.x < PROJ_CONS) {
    const uint32_t dst0 = cluster_map(m.ring, 0) + rank * (PROJ_G * k * 4);
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const uint32_t idx = proj_val_index<NT>(k, t, e);
        if (idx != 0xFFFFFFFFu) st_cluster_f32(dst0 + idx * 4, vals[2 * t + e]);
      }
  }
  cluster_sync_all();
  if (rank != 0 || threadIdx.x >= PROJ_CONS) return;
  for (uint32_t idx = threadIdx.x; idx < PROJ_G * k; idx += PROJ_CONS) {
    float v = m.part[idx];
    for (uint32_t r = 1; r < CS; ++r) v += m.part[(size_t)r * PROJ_G * k + idx];
    m.part[idx] = v;
  }
  asm volatile("bar.sync 1, %0;" ::"n"(PROJ_CONS) : "memory");
  finish_group(m.part, k, B, b0, fp, rq);
}

__global__ void __launch_bounds__(NRM_THREADS)
k_normalise(MeanSrc src, __nv_bfloat16* __restrict__ fp, float* __restrict__ rq) {
  griddep_sync();
  extern __shared__ float nrm_sm[];              // [d] + [32]
  normalise_seq(src, blockIdx.x, nrm_sm, nrm_sm + src.d, threadIdx.x, 1, fp, rq);
}

// rq[b] = 1/||fp[b]|| for fingerprints supplied by the caller; one warp per row.
__global__ void k_rownorm(const __nv_bfloat16* __restrict__ fp, uint32_t B, uint32_t k, float* __restrict__ rq) {
  griddep_sync();
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
// Launch shapes.
// ---------------------------------------------------------------------------
constexpr uint32_t PROJ_RING_BYTES = 128 * 1024;
constexpr uint32_t PROJ_STAGE_BYTES = 32 * 1024;
constexpr uint32_t PROJ_A_ROWS = 1024;            // most rows of P per refill of the A operand

// NT: 8-column tiles per consumer warp; split: blocks (of one cluster) that share the rows of P of a group.
struct ProjPlan { int NT; uint32_t split, groups, rows_per; ProjShape shape; size_t smem; };

// max_blocks: number of blocks the groups may be spread over by splitting the rows of P (1: no splitting).
static ProjPlan proj_plan(uint32_t B, uint32_t d, uint32_t k, uint32_t max_blocks) {
  ProjPlan P;
  const uint32_t tiles = k / 8, warps = PROJ_CONS / 32;
  P.NT = 1;
  while ((uint32_t)P.NT * warps < tiles) P.NT *= 2;
  P.groups = (B + PROJ_G - 1) / PROJ_G;
  ProjShape& sh = P.shape;
  sh.k = k;
  const uint32_t row_bytes = k * 2;
  sh.stage_rows = (PROJ_STAGE_BYTES / row_bytes) / PROJ_KSTEP * PROJ_KSTEP;
  if (sh.stage_rows < PROJ_KSTEP) sh.stage_rows = PROJ_KSTEP;
  if (sh.stage_rows > 256) sh.stage_rows = 256;                                // most rows of a TMA box
  const uint32_t stage_bytes = sh.stage_rows * row_bytes;
  sh.stages = PROJ_RING_BYTES / stage_bytes;
  if (sh.stages < 2) sh.stages = 2;
  if (sh.stages > 8) sh.stages = 8;
  size_t ring = (size_t)sh.stages * stage_bytes;
  if (ring < (size_t)PROJ_G * k * 4) ring = (size_t)PROJ_G * k * 4;            // the ring is reused for the group's result
  sh.ring_bytes = (uint32_t)((ring + 127) / 128 * 128);
  sh.a_rows = PROJ_A_ROWS / sh.stage_rows * sh.stage_rows;
  if (sh.a_rows < sh.stage_rows) sh.a_rows = sh.stage_rows;
  sh.a_stride = (sh.a_rows * 2 + 127) / 128 * 128 + 16;
  // spread the rows of P over the blocks of a cluster while SMs are idle, an item keeps at least 128 rows and
  // block 0's ring can take the partial results
  uint32_t S = 1;
  while (S < 8 && (unsigned long long)P.groups * S * 2 <= (unsigned long long)max_blocks && (d + 2 * S - 1) / (2 * S) >= 128 &&
         (size_t)2 * S * PROJ_G * k * 4 <= sh.ring_bytes)
    S *= 2;
  P.split = S;
  P.rows_per = (d + S - 1) / S;
  P.smem = (size_t)SMEM_HEAD + sh.ring_bytes + (size_t)3 * PROJ_G * sh.a_stride;
  return P;
}

// Dynamic shared memory of the fingerprint's second kernel.
size_t project_smem_bytes(uint32_t d, uint32_t k, bool has_proj) {
  if (!has_proj) return (size_t)d * sizeof(float) + 128;
  return proj_plan(1, d, k, 1).smem;
}

template <int NT>
static cudaError_t set_smem_limit_nt() {
  const int lim = 220 * 1024;
  return cudaFuncSetAttribute(k_project<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
}

cudaError_t setup_fingerprint_kernels() {
  const int lim = 220 * 1024;
  cudaError_t e = tensor_map_setup();
  if (e == cudaSuccess) e = set_smem_limit_nt<1>();
  if (e == cudaSuccess) e = set_smem_limit_nt<2>();
  if (e == cudaSuccess) e = set_smem_limit_nt<4>();
  if (e == cudaSuccess) e = set_smem_limit_nt<8>();
  if (e == cudaSuccess) e = set_smem_limit_nt<16>();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_pool<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_pool<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, lim);
  return e;
}

// Launch shape of the pooling pass.  The scratch it needs is grid * Jmax * d floats, which never exceeds
// (B + 3 * POOL_MAX_GRID) * d.
PoolPlan pool_plan(uint32_t B, uint32_t n, uint32_t d, bool bf16, int sm_count) {
  PoolPlan P;
  P.V = bf16 ? d / 8 : d / 4;
  P.R = 512 / P.V; if (P.R < 1) P.R = 1;
  if (P.R > n) P.R = n;
  P.cons_threads = (P.V * P.R + 31) / 32 * 32;
  P.threads = P.cons_threads + 32;                                    // + the producer's warp
  const uint32_t row_bytes = P.V * 16;
  // a stage holds a whole number of passes of R rows, about 16 KB; the ring about 160 KB
  uint32_t passes = 16384 / (P.R * row_bytes); if (passes < 1) passes = 1;
  P.stage_rows = P.R * passes;
  const uint32_t stage_bytes = P.stage_rows * row_bytes;
  P.stages = (160 * 1024) / stage_bytes;
  if (P.stages > 16) P.stages = 16;
  if (P.stages < 2) P.stages = 2;
  const unsigned long long rows = (unsigned long long)B * n;
  unsigned long long grid = (unsigned long long)sm_count;              // one block per SM
  if (grid > POOL_MAX_GRID) grid = POOL_MAX_GRID;
  const unsigned long long min_rows = 2ull * P.stage_rows;             // keep spans long enough to pipeline
  if (grid * min_rows > rows) grid = (rows + min_rows - 1) / min_rows;
  if (grid < 1) grid = 1;
  P.L = (uint32_t)((rows + grid - 1) / grid);
  P.grid = (uint32_t)((rows + P.L - 1) / P.L);
  P.Jmax = (P.L + n - 1) / n + 1;
  P.smem = (size_t)SMEM_HEAD + (size_t)P.stages * stage_bytes + (size_t)P.R * d * sizeof(float);
  return P;
}

static PoolShape pool_shape(const PoolPlan& P, uint32_t B, uint32_t n, uint32_t d, bool early) {
  return PoolShape{B, n, d, P.V, P.R, P.L, P.Jmax, P.stage_rows, P.stages, P.cons_threads, early ? 1u : 0u};
}

static cudaError_t launch_pool(const PoolPlan& P, bool bf16, const void* h_in, float* partial, uint32_t* status,
                               uint32_t B, uint32_t n, uint32_t d, cudaStream_t st, bool early = false) {
  return launch_k(bf16 ? k_pool<true> : k_pool<false>, dim3(P.grid), dim3(P.threads), P.smem, st,
                  (const uint4*)h_in, partial, status, pool_shape(P, B, n, d, early));
}

// Second kernel of the fingerprint: from the pooling pass's partial sums (pooled == nullptr) or from given
// position means.  L, Jmax: shape of the pooling pass that wrote `partial`.
static cudaError_t launch_project(uint32_t L, uint32_t Jmax, const float* partial, const float* pooled, uint32_t ld,
                                  const __nv_bfloat16* proj, const float* center, __nv_bfloat16* fp, float* rq,
                                  uint32_t* status, uint32_t B, uint32_t n, uint32_t d, uint32_t k, int sm_count,
                                  cudaStream_t st) {
  const MeanSrc src{partial, pooled, center, ld, n, d, L, Jmax};
  if (!proj)
    return launch_k(k_normalise, dim3(B), dim3(NRM_THREADS), (size_t)d * sizeof(float) + 128, st, src, fp, rq);
  const ProjPlan P = proj_plan(B, d, k, (uint32_t)sm_count);
  alignas(64) CUtensorMap map_p;
  if (!make_tensor_map_bf16(&map_p, proj, d, k, P.shape.stage_rows)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(P.groups * P.split);
  cfg.blockDim = dim3(PROJ_THREADS);
  cfg.dynamicSmemBytes = P.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = P.split;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  auto kern = P.NT == 1 ? k_project<1> : P.NT == 2 ? k_project<2> : P.NT == 4 ? k_project<4> : P.NT == 8 ? k_project<8> : k_project<16>;
  return cudaLaunchKernelEx(&cfg, kern, map_p, src, fp, rq, status, B, P.shape, P.rows_per);
}

cudaError_t launch_fingerprint(llmcache_bank* bk, const void* h_in, uint32_t B,
                               __nv_bfloat16* fp, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const bool bf16 = D.hidden_dtype == LLMCACHE_BF16;
  const PoolPlan P = pool_plan(B, D.seq_len, D.d_model, bf16, bk->sm_count);
  cudaError_t e;
  {
    ProfScope prof(bk, LLMCACHE_K_POOL, st);
    e = launch_pool(P, bf16, h_in, bk->a.pool_partial, bk->a.status, B, D.seq_len, D.d_model, st, bk->input_stable);
  }
  if (e != cudaSuccess) return e;
  ProfScope prof(bk, LLMCACHE_K_PROJECT, st);
  return launch_project(P.L, P.Jmax, bk->a.pool_partial, nullptr, 0, bk->a.proj, bk->a.center, fp, rq, bk->a.status, B,
                        D.seq_len, D.d_model, D.fp_dim, bk->sm_count, st);
}

// Step 1a alone: position means of h_in -> pooled[b * ld + c].
cudaError_t launch_pool_only(llmcache_bank* bk, const void* h_in, uint32_t B, float* pooled, uint32_t ld, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  const bool bf16 = D.hidden_dtype == LLMCACHE_BF16;
  const PoolPlan P = pool_plan(B, D.seq_len, D.d_model, bf16, bk->sm_count);
  cudaError_t e;
  {
    ProfScope prof(bk, LLMCACHE_K_POOL, st);
    e = launch_pool(P, bf16, h_in, bk->a.pool_partial, bk->a.status, B, D.seq_len, D.d_model, st);
  }
  if (e != cudaSuccess) return e;
  return launch_pool_finish_plain(bk, P, B, pooled, ld, st);
}

// Step 1b alone: fingerprints from given position means pooled[b * ld + c], c < d.
cudaError_t launch_fingerprint_pooled(llmcache_bank* bk, const float* pooled, uint32_t ld, uint32_t B,
                                      __nv_bfloat16* fp, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const llmcache_bank_desc& D = bk->desc;
  ProfScope prof(bk, LLMCACHE_K_PROJECT, st);
  return launch_project(1, 1, nullptr, pooled, ld, bk->a.proj, bk->a.center, fp, rq, bk->a.status, B, D.seq_len,
                        D.d_model, D.fp_dim, bk->sm_count, st);
}

cudaError_t launch_rownorm(llmcache_bank* bk, const __nv_bfloat16* fp, uint32_t B, uint32_t k, float* rq, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  ProfScope prof(bk, LLMCACHE_K_ROWNORM, st);
  return launch_k(k_rownorm, dim3((B + 7) / 8), dim3(256), 0, st, fp, B, k, rq);
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
// Word 0 is set by the kernels if one of their bounded waits ever expired (stays zero otherwise); words 1-3
// are the diagnostic knobs every status word carries, never set here.
static __device__ __align__(16) uint32_t g_fp_static_status[4];

constexpr int STATIC_MAX_DEVICES = 64;
struct StaticDev { bool ready = false; float* scratch = nullptr; uint32_t* status = nullptr; int sm_count = 0; };
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
    uint32_t* sptr = nullptr;
    e = cudaGetSymbolAddress((void**)&sptr, g_fp_static_status);
    if (e != cudaSuccess) return e;
    if (!sptr) return cudaErrorInvalidSymbol;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = llmc::setup_fingerprint_kernels();
    if (e != cudaSuccess) return e;
    sd.scratch = ptr;
    sd.status = sptr;
    sd.sm_count = sms;
    sd.ready = true;
  }
  *out = &sd;
  return cudaSuccess;
}

}  // namespace

extern "C" const char* llmcache_fingerprint_static_error(void) { return g_static_err; }

extern "C" int llmcache_fingerprint_static_status(void) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  uint32_t* sptr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_dev[dev].ready) return LLMCACHE_OK;             // never used on this device
    sptr = g_static_dev[dev].status;
  }
  uint32_t s = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(&s, sptr, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  return s ? LLMCACHE_ERR_TIMEOUT : LLMCACHE_OK;
}

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
  if (n == 0 || d == 0 || d % 8 != 0 || d > (bf16 ? 7680u : 3840u)) return fail(LLMCACHE_ERR_SHAPE, "d_model not supported");
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

  const PoolPlan P = pool_plan(B, n, d, bf16, sd->sm_count);
  const unsigned long long need = (unsigned long long)P.grid * P.Jmax * d;
  if (need > (unsigned long long)LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS) {
    std::snprintf(g_static_err, sizeof(g_static_err),
                  "batch too large for the fixed scratch: %llu floats of partial sums needed, limit %llu",
                  need, (unsigned long long)LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS);
    return LLMCACHE_ERR_SHAPE;
  }
  cudaStream_t st = (cudaStream_t)stream;
  // every partial sum that the second kernel reads is written by the first one in this call, so
  // nothing in the shared array has to start at zero
  e = launch_pool(P, bf16, h_in, sd->scratch, sd->status, B, n, d, st);
  if (e == cudaSuccess)
    e = launch_project(P.L, P.Jmax, sd->scratch, nullptr, 0, (const __nv_bfloat16*)proj, center, (__nv_bfloat16*)fp, rq,
                       sd->status, B, n, d, k, sd->sm_count, st);
  if (e != cudaSuccess) return fail(LLMCACHE_ERR_CUDA, cudaGetErrorString(e));
  return LLMCACHE_OK;
}
