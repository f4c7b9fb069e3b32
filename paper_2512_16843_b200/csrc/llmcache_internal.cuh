// Internal definitions shared by the translation units of libllmcache.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <vector>
#include <utility>
#include "llmcache.h"

namespace llmc {

constexpr uint32_t M_CAP = (1u << 30) - 1u;   // ceiling of the decayed match rate (Q8)
constexpr uint32_t HIT_Q8 = 256u;             // one match in Q8
constexpr uint32_t POOL_MAX_GRID = 640;       // most blocks the pooling pass ever launches
// floats of one set of partial sums of a pooling (or moving) pass
inline size_t move_partial_floats(uint32_t max_batch, uint32_t d) { return ((size_t)max_batch + 3 * POOL_MAX_GRID) * d; }

// Counters kept on the device (index into Bank::d_stats).
enum { ST_SEQ = 0, ST_HIT, ST_MISS, ST_DEGEN, ST_INSERT, ST_EVICT, ST_DROP, ST_FLUSH, ST_COUNT };

struct PolicyParams {
  uint32_t policy, half_life, stale_floor, min_age, max_idle;
};

// Device arrays of one bank.  All sub-allocations are 256-byte aligned.
struct BankArrays {
  __nv_bfloat16* fp;        // [N,k]
  float*    rb;             // [N]
  uint8_t*  valid;          // [N]
  uint32_t* last_use;       // [N]
  uint32_t* insert_tick;    // [N]
  uint32_t* hits;           // [N]
  uint32_t* rate;           // [N]
  uint32_t* rate_epoch;     // [N]
  __nv_bfloat16* act;       // [act_rows, n*d]
  __nv_bfloat16* proj;      // [d,k] or nullptr
  float*    center;         // [d] or nullptr
  // scratch
  float*    pool_partial;   // [(max_batch + 3 * POOL_MAX_GRID), d] partial sums of the pooling pass
  float*    move_partial;   // 2 x the same: partial sums of the rows moved for hits / for misses (or nullptr)
  float*    pooled_own;     // [max_batch, d] position means of the rows this bank's passes wrote (fused_pool banks;
                            // used by llmcache_infer to hand them to the next layer's probe), or nullptr
  unsigned long long* best; // [max_batch] packed (orderable score << 32 | ~slot); 0 = none
  uint32_t* hitcnt;         // [N] matches per slot within the current probe (zero between calls)
  int32_t*  victims;        // [min(max_batch,N)]
  uint32_t* bits;           // [N, k/32] SimHash codes of the stored fingerprints (sign bits), packed lazily
  uint32_t* qbits;          // [max_batch, k/32]
  int32_t*  new_slot;       // [max_batch] slot each miss of the open probe will be stored in (-1: dropped)
  unsigned long long* sort_key;   // [pow2 >= min(max_batch,N)]
  uint32_t* sort_slot;      // same length
  unsigned long long* stats;      // [ST_COUNT]
  uint32_t* status;         // [1] sticky device status
  uint32_t* misc;           // [8] small per-call words
  // scratch of the multi-block decision and victim selection (large batches / large banks)
  uint32_t* blk_cnt;        // [2 * ceil(max_batch / 1024)] hits and degenerate inputs per block of the decision
  unsigned long long* sel_keys;   // [N] taking-order key of every slot
  uint32_t* sel_state;      // [SEL_STATE_WORDS] radix-select state and digit histograms (zeroed per selection)
  uint32_t* sel_blk;        // [2 * ceil(N / 1024)] keys below / equal to the threshold per block
  uint32_t* sel_mcnt;       // [ceil(max_batch / 1024)] insertable misses per block
};
constexpr uint32_t SEL_STATE_WORDS = 64 + 8 * 256;

}  // namespace llmc

struct llmcache_bank {
  llmcache_bank_desc desc{};
  llmc::BankArrays a{};
  llmc::PolicyParams pol{};
  void*    base = nullptr;  // start of the bank's device memory
  size_t   bytes = 0;
  bool     owns_memory = false;
  uint64_t tick = 0;        // probe calls so far
  uint64_t generation = 0;  // bumped by every probe
  bool     probe_open = false;   // a probe happened and was not yet committed
  uint32_t last_B = 0;
  uint64_t n_probes = 0;
  int      sm_count = 0;
  uint32_t sort_len = 0;    // length of sort_key / sort_slot
  // TMA descriptor of the fingerprint matrix (opaque 128-byte blob)
  alignas(64) unsigned char tmap_bank[128] = {};
  bool     has_tmap = false;
  // side stream on which the victim selection of a probe runs next to its gather
  cudaStream_t side = nullptr;
  cudaEvent_t  ev_fork = nullptr, ev_join = nullptr;
  bool     join_pending = false;
  bool     select_deferred = false;   // large bank: the victim selection runs at commit instead
  bool     bits_dirty = true;    // stored fingerprints changed since the SimHash codes were packed
  bool     input_stable = false; // llmcache_bank_input_stable: h_in is never the output of the preceding kernel
  // fingerprint-on-write: where the position means of the rows written in a tick go (nullptr: off)
  float*   pool_out = nullptr;
  uint32_t pool_out_ld = 0;
  uint32_t move_grid[2] = {0, 0};   // launch shapes of the two moving passes of the current tick
  uint32_t move_jmax = 0;
  bool     moved[2] = {false, false};
  // instrumentation
  uint64_t n_launches = 0;
  bool     prof_on = false;
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_used[LLMCACHE_K_COUNT];
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> prof_free;
};

namespace llmc {

// Counts a kernel launch and, while profiling is on, brackets it with events.
struct ProfScope {
  llmcache_bank* bk; int kid; cudaStream_t st; cudaEvent_t stop = nullptr;
  ProfScope(llmcache_bank* b, int k, cudaStream_t s) : bk(b), kid(k), st(s) {
    bk->n_launches += 1;
    if (!bk->prof_on) return;
    std::pair<cudaEvent_t, cudaEvent_t> ev;
    if (!bk->prof_free.empty()) { ev = bk->prof_free.back(); bk->prof_free.pop_back(); }
    else if (cudaEventCreate(&ev.first) != cudaSuccess || cudaEventCreate(&ev.second) != cudaSuccess) return;
    cudaEventRecord(ev.first, st);
    stop = ev.second;
    bk->prof_used[kid].push_back(ev);
  }
  ~ProfScope() { if (stop) cudaEventRecord(stop, st); }
};

// ---- launch wrappers implemented in the kernel translation units ----------
size_t project_smem_bytes(uint32_t d, uint32_t k, bool has_proj);
cudaError_t setup_fingerprint_kernels();
cudaError_t setup_scan_kernels();
cudaError_t setup_rows_kernels();
struct PoolPlan { uint32_t V, R, cons_threads, threads, stage_rows, stages, grid, L, Jmax; size_t smem; };
PoolPlan pool_plan(uint32_t B, uint32_t n, uint32_t d, bool bf16, int sm_count);
cudaError_t launch_fingerprint(llmcache_bank* bk, const void* h_in, uint32_t B,
                               __nv_bfloat16* fp, float* rq, cudaStream_t st);
cudaError_t launch_rownorm(llmcache_bank* bk, const __nv_bfloat16* fp, uint32_t B, uint32_t k, float* rq, cudaStream_t st);
cudaError_t launch_pool_only(llmcache_bank* bk, const void* h_in, uint32_t B, float* pooled, uint32_t ld, cudaStream_t st);
cudaError_t launch_fingerprint_pooled(llmcache_bank* bk, const float* pooled, uint32_t ld, uint32_t B,
                                      __nv_bfloat16* fp, float* rq, cudaStream_t st);
cudaError_t setup_move_kernels();
cudaError_t launch_move_pool(llmcache_bank* bk, int which, const void* miss_out, void* h_out,
                             const llmcache_probe_io* io, int32_t* new_slot_out, uint32_t B, cudaStream_t st);
cudaError_t launch_pool_finish_moved(llmcache_bank* bk, const llmcache_probe_io* io, uint32_t B,
                                     float* pooled, uint32_t ld, cudaStream_t st);
cudaError_t launch_pool_finish_plain(llmcache_bank* bk, const PoolPlan& P, uint32_t B, float* pooled, uint32_t ld,
                                     cudaStream_t st);
cudaError_t launch_scan(llmcache_bank* bk, const __nv_bfloat16* q, uint32_t B, cudaStream_t st,
                        unsigned long long* words = nullptr, uint32_t slot_base = 0);
cudaError_t launch_decide(llmcache_bank* bk, uint32_t B, float tau, const float* rq,
                          const llmcache_probe_io* io, cudaStream_t st, uint32_t sim_k = 0, int32_t ham_max = -1,
                          unsigned long long* words = nullptr, uint32_t slot_base = 0, uint32_t n_total = 0);
cudaError_t launch_simhash_scan(llmcache_bank* bk, const __nv_bfloat16* q, uint32_t B, cudaStream_t st);
cudaError_t launch_gather(llmcache_bank* bk, const void* h_in, void* h_out,
                          const llmcache_probe_io* io, uint32_t B, cudaStream_t st, uint32_t slot_base = 0,
                          uint32_t n_total = 0);
cudaError_t launch_select_victims(llmcache_bank* bk, const llmcache_probe_io* io, uint32_t B, cudaStream_t st);
cudaError_t setup_select_kernels();
cudaError_t launch_count_valid(llmcache_bank* bk, uint32_t* count_dev, cudaStream_t st);
cudaError_t launch_select_victims_mb(llmcache_bank* bk, const llmcache_probe_io* io, uint32_t B, cudaStream_t st);
cudaError_t launch_scatter_insert(llmcache_bank* bk, const void* miss_out, const llmcache_probe_io* io,
                                  void* h_out, int32_t* new_slot_out, uint32_t B, cudaStream_t st);
cudaError_t launch_evict(llmcache_bank* bk, uint32_t mode, const int32_t* slots, uint32_t n,
                         uint32_t* n_evicted, cudaStream_t st);

// Launch with programmatic dependent launch allowed: the grid may be scheduled while its predecessor
// in the stream is still running; every kernel starts with griddep_sync(), which waits until the
// predecessor has completed and its writes are visible, so only launch latency is overlapped.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                            Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- small device helpers ---------------------------------------------------
// Range checks of computed indices (slots, batch indices, rows).  In the ordinary build they cost nothing
// (the function is `true`).  A library built with -DLLMCACHE_DEBUG_BOUNDS evaluates them: the first violation
// is recorded in the status word as STATUS_BOUNDS | site and the access is skipped, so that a wrong index
// shows up as LLMCACHE_ERR_BOUNDS instead of a memory fault.
constexpr uint32_t STATUS_TIMEOUT = 1u;
constexpr uint32_t STATUS_BOUNDS = 0x100u;
enum { SITE_GATHER_HIT = 1, SITE_GATHER_MISS, SITE_SCATTER, SITE_DECIDE, SITE_SELECT, SITE_MOVE };
#ifdef LLMCACHE_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(bool ok, uint32_t* status, uint32_t site) {
  if (!ok) atomicCAS(status, 0u, STATUS_BOUNDS | site);
  return ok;
}
#else
__device__ __forceinline__ bool bounds_ok(bool, uint32_t*, uint32_t) { return true; }
#endif

// First statement of every kernel: wait for the previous grid of the stream, then let the next one
// be scheduled.
__device__ __forceinline__ void griddep_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ uint32_t float_orderable(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float orderable_float(uint32_t o) {
  uint32_t u = (o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o;
  return __uint_as_float(u);
}
__device__ __forceinline__ unsigned long long pack_best(float s, uint32_t slot) {
  return ((unsigned long long)float_orderable(s) << 32) | (unsigned long long)(0xFFFFFFFFu - slot);
}

__device__ __forceinline__ uint32_t rate_now(uint32_t rate, uint32_t rate_epoch, uint32_t epoch) {
  uint32_t sh = epoch - rate_epoch;
  return sh > 31u ? (rate >> 31) : (rate >> sh);
}

// Eviction key of an occupied slot; smaller goes first.  Ties are broken by slot.
__device__ __forceinline__ unsigned long long evict_key(const PolicyParams& p, uint32_t tick, uint32_t epoch,
                                                        uint32_t rate, uint32_t rate_epoch,
                                                        uint32_t insert_tick, uint32_t last_use) {
  if (p.policy == LLMCACHE_LRU) return (unsigned long long)last_use;
  uint32_t r = rate_now(rate, rate_epoch, epoch);
  bool stale = (r < p.stale_floor) && (tick - insert_tick >= p.min_age);
  return ((unsigned long long)(stale ? 0u : 1u) << 62) | ((unsigned long long)r << 32) | (unsigned long long)last_use;
}

// 16-byte streaming load / store (data touched once: keep it out of L1).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
// 16-byte read-only load that is kept in issue order (several can be put in flight back to back).
__device__ __forceinline__ uint4 ld_nc16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream16(void* p, uint4 v) {
  asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

}  // namespace llmc
