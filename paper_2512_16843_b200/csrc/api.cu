// C ABI of libllmcache: argument checking, bank life cycle, call sequencing.
// Every step of the path runs in the CUDA kernels; nothing here computes.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include "llmcache_internal.cuh"

using namespace llmc;

namespace {

constexpr size_t ALIGN = 256;
inline size_t up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }
inline uint32_t pow2_ceil(uint32_t x) { uint32_t p = 1; while (p < x) p <<= 1; return p; }

struct Layout {
  size_t fp, rb, valid, last_use, insert_tick, hits, rate, rate_epoch, act, proj, center;
  size_t pool_partial, move_partial, pooled_own, best, hitcnt, victims, new_slot, bits, qbits, sort_key, sort_slot, stats, status, misc, blk_cnt, sel_keys, sel_state, sel_blk, sel_mcnt, total;
  uint32_t sort_len;
};

// Device guard: make the bank's device current for the duration of a call.
struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int check_desc(const llmcache_bank_desc* d) {
  if (!d) return LLMCACHE_ERR_ARG;
  if (d->struct_size != sizeof(llmcache_bank_desc)) return LLMCACHE_ERR_ARG;
  if (d->capacity == 0 || d->seq_len == 0 || d->d_model == 0 || d->fp_dim == 0 || d->max_batch == 0)
    return LLMCACHE_ERR_SHAPE;
  if (d->hidden_dtype != LLMCACHE_F32 && d->hidden_dtype != LLMCACHE_BF16) return LLMCACHE_ERR_ARG;
  if (d->cmp != LLMCACHE_GT && d->cmp != LLMCACHE_GE) return LLMCACHE_ERR_ARG;
  if (d->policy != LLMCACHE_LRU && d->policy != LLMCACHE_LRU_STALENESS) return LLMCACHE_ERR_ARG;
  if (d->d_model % 8 != 0 || d->d_model > (d->hidden_dtype == LLMCACHE_BF16 ? 7680u : 3840u)) return LLMCACHE_ERR_SHAPE;
  if (d->fp_dim % 64 != 0 || d->fp_dim > 2048) return LLMCACHE_ERR_SHAPE;
  if (!d->proj && d->fp_dim != d->d_model) return LLMCACHE_ERR_SHAPE;
  if (d->capacity > (1u << 30) || d->max_batch > (1u << 24)) return LLMCACHE_ERR_SHAPE;
  if (d->act_rows > d->capacity) return LLMCACHE_ERR_SHAPE;
  if (d->fused_pool > 1 || (d->fused_pool && !d->store_act)) return LLMCACHE_ERR_ARG;
  if (!(d->tau == d->tau)) return LLMCACHE_ERR_ARG;
  if (project_smem_bytes(d->d_model, d->fp_dim, d->proj != nullptr) > 200 * 1024) return LLMCACHE_ERR_UNSUPPORTED;
  if (d->arena && ((uintptr_t)d->arena % ALIGN) != 0) return LLMCACHE_ERR_ARG;
  if (((uintptr_t)d->proj % 16) != 0 || ((uintptr_t)d->center % 16) != 0) return LLMCACHE_ERR_ARG;
  return LLMCACHE_OK;
}

Layout make_layout(const llmcache_bank_desc& d) {
  Layout L{};
  const size_t N = d.capacity, k = d.fp_dim, dm = d.d_model, n = d.seq_len;
  const size_t act_rows = d.store_act ? (d.act_rows ? d.act_rows : d.capacity) : 0;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += up(bytes); return at; };
  L.fp = take(N * k * 2);
  L.rb = take(N * 4);
  L.valid = take(N);
  L.last_use = take(N * 4);
  L.insert_tick = take(N * 4);
  L.hits = take(N * 4);
  L.rate = take(N * 4);
  L.rate_epoch = take(N * 4);
  L.act = take(act_rows * n * dm * 2);
  L.proj = take(d.proj ? dm * k * 2 : 0);
  L.center = take(d.center ? dm * 4 : 0);
  // scratch: one vector of partial sums per (pool block, sequence it touches)
  L.pool_partial = take(((size_t)d.max_batch + 3 * POOL_MAX_GRID) * dm * 4);
  L.move_partial = take(d.fused_pool ? 2 * move_partial_floats(d.max_batch, d.d_model) * 4 : 0);
  L.pooled_own = take(d.fused_pool ? (size_t)d.max_batch * dm * 4 : 0);
  L.best = take((size_t)d.max_batch * 8);
  L.hitcnt = take(N * 4);
  const uint32_t vmax = d.max_batch < d.capacity ? d.max_batch : d.capacity;
  L.victims = take((size_t)vmax * 4);
  L.new_slot = take((size_t)d.max_batch * 4);
  L.bits = take(N * (k / 8));
  L.qbits = take((size_t)d.max_batch * (k / 8));
  L.sort_len = pow2_ceil(vmax);
  L.sort_key = take((size_t)L.sort_len * 8);
  L.sort_slot = take((size_t)L.sort_len * 4);
  L.stats = take(ST_COUNT * 8);
  L.status = take(16);                  // status word + three words of diagnostic knobs
  L.misc = take(64);
  L.blk_cnt = take(((size_t)d.max_batch + 1023) / 1024 * 8);
  L.sel_keys = take(N * 8);
  L.sel_state = take((size_t)SEL_STATE_WORDS * 4);
  L.sel_blk = take((N + 1023) / 1024 * 8);
  L.sel_mcnt = take(((size_t)d.max_batch + 1023) / 1024 * 4);
  L.total = o;
  return L;
}

thread_local char g_last_err[256] = "";
// Remember and clear a CUDA error; returns LLMCACHE_ERR_CUDA.
int cuda_fail(cudaError_t e, const char* where) {
  std::snprintf(g_last_err, sizeof(g_last_err), "%s: %s", where, cudaGetErrorString(e));
  cudaGetLastError();
  return LLMCACHE_ERR_CUDA;
}

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

int check_io(const llmcache_probe_io* io) {
  if (!io) return LLMCACHE_ERR_ARG;
  if (!io->hit || !io->slot || !io->score || !io->hit_idx || !io->miss_idx || !io->counts || !io->fp || !io->rq)
    return LLMCACHE_ERR_ARG;
  if (!aligned16(io->fp) || !aligned16(io->h_miss)) return LLMCACHE_ERR_ARG;
  return LLMCACHE_OK;
}

int array_of(llmcache_bank* bk, uint32_t what, void** ptr, size_t* bytes) {
  const size_t N = bk->desc.capacity;
  switch (what) {
    case LLMCACHE_WHAT_FP: *ptr = bk->a.fp; *bytes = N * bk->desc.fp_dim * 2; break;
    case LLMCACHE_WHAT_RB: *ptr = bk->a.rb; *bytes = N * 4; break;
    case LLMCACHE_WHAT_VALID: *ptr = bk->a.valid; *bytes = N; break;
    case LLMCACHE_WHAT_LAST_USE: *ptr = bk->a.last_use; *bytes = N * 4; break;
    case LLMCACHE_WHAT_INSERT_TICK: *ptr = bk->a.insert_tick; *bytes = N * 4; break;
    case LLMCACHE_WHAT_HITS: *ptr = bk->a.hits; *bytes = N * 4; break;
    case LLMCACHE_WHAT_RATE: *ptr = bk->a.rate; *bytes = N * 4; break;
    case LLMCACHE_WHAT_RATE_EPOCH: *ptr = bk->a.rate_epoch; *bytes = N * 4; break;
    case LLMCACHE_WHAT_ACT:
      if (!bk->a.act) return LLMCACHE_ERR_UNSUPPORTED;
      *ptr = bk->a.act;
      *bytes = (size_t)bk->desc.act_rows * bk->desc.seq_len * bk->desc.d_model * 2;
      break;
    default: return LLMCACHE_ERR_ARG;
  }
  return LLMCACHE_OK;
}

}  // namespace

extern "C" {

uint32_t llmcache_abi_version(void) { return LLMCACHE_ABI_VERSION; }
const char* llmcache_last_cuda_error(void) { return g_last_err; }

const char* llmcache_strerror(int s) {
  switch (s) {
    case LLMCACHE_OK: return "ok";
    case LLMCACHE_ERR_ARG: return "invalid argument";
    case LLMCACHE_ERR_SHAPE: return "shape not supported by this bank";
    case LLMCACHE_ERR_NOMEM: return "out of device memory or arena too small";
    case LLMCACHE_ERR_CUDA: return "CUDA call failed";
    case LLMCACHE_ERR_STATE: return "calls out of order";
    case LLMCACHE_ERR_TIMEOUT: return "bounded device wait expired";
    case LLMCACHE_ERR_UNSUPPORTED: return "not supported";
    case LLMCACHE_ERR_BOUNDS: return "index out of range (debug build)";
    default: return "unknown status";
  }
}

int llmcache_bank_bytes(const llmcache_bank_desc* desc, size_t* bytes_out) {
  if (!bytes_out) return LLMCACHE_ERR_ARG;
  int rc = check_desc(desc);
  if (rc != LLMCACHE_OK) return rc;
  *bytes_out = make_layout(*desc).total;
  return LLMCACHE_OK;
}

int llmcache_bank_create(const llmcache_bank_desc* desc, llmcache_bank_t** bank_out) {
  if (!bank_out) return LLMCACHE_ERR_ARG;
  *bank_out = nullptr;
  int rc = check_desc(desc);
  if (rc != LLMCACHE_OK) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  if (desc->device < 0 || desc->device >= ndev) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(desc->device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;

  llmcache_bank* bk = new (std::nothrow) llmcache_bank();
  if (!bk) return LLMCACHE_ERR_NOMEM;
  bk->desc = *desc;
  if (bk->desc.act_rows == 0) bk->desc.act_rows = bk->desc.capacity;
  bk->pol.policy = desc->policy;
  bk->pol.half_life = desc->half_life_ticks ? desc->half_life_ticks : 8;
  bk->pol.stale_floor = desc->stale_floor_q8 ? desc->stale_floor_q8 : 64;
  bk->pol.min_age = desc->min_age_ticks ? desc->min_age_ticks : 4;
  bk->pol.max_idle = desc->max_idle_ticks ? desc->max_idle_ticks : 32;
  bk->desc.half_life_ticks = bk->pol.half_life;
  bk->desc.stale_floor_q8 = bk->pol.stale_floor;
  bk->desc.min_age_ticks = bk->pol.min_age;
  bk->desc.max_idle_ticks = bk->pol.max_idle;

  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, desc->device) != cudaSuccess) { delete bk; return LLMCACHE_ERR_CUDA; }
  bk->sm_count = prop.multiProcessorCount;

  const Layout L = make_layout(*desc);
  bk->bytes = L.total;
  if (desc->arena) {
    if (desc->arena_bytes < L.total) { delete bk; return LLMCACHE_ERR_NOMEM; }
    bk->base = desc->arena;
    bk->owns_memory = false;
  } else {
    if (cudaMalloc(&bk->base, L.total) != cudaSuccess) { cudaGetLastError(); delete bk; return LLMCACHE_ERR_NOMEM; }
    bk->owns_memory = true;
  }
  char* base = (char*)bk->base;
  BankArrays& a = bk->a;
  a.fp = (__nv_bfloat16*)(base + L.fp);
  a.rb = (float*)(base + L.rb);
  a.valid = (uint8_t*)(base + L.valid);
  a.last_use = (uint32_t*)(base + L.last_use);
  a.insert_tick = (uint32_t*)(base + L.insert_tick);
  a.hits = (uint32_t*)(base + L.hits);
  a.rate = (uint32_t*)(base + L.rate);
  a.rate_epoch = (uint32_t*)(base + L.rate_epoch);
  a.act = desc->store_act ? (__nv_bfloat16*)(base + L.act) : nullptr;
  a.proj = desc->proj ? (__nv_bfloat16*)(base + L.proj) : nullptr;
  a.center = desc->center ? (float*)(base + L.center) : nullptr;
  a.pool_partial = (float*)(base + L.pool_partial);
  a.move_partial = desc->fused_pool ? (float*)(base + L.move_partial) : nullptr;
  a.pooled_own = desc->fused_pool ? (float*)(base + L.pooled_own) : nullptr;
  a.best = (unsigned long long*)(base + L.best);
  a.hitcnt = (uint32_t*)(base + L.hitcnt);
  a.victims = (int32_t*)(base + L.victims);
  a.new_slot = (int32_t*)(base + L.new_slot);
  a.bits = (uint32_t*)(base + L.bits);
  a.qbits = (uint32_t*)(base + L.qbits);
  a.sort_key = (unsigned long long*)(base + L.sort_key);
  a.sort_slot = (uint32_t*)(base + L.sort_slot);
  a.stats = (unsigned long long*)(base + L.stats);
  a.status = (uint32_t*)(base + L.status);
  a.misc = (uint32_t*)(base + L.misc);
  a.blk_cnt = (uint32_t*)(base + L.blk_cnt);
  a.sel_keys = (unsigned long long*)(base + L.sel_keys);
  a.sel_state = (uint32_t*)(base + L.sel_state);
  a.sel_blk = (uint32_t*)(base + L.sel_blk);
  a.sel_mcnt = (uint32_t*)(base + L.sel_mcnt);
  bk->sort_len = L.sort_len;

  cudaError_t e = cudaSuccess;
  e = cudaMemset(base, 0, L.total);
  if (e == cudaSuccess && desc->proj)
    e = cudaMemcpy(a.proj, desc->proj, (size_t)desc->d_model * desc->fp_dim * 2, cudaMemcpyDefault);
  if (e == cudaSuccess && desc->center)
    e = cudaMemcpy(a.center, desc->center, (size_t)desc->d_model * 4, cudaMemcpyDefault);
  if (e == cudaSuccess) e = setup_fingerprint_kernels();
  if (e == cudaSuccess) e = setup_scan_kernels();
  if (e == cudaSuccess) e = setup_rows_kernels();
  if (e == cudaSuccess) e = setup_move_kernels();
  if (e == cudaSuccess) e = setup_select_kernels();
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&bk->side, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&bk->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&bk->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    if (bk->side) cudaStreamDestroy(bk->side);
    if (bk->ev_fork) cudaEventDestroy(bk->ev_fork);
    if (bk->ev_join) cudaEventDestroy(bk->ev_join);
    if (bk->owns_memory) cudaFree(bk->base);
    delete bk;
    return cuda_fail(e, "bank_create");
  }
  *bank_out = bk;
  return LLMCACHE_OK;
}

int llmcache_bank_destroy(llmcache_bank_t* bk) {
  if (!bk) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaError_t e = cudaDeviceSynchronize();
  if (bk->side) cudaStreamDestroy(bk->side);
  if (bk->ev_fork) cudaEventDestroy(bk->ev_fork);
  if (bk->ev_join) cudaEventDestroy(bk->ev_join);
  if (bk->owns_memory && bk->base) cudaFree(bk->base);
  for (int i = 0; i < LLMCACHE_K_COUNT; ++i)
    for (auto& ev : bk->prof_used[i]) bk->prof_free.push_back(ev);
  for (auto& ev : bk->prof_free) { cudaEventDestroy(ev.first); cudaEventDestroy(ev.second); }
  delete bk;
  return e == cudaSuccess ? LLMCACHE_OK : LLMCACHE_ERR_CUDA;
}

int llmcache_fingerprint(llmcache_bank_t* bk, const void* h_in, uint32_t B, void* fp, float* rq, void* stream) {
  if (!bk || (B && (!h_in || !fp || !rq))) return LLMCACHE_ERR_ARG;
  if (B > bk->desc.max_batch) return LLMCACHE_ERR_SHAPE;
  if (!aligned16(h_in) || !aligned16(fp)) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaError_t e = launch_fingerprint(bk, h_in, B, (__nv_bfloat16*)fp, rq, (cudaStream_t)stream);
  return e == cudaSuccess ? LLMCACHE_OK : cuda_fail(e, __func__);
}

int llmcache_pool(llmcache_bank_t* bk, const void* h_in, uint32_t B, float* pooled, uint32_t ld, void* stream) {
  if (!bk || (B && (!h_in || !pooled))) return LLMCACHE_ERR_ARG;
  if (B > bk->desc.max_batch || ld < bk->desc.d_model) return LLMCACHE_ERR_SHAPE;
  if (!aligned16(h_in) || ((uintptr_t)pooled & 3u)) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaError_t e = launch_pool_only(bk, h_in, B, pooled, ld, (cudaStream_t)stream);
  return e == cudaSuccess ? LLMCACHE_OK : cuda_fail(e, __func__);
}

int llmcache_fingerprint_pooled(llmcache_bank_t* bk, const float* pooled, uint32_t ld, uint32_t B,
                                void* fp, float* rq, void* stream) {
  if (!bk || (B && (!pooled || !fp || !rq))) return LLMCACHE_ERR_ARG;
  if (B > bk->desc.max_batch || ld < bk->desc.d_model) return LLMCACHE_ERR_SHAPE;
  if (!aligned16(fp) || ((uintptr_t)pooled & 3u)) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaError_t e = launch_fingerprint_pooled(bk, pooled, ld, B, (__nv_bfloat16*)fp, rq, (cudaStream_t)stream);
  return e == cudaSuccess ? LLMCACHE_OK : cuda_fail(e, __func__);
}

int llmcache_bank_pool_out(llmcache_bank_t* bk, float* pooled_out, uint32_t ld) {
  if (!bk) return LLMCACHE_ERR_ARG;
  if (bk->probe_open && bk->last_B) return LLMCACHE_ERR_STATE;      // not between a probe and its commit
  if (!pooled_out) { bk->pool_out = nullptr; bk->pool_out_ld = 0; return LLMCACHE_OK; }
  if (!bk->a.move_partial || !bk->a.act) return LLMCACHE_ERR_UNSUPPORTED;
  if (ld < bk->desc.d_model) return LLMCACHE_ERR_SHAPE;
  if ((uintptr_t)pooled_out & 3u) return LLMCACHE_ERR_ARG;
  bk->pool_out = pooled_out;
  bk->pool_out_ld = ld;
  return LLMCACHE_OK;
}

// Largest Hamming distance that still matches: the SimHash angle estimate is pi * ham / k and a match
// needs cos(angle) > tau, i.e. ham < k * acos(tau) / pi.
static int32_t hamming_threshold(float tau, uint32_t k) {
  const double t = (double)tau;
  if (t >= 1.0) return -1;
  if (t <= -1.0) return (int32_t)k;
  const double x = (double)k * std::acos(t) / 3.14159265358979323846;
  long h = (long)std::ceil(x) - 1;
  if (h < -1) h = -1;
  if (h > (long)k) h = (long)k;
  return (int32_t)h;
}

static int probe_common(llmcache_bank_t* bk, const void* h_in, bool compute_fp, uint32_t B, float tau,
                        void* h_out, llmcache_probe_io* io, void* stream, bool simhash = false,
                        const float* pooled = nullptr, uint32_t pooled_ld = 0) {
  if (!bk) return LLMCACHE_ERR_ARG;
  if (B > bk->desc.max_batch) return LLMCACHE_ERR_SHAPE;
  if (B) {
    int rc = check_io(io);
    if (rc != LLMCACHE_OK) return rc;
    if (compute_fp && !h_in && !pooled) return LLMCACHE_ERR_ARG;
    if (pooled && (pooled_ld < bk->desc.d_model || ((uintptr_t)pooled & 3u))) return LLMCACHE_ERR_SHAPE;
    if (bk->pool_out && !h_out) return LLMCACHE_ERR_ARG;             // every row of h_out must pass through
    if (!aligned16(h_in) || !aligned16(h_out)) return LLMCACHE_ERR_ARG;
  } else if (!io) {
    return LLMCACHE_ERR_ARG;
  }
  if (std::isnan(tau)) tau = bk->desc.tau;
  if (bk->tick >= 0xFFFFFFFFull) return LLMCACHE_ERR_STATE;       // the device keeps ticks in 32 bits
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;

  bk->tick += 1;
  bk->generation += 1;
  bk->n_probes += 1;
  io->generation = bk->generation;
  bk->probe_open = true;
  bk->last_B = B;
  cudaError_t e = cudaSuccess;
  if (bk->join_pending) {          // a previous probe was never committed: its victim selection must be over
    e = cudaStreamWaitEvent(st, bk->ev_join, 0);
    bk->join_pending = false;
  }
  if (e != cudaSuccess) return cuda_fail(e, __func__);
  if (B == 0) {
    if (io->counts) e = cudaMemsetAsync(io->counts, 0, 2 * sizeof(uint32_t), st);
  } else {
    if (pooled)          e = launch_fingerprint_pooled(bk, pooled, pooled_ld, B, (__nv_bfloat16*)io->fp, io->rq, st);
    else if (compute_fp) e = launch_fingerprint(bk, h_in, B, (__nv_bfloat16*)io->fp, io->rq, st);
    else                 e = launch_rownorm(bk, (const __nv_bfloat16*)io->fp, B, bk->desc.fp_dim, io->rq, st);
    if (simhash) {
      if (e == cudaSuccess) e = launch_simhash_scan(bk, (const __nv_bfloat16*)io->fp, B, st);
      if (e == cudaSuccess) e = launch_decide(bk, B, tau, io->rq, io, st, bk->desc.fp_dim, hamming_threshold(tau, bk->desc.fp_dim));
    } else {
      if (e == cudaSuccess) e = launch_scan(bk, (const __nv_bfloat16*)io->fp, B, st);
      if (e == cudaSuccess) e = launch_decide(bk, B, tau, io->rq, io, st);
    }
    // The slots for this batch's misses are chosen now, on the side stream, while the gather runs:
    // the choice depends only on the metadata after this probe's refresh, which the gather does not touch.
    // (A bank that stores keys only has no gather to hide the selection behind, and over a very large bank it
    // takes a few dozen launches; there it is left to the commit, so that probes that are never committed do
    // not pay for it.)
    bk->select_deferred = !bk->a.act || bk->desc.capacity > 65536u;
    if (!bk->select_deferred) {
      if (e == cudaSuccess) e = cudaEventRecord(bk->ev_fork, st);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(bk->side, bk->ev_fork, 0);
      if (e == cudaSuccess) e = launch_select_victims(bk, io, B, bk->side);
      if (e == cudaSuccess) e = cudaEventRecord(bk->ev_join, bk->side);
      if (e == cudaSuccess) bk->join_pending = true;
    }
    bk->moved[0] = bk->moved[1] = false;
    if (bk->pool_out) {
      // the reused rows are summed while they are copied; the miss inputs (if wanted) go the plain way
      if (e == cudaSuccess) e = launch_move_pool(bk, 0, nullptr, h_out, io, nullptr, B, st);
      if (e == cudaSuccess) bk->moved[0] = true;
      if (e == cudaSuccess && h_in && io->h_miss) e = launch_gather(bk, h_in, nullptr, io, B, st);
    } else {
      if (e == cudaSuccess) e = launch_gather(bk, h_in, h_out, io, B, st);
    }
  }
  if (e == cudaSuccess && io->counts_host && io->counts)
    e = cudaMemcpyAsync(io->counts_host, io->counts, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
  if (e != cudaSuccess) return cuda_fail(e, __func__);
  return LLMCACHE_OK;
}

int llmcache_probe(llmcache_bank_t* bk, const void* h_in, uint32_t B, float tau, void* h_out,
                   llmcache_probe_io* io, void* stream) {
  return probe_common(bk, h_in, true, B, tau, h_out, io, stream);
}

int llmcache_probe_simhash(llmcache_bank_t* bk, const void* h_in, uint32_t B, float tau, void* h_out,
                           llmcache_probe_io* io, void* stream) {
  return probe_common(bk, h_in, true, B, tau, h_out, io, stream, true);
}

int llmcache_probe_fp(llmcache_bank_t* bk, const void* h_in, uint32_t B, float tau, void* h_out,
                      llmcache_probe_io* io, void* stream) {
  return probe_common(bk, h_in, false, B, tau, h_out, io, stream);
}

int llmcache_probe_pooled(llmcache_bank_t* bk, const float* pooled, uint32_t ld, const void* h_in, uint32_t B,
                          float tau, void* h_out, llmcache_probe_io* io, void* stream) {
  if (B && !pooled) return LLMCACHE_ERR_ARG;
  return probe_common(bk, h_in, true, B, tau, h_out, io, stream, false, pooled, ld);
}

int llmcache_commit(llmcache_bank_t* bk, const void* miss_out, const llmcache_probe_io* io, void* h_out,
                    int32_t* new_slot, void* stream) {
  if (!bk || !io) return LLMCACHE_ERR_ARG;
  if (!bk->probe_open || io->generation != bk->generation) return LLMCACHE_ERR_STATE;
  if (bk->desc.act_rows != bk->desc.capacity) return LLMCACHE_ERR_UNSUPPORTED;
  const uint32_t B = bk->last_B;
  if (B) {
    int rc = check_io(io);
    if (rc != LLMCACHE_OK) return rc;
    if (!aligned16(miss_out) || !aligned16(h_out)) return LLMCACHE_ERR_ARG;
    if (bk->a.act && !miss_out) return LLMCACHE_ERR_ARG;
    if (bk->pool_out && !miss_out) return LLMCACHE_ERR_ARG;
  }
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  bk->probe_open = false;
  if (B == 0) return LLMCACHE_OK;
  // the slots were chosen during the probe (side stream); here the rows move
  cudaError_t e = cudaSuccess;
  if (bk->join_pending) {
    e = cudaStreamWaitEvent(st, bk->ev_join, 0);
    bk->join_pending = false;
  }
  bk->bits_dirty = true;
  if (e == cudaSuccess && bk->select_deferred) e = launch_select_victims(bk, io, B, st);
  bk->select_deferred = false;
  if (bk->pool_out && bk->moved[0]) {
    // the rows (summed while they move) with the keys and metadata of the new entries, then the means
    if (e == cudaSuccess) e = launch_move_pool(bk, 1, miss_out, h_out, io, new_slot, B, st);
    if (e == cudaSuccess) e = launch_pool_finish_moved(bk, io, B, bk->pool_out, bk->pool_out_ld, st);
    bk->moved[0] = bk->moved[1] = false;
  } else {
    if (e == cudaSuccess) e = launch_scatter_insert(bk, miss_out, io, h_out, new_slot, B, st);
  }
  if (e != cudaSuccess) return cuda_fail(e, __func__);
  return LLMCACHE_OK;
}

int llmcache_evict(llmcache_bank_t* bk, uint32_t mode, const int32_t* slots, uint32_t n,
                   uint32_t* n_evicted_dev, void* stream) {
  if (!bk) return LLMCACHE_ERR_ARG;
  if (mode > LLMCACHE_EVICT_SLOTS) return LLMCACHE_ERR_ARG;
  if (mode == LLMCACHE_EVICT_SLOTS && n && !slots) return LLMCACHE_ERR_ARG;
  if (bk->probe_open && bk->last_B) return LLMCACHE_ERR_STATE;   // the open probe's slot choice would go stale
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaError_t e = launch_evict(bk, mode, slots, n, n_evicted_dev, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, __func__);
  return LLMCACHE_OK;
}

int llmcache_bank_export(llmcache_bank_t* bk, uint32_t what, void* ptr, size_t bytes, void* stream) {
  if (!bk || !ptr) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  if (what == LLMCACHE_WHAT_TICK) {
    if (bytes != 8) return LLMCACHE_ERR_SHAPE;
    return cudaMemcpy(ptr, &bk->tick, 8, cudaMemcpyDefault) == cudaSuccess ? LLMCACHE_OK : LLMCACHE_ERR_CUDA;
  }
  void* src; size_t sz;
  int rc = array_of(bk, what, &src, &sz);
  if (rc != LLMCACHE_OK) return rc;
  if (bytes != sz) return LLMCACHE_ERR_SHAPE;
  cudaError_t e = cudaMemcpyAsync(ptr, src, sz, cudaMemcpyDefault, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, __func__);
  return LLMCACHE_OK;
}

int llmcache_bank_import(llmcache_bank_t* bk, uint32_t what, const void* ptr, size_t bytes, void* stream) {
  if (!bk || !ptr) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  if (what == LLMCACHE_WHAT_TICK) {
    if (bytes != 8) return LLMCACHE_ERR_SHAPE;
    uint64_t t;
    if (cudaMemcpy(&t, ptr, 8, cudaMemcpyDefault) != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
    bk->tick = t;
    bk->probe_open = false;
    return LLMCACHE_OK;
  }
  void* dst; size_t sz;
  int rc = array_of(bk, what, &dst, &sz);
  if (rc != LLMCACHE_OK) return rc;
  if (bytes != sz) return LLMCACHE_ERR_SHAPE;
  if (what == LLMCACHE_WHAT_FP) bk->bits_dirty = true;
  cudaError_t e = cudaMemcpyAsync(dst, ptr, sz, cudaMemcpyDefault, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, __func__);
  return LLMCACHE_OK;
}

int llmcache_bank_stats(llmcache_bank_t* bk, llmcache_stats* out) {
  if (!bk || !out) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  unsigned long long h[ST_COUNT];
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(h, bk->a.stats, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  // occupied slots, counted on the device (misc[4] is free between calls: the device is idle here)
  uint32_t res = 0;
  if (launch_count_valid(bk, bk->a.misc + 4, nullptr) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&res, bk->a.misc + 4, sizeof(res), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  out->probes = bk->n_probes;
  out->sequences = h[ST_SEQ];
  out->hits = h[ST_HIT];
  out->misses = h[ST_MISS];
  out->degenerate = h[ST_DEGEN];
  out->inserts = h[ST_INSERT];
  out->evictions = h[ST_EVICT];
  out->dropped = h[ST_DROP];
  out->flushed = h[ST_FLUSH];
  out->resident = res;
  out->kernel_launches = bk->n_launches;
  return LLMCACHE_OK;
}

int llmcache_bank_profile(llmcache_bank_t* bk, int enable) {
  if (!bk) return LLMCACHE_ERR_ARG;
  bk->prof_on = enable != 0;
  return LLMCACHE_OK;
}

int llmcache_bank_profile_read(llmcache_bank_t* bk, uint32_t kid, double* total_ms, uint64_t* launches) {
  if (!bk || kid >= LLMCACHE_K_COUNT || !total_ms || !launches) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  double sum = 0.0;
  for (auto& ev : bk->prof_used[kid]) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ev.first, ev.second) == cudaSuccess) sum += ms; else cudaGetLastError();
    bk->prof_free.push_back(ev);
  }
  *launches = bk->prof_used[kid].size();
  *total_ms = sum;
  bk->prof_used[kid].clear();
  return LLMCACHE_OK;
}

int llmcache_bank_status(llmcache_bank_t* bk) {
  if (!bk) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  uint32_t s = 0;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&s, bk->a.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  if (s & STATUS_BOUNDS) return LLMCACHE_ERR_BOUNDS;
  return s ? LLMCACHE_ERR_TIMEOUT : LLMCACHE_OK;
}

int llmcache_debug_bounds_build(void) {
#ifdef LLMCACHE_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

// ---- a bank split over several objects (or GPUs): scan, exchange of the best words by the caller, decision
int llmcache_shard_scan(llmcache_bank_t* bk, const void* fp, uint32_t B, uint32_t slot_base, uint64_t* words,
                        void* stream) {
  if (!bk || (B && (!fp || !words))) return LLMCACHE_ERR_ARG;
  if (B > bk->desc.max_batch) return LLMCACHE_ERR_SHAPE;
  if (!aligned16(fp) || ((uintptr_t)words & 7u)) return LLMCACHE_ERR_ARG;
  if ((unsigned long long)slot_base + bk->desc.capacity > (1ull << 31)) return LLMCACHE_ERR_SHAPE;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaError_t e = launch_scan(bk, (const __nv_bfloat16*)fp, B, (cudaStream_t)stream, (unsigned long long*)words, slot_base);
  return e == cudaSuccess ? LLMCACHE_OK : cuda_fail(e, __func__);
}

int llmcache_shard_decide(llmcache_bank_t* bk, uint64_t* words, uint32_t B, float tau, uint32_t slot_base,
                          uint32_t n_total, void* h_out, llmcache_probe_io* io, void* stream) {
  if (!bk || !io) return LLMCACHE_ERR_ARG;
  if (B > bk->desc.max_batch) return LLMCACHE_ERR_SHAPE;
  if ((unsigned long long)slot_base + bk->desc.capacity > n_total || n_total > (1u << 31)) return LLMCACHE_ERR_SHAPE;
  if (B) {
    int rc = check_io(io);
    if (rc != LLMCACHE_OK) return rc;
    if (!words || ((uintptr_t)words & 7u) || !aligned16(h_out)) return LLMCACHE_ERR_ARG;
  }
  if (std::isnan(tau)) tau = bk->desc.tau;
  if (bk->tick >= 0xFFFFFFFFull) return LLMCACHE_ERR_STATE;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  bk->tick += 1;
  bk->generation += 1;
  bk->n_probes += 1;
  io->generation = bk->generation;
  bk->probe_open = true;
  bk->last_B = B;
  cudaError_t e = cudaSuccess;
  if (bk->join_pending) {
    e = cudaStreamWaitEvent(st, bk->ev_join, 0);
    bk->join_pending = false;
  }
  bk->select_deferred = true;                       // the slots for this part's share of the misses are chosen at commit
  bk->moved[0] = bk->moved[1] = false;
  if (B == 0) {
    if (e == cudaSuccess) e = cudaMemsetAsync(io->counts, 0, 2 * sizeof(uint32_t), st);
  } else {
    if (e == cudaSuccess) e = launch_rownorm(bk, (const __nv_bfloat16*)io->fp, B, bk->desc.fp_dim, io->rq, st);
    if (e == cudaSuccess) e = launch_decide(bk, B, tau, io->rq, io, st, 0, -1, (unsigned long long*)words, slot_base, n_total);
    if (e == cudaSuccess && h_out && bk->a.act) e = launch_gather(bk, nullptr, h_out, io, B, st, slot_base, n_total);
  }
  if (e == cudaSuccess && io->counts_host && io->counts)
    e = cudaMemcpyAsync(io->counts_host, io->counts, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
  return e == cudaSuccess ? LLMCACHE_OK : cuda_fail(e, __func__);
}

int llmcache_bank_input_stable(llmcache_bank_t* bk, int stable) {
  if (!bk) return LLMCACHE_ERR_ARG;
  bk->input_stable = stable != 0;
  return LLMCACHE_OK;
}

int llmcache_bank_debug_knobs(llmcache_bank_t* bk, uint64_t wait_limit_ns, uint32_t flags) {
  if (!bk) return LLMCACHE_ERR_ARG;
  DeviceGuard guard(bk->desc.device);
  if (!guard.ok) return LLMCACHE_ERR_CUDA;
  uint32_t w[3] = {flags, (uint32_t)(wait_limit_ns & 0xFFFFFFFFull), (uint32_t)(wait_limit_ns >> 32)};
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(bk->a.status + 1, w, sizeof(w), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  return LLMCACHE_OK;
}

}  // extern "C"
