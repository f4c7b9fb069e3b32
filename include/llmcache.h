/*
 * llmcache.h -- C ABI of the per-layer cache probe of LLMCache
 * ("Layer-Wise Caching Strategies for Accelerated Reuse in Transformer
 * Inference"), implemented as hand-written CUDA for sm_100a.
 *
 * One bank object stands for the cache C_l of one transformer layer
 * (Sec. III-B: an independent set of (fingerprint, layer output) tuples).
 * Per batch of B sequences entering the layer the caller does
 *
 *     llmcache_probe(bank, h_in, ...)      lookup + reuse      (Algorithm 1, if-branch)
 *     <run the layer on the M compacted misses>
 *     llmcache_commit(bank, miss_out, ...) scatter + insert    (Algorithm 1, else-branch)
 *
 * and, whenever it wants to bound growth or drop outdated keys,
 *     llmcache_evict(bank, mode, ...)      refresh controller  (Sec. III-E, IV-D).
 *
 * Conventions that hold for every function:
 *  - Plain C types only.  "device" pointers are CUDA device addresses on the
 *    bank's GPU; "host" pointers are ordinary process memory.  `stream` is a
 *    cudaStream_t passed as void* (NULL = the legacy default stream).
 *  - All GPU work is enqueued on `stream` and the call returns without
 *    waiting unless stated otherwise.  A bank must be driven from one stream
 *    at a time; probe and commit of one bank alternate.
 *  - The caller owns every input/output buffer; the bank owns its storage
 *    (or borrows `arena`) until llmcache_bank_destroy.
 *  - Return value: LLMCACHE_OK (0) or a negative llmcache_status.  Argument
 *    errors are detected on the host before anything is launched.  There is no
 *    CPU fallback: without a usable CUDA device every call fails with
 *    LLMCACHE_ERR_CUDA.
 *  - Shapes: n = seq_len, d = d_model, k = fp_dim, N = capacity.
 *    d must be a multiple of 8, k a multiple of 64, rows are row-major and
 *    densely packed, every device pointer must be 16-byte aligned.
 */
#ifndef LLMCACHE_H
#define LLMCACHE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LLMCACHE_ABI_VERSION 2u

typedef struct llmcache_bank llmcache_bank_t;

typedef enum {
  LLMCACHE_OK = 0,
  LLMCACHE_ERR_ARG = -1,          /* null pointer, bad enum, bad struct_size, misaligned pointer */
  LLMCACHE_ERR_SHAPE = -2,        /* size outside what the bank was created for */
  LLMCACHE_ERR_NOMEM = -3,        /* allocation failed or arena too small */
  LLMCACHE_ERR_CUDA = -4,         /* a CUDA runtime/driver call failed (incl. no device) */
  LLMCACHE_ERR_STATE = -5,        /* calls out of order (commit without matching probe, ...) */
  LLMCACHE_ERR_TIMEOUT = -6,      /* a bounded device-side wait expired (sticky, see bank_status) */
  LLMCACHE_ERR_UNSUPPORTED = -7,  /* valid request this build does not serve */
  LLMCACHE_ERR_BOUNDS = -8        /* debug build only: a computed slot, row or batch index was out of range
                                     (sticky, see bank_status); the access was skipped */
} llmcache_status;

enum { LLMCACHE_F32 = 0, LLMCACHE_BF16 = 1 };                 /* dtype of probe inputs h_in */
enum { LLMCACHE_GT = 0, LLMCACHE_GE = 1 };                    /* hit iff sim > tau  |  sim >= tau */
enum { LLMCACHE_LRU = 0, LLMCACHE_LRU_STALENESS = 1 };        /* eviction policy */
enum { LLMCACHE_EVICT_STALE = 0, LLMCACHE_EVICT_IDLE = 1, LLMCACHE_EVICT_ALL = 2, LLMCACHE_EVICT_SLOTS = 3 };
enum {                                                        /* arrays addressable by export/import */
  LLMCACHE_WHAT_FP = 0,          /* bf16  [N,k]   stored fingerprints (unit length, rounded)   */
  LLMCACHE_WHAT_RB = 1,          /* f32   [N]     1/||stored fingerprint||                      */
  LLMCACHE_WHAT_VALID = 2,       /* u8    [N]     1 = slot occupied                             */
  LLMCACHE_WHAT_LAST_USE = 3,    /* u32   [N]     tick of last hit (or of insertion)            */
  LLMCACHE_WHAT_INSERT_TICK = 4, /* u32   [N]                                                   */
  LLMCACHE_WHAT_HITS = 5,        /* u32   [N]     matches since insertion (saturating)          */
  LLMCACHE_WHAT_RATE = 6,        /* u32   [N]     decayed match rate, Q8, as of RATE_EPOCH      */
  LLMCACHE_WHAT_RATE_EPOCH = 7,  /* u32   [N]     tick / half_life_ticks at the last update     */
  LLMCACHE_WHAT_ACT = 8,         /* bf16  [act_rows, n*d]  cached layer outputs                 */
  LLMCACHE_WHAT_TICK = 9         /* u64   [1]     number of probe calls so far                  */
};

/* Bank description (Sec. III-B; the knobs of Sec. IV-E/VI-D: threshold, cache
 * size, eviction policy).  Zero-initialise, set struct_size = sizeof, fill in. */
typedef struct llmcache_bank_desc {
  uint32_t struct_size;
  int32_t  device;            /* CUDA device ordinal */
  uint32_t capacity;          /* N >= 1 slots */
  uint32_t seq_len;           /* n >= 1 */
  uint32_t d_model;           /* d, multiple of 8, <= 7680 (bf16 inputs) or 3840 (f32 inputs) */
  uint32_t fp_dim;            /* k, multiple of 64, <= 2048; must equal d_model when proj == NULL */
  uint32_t hidden_dtype;      /* LLMCACHE_F32 | LLMCACHE_BF16 */
  uint32_t act_rows;          /* rows of the activation store; 0 => capacity.  slot j uses row j % act_rows.
                                 A bank with act_rows < capacity can be probed but not committed to. */
  uint32_t max_batch;         /* largest B any call will pass (sizes internal scratch) */
  float    tau;               /* default similarity threshold */
  uint32_t cmp;               /* LLMCACHE_GT (Sec. IV-A, Algorithm 1) | LLMCACHE_GE (Sec. III-C) */
  uint32_t policy;            /* LLMCACHE_LRU | LLMCACHE_LRU_STALENESS (Sec. IV-D) */
  uint32_t half_life_ticks;   /* decayed match rate halves every this many probe calls (0 => 8) */
  uint32_t stale_floor_q8;    /* stale if rate (Q8) below this ...                       (0 => 64) */
  uint32_t min_age_ticks;     /* ... and at least this old                              (0 => 4) */
  uint32_t max_idle_ticks;    /* LLMCACHE_EVICT_IDLE drops entries unused for longer    (0 => 32) */
  uint32_t store_act;         /* 1 = keep layer outputs (normal); 0 = keys only (scan benchmarks) */
  uint32_t fused_pool;        /* 1 = reserve the scratch llmcache_bank_pool_out needs (bf16 outputs, store_act) */
  const void*  proj;          /* device, bf16 [d,k] row-major projection (Sec. IV-B "Dimensionality
                                 Reduction"), copied at create; NULL => identity (k == d) */
  const float* center;        /* device, f32 [d] subtracted before projection, copied; NULL => 0 */
  void*    arena;             /* device memory to build the bank in (256-byte aligned), or NULL to
                                 let the library cudaMalloc it */
  size_t   arena_bytes;       /* size of arena; llmcache_bank_bytes tells how much is needed */
} llmcache_bank_desc;

/* Per-call outputs of a probe, all caller-owned DEVICE buffers sized for the
 * call's B (counts_host excepted).  commit reads the same struct back. */
typedef struct llmcache_probe_io {
  uint8_t*  hit;          /* [B]   1 = reuse                                                    */
  int32_t*  slot;         /* [B]   matching slot, -1 on miss                                    */
  float*    score;        /* [B]   best cosine (-inf: bank empty; 0: degenerate fingerprint)    */
  int32_t*  hit_idx;      /* [B]   first H entries: indices of hits, ascending                  */
  int32_t*  miss_idx;     /* [B]   first M entries: indices of misses, ascending                */
  uint32_t* counts;       /* [2]   {H, M}                                                       */
  uint32_t* counts_host;  /* optional pinned HOST [2]; filled by an async copy on the stream    */
  void*     fp;           /* [B,k] bf16 query fingerprints (probe writes; probe_fp: caller's)   */
  float*    rq;           /* [B]   1/||fp|| (0 marks a degenerate fingerprint)                  */
  void*     h_miss;       /* optional [B,n,d] (dtype of h_in): rows of the misses, compacted    */
  uint64_t  generation;   /* written by probe, checked by commit                                */
} llmcache_probe_io;

typedef struct llmcache_stats {
  uint64_t probes, sequences, hits, misses, degenerate;
  uint64_t inserts, evictions, dropped, flushed, resident;
  uint64_t kernel_launches;   /* kernels this bank has enqueued so far */
} llmcache_stats;

/* Kernels of the path, for llmcache_bank_profile_read. */
enum {
  LLMCACHE_K_POOL = 0,      /* Sec. IV-B pooled reduction                          */
  LLMCACHE_K_PROJECT = 1,   /* Sec. IV-B projection + unit length + rounding       */
  LLMCACHE_K_ROWNORM = 2,   /* inverse norms of caller-supplied fingerprints       */
  LLMCACHE_K_SCAN = 3,      /* Sec. III-C cosine scan + best slot                  */
  LLMCACHE_K_DECIDE = 4,    /* Sec. IV-A threshold + hit/miss compaction           */
  LLMCACHE_K_TOUCH = 5,     /* (unused: the metadata refresh runs inside DECIDE)  */
  LLMCACHE_K_GATHER = 6,    /* Algorithm 1 reuse: copy of cached outputs           */
  LLMCACHE_K_SELECT = 7,    /* Sec. IV-D victim selection (side stream, during GATHER) */
  LLMCACHE_K_SCATTER = 8,   /* Algorithm 1 insert: write-back + store              */
  LLMCACHE_K_EVICT = 9,     /* Sec. III-E flushes                                  */
  LLMCACHE_K_POOL_FINISH = 10, /* partial column sums -> position means               */
  LLMCACHE_K_COUNT = 11
};

uint32_t    llmcache_abi_version(void);
const char* llmcache_strerror(int status);
/* Text of the most recent CUDA error seen by this thread inside the library ("" if none). */
const char* llmcache_last_cuda_error(void);

/* Bytes of device memory a bank of this description needs (for `arena`). */
int llmcache_bank_bytes(const llmcache_bank_desc* desc, size_t* bytes_out);

/* Build an empty bank C_l (Sec. III-B).  Synchronous. */
int llmcache_bank_create(const llmcache_bank_desc* desc, llmcache_bank_t** bank_out);

/* Release the bank (frees its memory unless it lives in a caller arena).  Synchronises the device. */
int llmcache_bank_destroy(llmcache_bank_t* bank);

/* Fingerprint only (Sec. IV-B): mean over the n positions of h_in[b], minus
 * center, times proj, scaled to unit length, rounded to bf16.
 * h_in: device [B,n,d] of the bank's hidden_dtype.  fp: device bf16 [B,k].  rq: device f32 [B]. */
int llmcache_fingerprint(llmcache_bank_t* bank, const void* h_in, uint32_t B,
                         void* fp, float* rq, void* stream);

/* The two halves of llmcache_fingerprint, for callers that have the position means from elsewhere, or
 * that build the fingerprint from more than one tensor (Sec. IV-B lists, besides the aggregated
 * embeddings, optional "Prefix Attention Stats" taken from the first self-attention outputs: pool both
 * tensors into the two halves of one [B, 2d] array and fingerprint that with a bank whose d_model is 2d).
 *   llmcache_pool: pooled[b * ld + c] = mean over the n positions of h_in[b, :, c], c < d_model (step
 *     "Embedding Aggregation").  h_in: device [B,n,d] of the bank's hidden_dtype; pooled: device f32,
 *     ld >= d_model floats between sequences (a column offset is applied by the caller to `pooled`).
 *   llmcache_fingerprint_pooled: fp[b] = unit-length bf16 of (pooled[b, :d_model] - center) . proj (step
 *     "Dimensionality Reduction"); same result as llmcache_fingerprint when pooled holds the means of h_in
 *     (up to the order of the fp32 sums).  seq_len of the bank plays no part. */
int llmcache_pool(llmcache_bank_t* bank, const void* h_in, uint32_t B, float* pooled, uint32_t ld, void* stream);
int llmcache_fingerprint_pooled(llmcache_bank_t* bank, const float* pooled, uint32_t ld, uint32_t B,
                                void* fp, float* rq, void* stream);

/* Fingerprint for callers that must not allocate device memory.  (The paper has no counterpart: this
 * is a packaging variant of llmcache_fingerprint.  It launches the same two kernels in the same shapes, so on
 * one device its fp and rq are bit-identical to llmcache_fingerprint's.)
 *
 * Who needs it: code that runs after its host application has handed all device memory to its own
 * pool (an inference server that reserves the GPU at start-up, say), or inside a latency-critical
 * loop where the device-wide stall of cudaMalloc / cudaFree is not acceptable.  Such a caller has no
 * bank arena to spare for scratch and cannot let the library allocate one.
 *
 * It takes no bank.  The call runs on the CURRENT device and performs no cudaMalloc, cudaFree or other
 * allocating call; the partial sums of the pooling pass live in one fixed array inside the library
 * image (LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS floats = 8 MiB, held by every GPU that loads the
 * library until the process exits).
 *   h_in   device [B, seq_len, d_model] of hidden_dtype (LLMCACHE_F32 | LLMCACHE_BF16)
 *   proj   device bf16 [d_model, fp_dim] or NULL (then fp_dim == d_model);  center  device f32 [d_model] or NULL
 *   fp     device bf16 [B, fp_dim] out;  rq  device f32 [B] out
 * Limits: same shape rules as a bank, and the partial sums must fit: (B + 3 * G) * d_model <=
 * LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS is always enough, where G <= min(SM count, 640) is the number
 * of blocks of the pooling pass (one per SM).  A larger call is refused with LLMCACHE_ERR_SHAPE before
 * anything is launched; llmcache_fingerprint_static_error() then holds the sizes.
 * The first call on each device looks up the array's device address and sets a kernel attribute; make
 * that first call outside any stream capture.  The address is cached per device for the life of the
 * process: after a cudaDeviceReset the cached address is stale and this entry point must not be used
 * on that device again.  All calls share the one array and it keeps whatever the previous call left
 * there (nothing in it needs to start at zero: each call overwrites what it reads).  Two calls that may
 * overlap on the GPU -- different streams, or different threads -- race on it: serialise them.
 * Every device-side wait of the two kernels is bounded; llmcache_fingerprint_static_status() tells
 * whether one ever ran out (the outputs of that call are then not valid). */
#define LLMCACHE_FINGERPRINT_STATIC_MAX_FLOATS (2u * 1024u * 1024u)
int llmcache_fingerprint_static(const void* h_in, uint32_t hidden_dtype, uint32_t B, uint32_t seq_len,
                                uint32_t d_model, uint32_t fp_dim, const void* proj, const float* center,
                                void* fp, float* rq, void* stream);
/* Text describing why the last llmcache_fingerprint_static call of this thread failed ("" if it did not). */
const char* llmcache_fingerprint_static_error(void);
/* Sticky device-side status of llmcache_fingerprint_static on the current device: LLMCACHE_OK, or
 * LLMCACHE_ERR_TIMEOUT once a bounded wait of one of its kernels has expired.  Synchronises the device. */
int llmcache_fingerprint_static_status(void);

/* Lookup and reuse for one batch (Sec. III-C, Sec. IV-A case equation,
 * Algorithm 1 "if exists (f',h') with sim > tau then h_l <- h'").
 * Advances the bank's tick.  For each sequence: fingerprint h_in[b], cosine
 * against every occupied slot, best slot (ties: lowest), hit iff best > tau
 * (>= under LLMCACHE_GE).  h_out[b] (device bf16 [B,n,d]) receives the stored
 * layer output of each hit, byte for byte; rows of misses are left untouched.
 * tau: NaN => the bank's default.  B == 0 is valid and does nothing but tick.  A bank serves 2^32 - 1 probe
 * calls (the recency stamps are 32-bit ticks); the next one returns LLMCACHE_ERR_STATE.
 * All sequences see the bank as it was when the call began. */
int llmcache_probe(llmcache_bank_t* bank, const void* h_in, uint32_t B, float tau,
                   void* h_out, llmcache_probe_io* io, void* stream);

/* Lookup by SimHash codes (Sec. III-A and the dimensionality-reduction step of Sec. IV-B, which names SimHash
 * as one way to shorten the fingerprint): the code of a
 * fingerprint is the sign bit of each projected component (the projection matrix is the random-hyperplane
 * matrix), k bits per key instead of 2k bytes.  The scan finds the occupied key nearest in Hamming distance
 * (ties: lowest slot); hit iff cos(pi * ham / k) > tau, i.e. ham < k * acos(tau) / pi; io->score receives
 * that angle estimate.  Everything else (compaction, gather, metadata, commit) is as in llmcache_probe.
 * The bank's codes are re-packed from its stored fingerprints when these changed since the last call. */
int llmcache_probe_simhash(llmcache_bank_t* bank, const void* h_in, uint32_t B, float tau,
                           void* h_out, llmcache_probe_io* io, void* stream);

/* A bank split over several objects, one per GPU (the paper's outlook, Sec. VI-E, names sharing one cache between
 * devices as future work; this is the lookup half of it).  Part p holds the slots [slot_base_p, slot_base_p +
 * capacity_p) of a bank of n_total slots; every part sees the same batch of query fingerprints.
 *   1. llmcache_shard_scan on every part: the best (score, slot) of each query over the part's keys is combined
 *      by a 64-bit maximum into words[b] (device u64 [B]; the caller sets them to zero before the first part's
 *      scan).  A word is (score in an order-preserving integer form) << 32 | (2^32 - 1 - slot of the whole bank),
 *      so that the unsigned maximum of two words is the better match, the lower slot on equal scores.
 *   2. the caller takes the element-wise unsigned maximum of the words over all parts (between GPUs: an
 *      all-reduce(max); as signed 64-bit integers after flipping the top bit).  This is the one exchange step.
 *   3. llmcache_shard_decide on every part with its own copy of the combined words: threshold, hit flags, slots of
 *      the whole bank, scores, ascending index lists and counts -- identical in every part --, the metadata
 *      refresh of the matched slots the part owns, and, with h_out, the stored outputs of the hits the part owns
 *      (rows of other parts' hits and of misses are left untouched).  io->fp holds the query fingerprints on entry
 *      (as for llmcache_probe_fp); io->rq is written.  The words are consumed (set to zero).  Advances the tick
 *      like a probe and opens a probe: llmcache_commit may follow, with an io that lists this part's share of the
 *      misses (miss_idx, counts[1], and miss_out rows in that order; fp and rq of the whole batch; the generation
 *      that llmcache_shard_decide wrote).  How the misses are shared out is the caller's choice.
 * slot_base + capacity <= n_total <= 2^31. */
int llmcache_shard_scan(llmcache_bank_t* bank, const void* fp, uint32_t B, uint32_t slot_base, uint64_t* words,
                        void* stream);
int llmcache_shard_decide(llmcache_bank_t* bank, uint64_t* words, uint32_t B, float tau, uint32_t slot_base,
                          uint32_t n_total, void* h_out, llmcache_probe_io* io, void* stream);

/* A promise about the inputs of llmcache_probe / llmcache_fingerprint on this bank: with stable != 0 the caller
 * states that h_in is never written by the kernel that precedes the call in its stream (it was produced earlier,
 * or on another stream that has been waited for).  The pooling pass then starts reading h_in while that
 * preceding kernel is still finishing, instead of after it.  Results are unchanged.  Do not set it when h_in is
 * the output of the previous layer's kernels enqueued just before (the layer-wise loop of Algorithm 1 as
 * llmcache_infer runs it): the pooling pass would read rows that are still being written.  Default: 0. */
int llmcache_bank_input_stable(llmcache_bank_t* bank, int stable);

/* Same with precomputed fingerprints (Algorithm 1 computes f_X once and reuses
 * it at every layer): io->fp holds bf16 [B,k] on entry; io->rq is written.
 * h_in may be NULL (then io->h_miss is not produced). */
int llmcache_probe_fp(llmcache_bank_t* bank, const void* h_in, uint32_t B, float tau,
                      void* h_out, llmcache_probe_io* io, void* stream);

/* llmcache_probe when the position means of h_in are already known (see llmcache_bank_pool_out):
 * pooled: device f32, pooled[b * ld + c] = mean_t h_in[b,t,c].  h_in is only needed for io->h_miss and
 * may be NULL otherwise.  Everything else as llmcache_probe. */
int llmcache_probe_pooled(llmcache_bank_t* bank, const float* pooled, uint32_t ld, const void* h_in, uint32_t B,
                          float tau, void* h_out, llmcache_probe_io* io, void* stream);

/* Fingerprint-on-write.  Algorithm 1 feeds layer l+1 with the output of layer l, and the fingerprint of
 * that input starts with its mean over the positions (Sec. IV-B).  With pooled_out set, the passes
 * that write the rows of h_out -- the copy of reused outputs in llmcache_probe*, the write-back in
 * llmcache_commit -- also sum what they move, and after the commit
 *     pooled_out[b * ld + c] = mean_t h_out[b,t,c]      (device f32, every b < B of the probe)
 * ready for llmcache_probe_pooled on the next layer's bank, which then does not read h_out at all.
 * Needs a bank created with fused_pool = 1 and store_act = 1; every probe must then pass h_out, and
 * every commit miss_out.  pooled_out == NULL switches it off.  ld >= d_model. */
int llmcache_bank_pool_out(llmcache_bank_t* bank, float* pooled_out, uint32_t ld);

/* After the layer ran on the misses (Algorithm 1 else-branch, "C_l[f_X] <- h_l";
 * victim choice per Sec. III-E / IV-D).  miss_out: device bf16 [M,n,d] in the
 * order of io->miss_idx.  Writes miss_out[m] to h_out[miss_idx[m]] (skipped when
 * h_out is NULL) and inserts it under the probe's fingerprint.  Victims: free
 * slots ascending, then occupied slots by ascending (stale first, decayed rate,
 * last use, slot).  Misses with rq == 0 and misses beyond capacity are dropped.
 * new_slot: optional device i32 [B]; [m] = slot taken, -1 = dropped. */
int llmcache_commit(llmcache_bank_t* bank, const void* miss_out, const llmcache_probe_io* io,
                    void* h_out, int32_t* new_slot, void* stream);

/* Refresh controller (Sec. III-E): drop every stale entry, every entry idle
 * for more than max_idle_ticks, all entries, or the n listed slots (device
 * i32).  n_evicted_dev: optional device u32 [1] receiving the count.  Not between a probe and its
 * commit (LLMCACHE_ERR_STATE): the slots for the open probe's misses are already chosen. */
int llmcache_evict(llmcache_bank_t* bank, uint32_t mode, const int32_t* slots, uint32_t n,
                   uint32_t* n_evicted_dev, void* stream);

/* Copy one of the bank's arrays (LLMCACHE_WHAT_*) out to / in from `ptr`
 * (host or device), `bytes` must equal the array's size.  Enqueued on stream;
 * host memory must stay valid until the stream has run.  TICK is synchronous. */
int llmcache_bank_export(llmcache_bank_t* bank, uint32_t what, void* ptr, size_t bytes, void* stream);
int llmcache_bank_import(llmcache_bank_t* bank, uint32_t what, const void* ptr, size_t bytes, void* stream);

/* Counters since creation.  Synchronises the device. */
int llmcache_bank_stats(llmcache_bank_t* bank, llmcache_stats* host_out);

/* Per-kernel device timing (the paper has no counterpart; this is instrumentation).  While
 * enabled, every kernel launch of this bank is bracketed by CUDA events on its stream.
 * profile_read synchronises the device, returns the summed duration and the number of launches
 * of kernel `kernel_id` since the last read, and clears them. */
int llmcache_bank_profile(llmcache_bank_t* bank, int enable);
int llmcache_bank_profile_read(llmcache_bank_t* bank, uint32_t kernel_id, double* total_ms, uint64_t* launches);

/* Sticky device-side status (LLMCACHE_OK, LLMCACHE_ERR_TIMEOUT, or LLMCACHE_ERR_BOUNDS in a debug build).
 * Synchronises the device. */
int llmcache_bank_status(llmcache_bank_t* bank);

/* Diagnostics for the failure path (the paper has no counterpart).  Every device-side wait of the library's
 * kernels is bounded; when one runs out the kernel records LLMCACHE_ERR_TIMEOUT in the object's status word,
 * lets its copies in flight land, releases its tensor memory and returns -- the CUDA context stays usable,
 * the object's outputs and contents are no longer valid.  These calls let a test take that path without a
 * fault: wait_limit_ns replaces the bound of every wait (0 => the built-in 2 s) and
 * LLMCACHE_KNOB_PRODUCER_IDLE keeps the thread that feeds a kernel's shared-memory ring idle, so that the
 * first wait of its consumers runs out.  They apply to the kernels launched for this object afterwards and
 * stay set until changed.  Synchronises the device.  Not for production use. */
#define LLMCACHE_KNOB_PRODUCER_IDLE 1u
int llmcache_bank_debug_knobs(llmcache_bank_t* bank, uint64_t wait_limit_ns, uint32_t flags);
/* 1 if the library was built with -DLLMCACHE_DEBUG_BOUNDS, else 0.  That build range-checks every slot, row
 * and batch index the row movers, the decision and the victim selection compute before using it; the first
 * violation is recorded in the bank's status word (llmcache_bank_status -> LLMCACHE_ERR_BOUNDS) and the access
 * is skipped.  (It stands in for a memory checker on systems where none can be run.) */
int llmcache_debug_bounds_build(void);

/* ------------------------------------------------------------------------------------------------
 * Miss-path transformer layer f_l and the layer-wise caching loop.
 *
 * Sec. IV-A: h_l = f_l(h_{l-1}); Algorithm 1 runs f_l only for the inputs that found no match.  The
 * layer is the textbook one (multi-head self-attention, output projection, residual, layer norm,
 * GELU feed-forward, residual, layer norm), in two arrangements: post-norm / bidirectional / GELU(erf)
 * (BERT-style) and pre-norm / causal / GELU(tanh) (GPT-2-style).  Head size is 64.
 * Weights are bf16 matrices in [out_features, in_features] row-major layout and f32 vectors, all
 * DEVICE pointers, 16-byte aligned, borrowed: they must outlive the layer object.
 * ------------------------------------------------------------------------------------------------ */
typedef struct llmcache_layer llmcache_layer_t;

typedef struct llmcache_layer_desc {
  uint32_t struct_size;
  int32_t  device;
  uint32_t d_model;          /* d = 64 * heads */
  uint32_t heads;
  uint32_t ffn;              /* feed-forward width, multiple of 64 */
  uint32_t seq_len;          /* n */
  uint32_t max_seqs;         /* most sequences one forward call will pass */
  uint32_t pre_ln;           /* 0: post-norm (BERT-style), 1: pre-norm (GPT-2-style) */
  uint32_t causal;           /* 1: position i attends to positions <= i */
  uint32_t tanh_gelu;        /* 0: GELU with erf, 1: tanh formula */
  float    eps;              /* layer-norm epsilon (<= 0 => 1e-5) */
  const void*  w_qkv;  const float* b_qkv;     /* [3d, d], [3d]  rows: q | k | v */
  const void*  w_o;    const float* b_o;       /* [d, d], [d] */
  const float* ln1_g;  const float* ln1_b;     /* [d] */
  const void*  w_1;    const float* b_1;       /* [ffn, d], [ffn] */
  const void*  w_2;    const float* b_2;       /* [d, ffn], [d] */
  const float* ln2_g;  const float* ln2_b;     /* [d] */
  void*    workspace;        /* device scratch (256-byte aligned) or NULL => the library cudaMallocs it;
                                layers that never run concurrently may share one workspace */
  size_t   workspace_bytes;  /* llmcache_layer_bytes tells how much is needed */
} llmcache_layer_desc;

int llmcache_layer_bytes(const llmcache_layer_desc* desc, size_t* bytes_out);
int llmcache_layer_create(const llmcache_layer_desc* desc, llmcache_layer_t** layer_out);
int llmcache_layer_destroy(llmcache_layer_t* layer);

/* out[s] = f_l(x[s]) for the first sequences of x: device bf16 [n_seqs, n, d] -> device bf16 [n_seqs, n, d].
 * n_seqs_dev: optional DEVICE u32: only min(n_seqs, *n_seqs_dev) sequences are processed (pass the miss
 * count io->counts + 1 of the preceding probe: no host sync is needed).  x and out must not overlap. */
int llmcache_layer_forward(llmcache_layer_t* layer, const void* x, uint32_t n_seqs, const uint32_t* n_seqs_dev,
                           void* out, void* stream);
/* LLMCACHE_OK or LLMCACHE_ERR_TIMEOUT (a bounded device-side wait expired).  Synchronises the device. */
int llmcache_layer_status(llmcache_layer_t* layer);
/* As llmcache_bank_debug_knobs, for the layer's kernels. */
int llmcache_layer_debug_knobs(llmcache_layer_t* layer, uint64_t wait_limit_ns, uint32_t flags);


/* Input embeddings, "h_0 <- E(X)" of Algorithm 1: the hidden states that enter layer 1.
 *   h0[s, i, :] = E_tok[tokens[s, i], :] + E_pos[i, :]                      (layer_norm == 0)
 *   h0[s, i, :] = LayerNorm(that sum) * ln_gain + ln_bias over d_model      (layer_norm != 0; fp32, biased variance)
 * tokens: device int64 [n_seqs, seq_len]; tok_emb: device bf16 [vocab, d_model]; pos_emb: device bf16
 * [seq_len, d_model] or NULL (no position term); ln_gain, ln_bias: device f32 [d_model], each may be NULL (1 and
 * 0); h0: device bf16 [n_seqs, seq_len, d_model], written once, rounded to nearest even.  The caller owns every
 * buffer; nothing is allocated and the call does not synchronise.  d_model: a multiple of 8, at most 16,384
 * (else LLMCACHE_ERR_SHAPE); tables and h0 16-byte aligned, tokens 8-byte aligned (else LLMCACHE_ERR_ARG).
 * A token id outside [0, vocab) cannot be checked on the host: its row of h0 is written as zeros and, if bad_ids
 * (device u32, caller-zeroed) is not NULL, counted there.  n_seqs == 0 is valid and does nothing (the pointers are then not looked at). */
int llmcache_embed(const int64_t* tokens, uint64_t n_seqs, uint32_t seq_len, uint32_t d_model, int64_t vocab,
                   const void* tok_emb, const void* pos_emb, int32_t layer_norm, const float* ln_gain,
                   const float* ln_bias, float ln_eps, void* h0, uint32_t* bad_ids, void* stream);

/* Algorithm 1 (LLMCache-Infer) for a batch of B sequences, without any host sync: for l = 1..n_layers,
 * probe banks[l] with the current hidden states (hits take the stored output), run layers[l] on the
 * compacted misses, commit (write back + insert).  banks == NULL runs every layer in full (no caching).
 * h0: device bf16 [B,n,d].  buf_a, buf_b: device [B,n,d] bf16 ping-pong outputs; h_miss, miss_out: device
 * [B,n,d] scratch (unused without banks); io: probe buffers for B.  *h_final receives the pointer (buf_a or
 * buf_b) that holds h_L once the stream has run.  When every bank was created with fused_pool = 1 the loop
 * takes the fingerprint-on-write path by itself (see llmcache_infer_pooled; the position means travel in
 * buffers the banks own): only layer 1 reads its input to pool it. */
int llmcache_infer(llmcache_bank_t** banks, llmcache_layer_t** layers, uint32_t n_layers, const void* h0, uint32_t B,
                   float tau, void* buf_a, void* buf_b, void* h_miss, void* miss_out, llmcache_probe_io* io,
                   void** h_final, void* stream);
/* The same loop with fingerprint-on-write: only layer 1 pools its input; every later probe takes the
 * position means that the previous layer's row movers produced (llmcache_bank_pool_out /
 * llmcache_probe_pooled).  pooled: device f32 [B, d] scratch.  The banks must have fused_pool = 1; their
 * pool_out setting is overwritten and left switched off. */
int llmcache_infer_pooled(llmcache_bank_t** banks, llmcache_layer_t** layers, uint32_t n_layers, const void* h0,
                          uint32_t B, float tau, void* buf_a, void* buf_b, void* h_miss, void* miss_out,
                          llmcache_probe_io* io, float* pooled, void** h_final, void* stream);

/* Divergence monitor (Sec. III-E, divergence tracking: watch how much the output served for a fingerprint
 * differs from a fresh computation; Sec. IV-D, the monitor that re-checks stored entries).  Call after the commit of a probe, with that probe's h_in and io.
 * For every stride-th hit (ascending batch order) the layer is recomputed on the sequence's input and
 * compared with the stored output it was served: rel = ||f_l(h) - h'|| / ||f_l(h)||.  Entries with
 * rel > bound are invalidated (not those re-inserted during the current tick).
 * h_sample, out_sample: device bf16 scratch [ceil(B/stride), n, d]; rel_out: device f32 [ceil(B/stride)];
 * counters_dev: device u32 [2] = {samples checked, entries invalidated}.  The layer must have
 * max_seqs >= ceil(B/stride).  bf16 banks that store activations only. */
int llmcache_divergence_check(llmcache_bank_t* bank, llmcache_layer_t* layer, const void* h_in,
                              const llmcache_probe_io* io, uint32_t stride, float bound, void* h_sample,
                              void* out_sample, float* rel_out, uint32_t* counters_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LLMCACHE_H */
