// C ABI of the miss-path transformer layer and of the layer-wise caching loop (Algorithm 1).
#include <cstdio>
#include <cstring>
#include <new>
#include "layer.cuh"

using namespace llmc;

struct llmcache_layer {
  llmcache_layer_desc desc{};
  int sm_count = 0;
  char* ws = nullptr;            // workspace
  bool owns_ws = false;
  __nv_bfloat16 *qkv = nullptr, *a = nullptr, *t = nullptr, *y = nullptr, *f = nullptr, *vt = nullptr;
  uint32_t* status = nullptr;    // device word: a bounded wait expired
};

namespace {
constexpr size_t WS_ALIGN = 256;
inline size_t up256(size_t x) { return (x + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN; }

int check_layer_desc(const llmcache_layer_desc* d) {
  if (!d || d->struct_size != sizeof(llmcache_layer_desc)) return LLMCACHE_ERR_ARG;
  if (d->d_model == 0 || d->heads == 0 || d->ffn == 0 || d->seq_len == 0 || d->max_seqs == 0) return LLMCACHE_ERR_SHAPE;
  if (d->d_model % 64 != 0 || d->ffn % 64 != 0) return LLMCACHE_ERR_SHAPE;
  if (d->d_model != d->heads * 64) return LLMCACHE_ERR_UNSUPPORTED;       // head size 64 only
  if ((unsigned long long)d->max_seqs * d->seq_len > 0xFFFFFFFFull) return LLMCACHE_ERR_SHAPE;
  const void* ptrs[] = {d->w_qkv, d->b_qkv, d->w_o, d->b_o, d->ln1_g, d->ln1_b, d->w_1, d->b_1, d->w_2, d->b_2,
                        d->ln2_g, d->ln2_b};
  for (const void* p : ptrs)
    if (!p || ((uintptr_t)p & 15u)) return LLMCACHE_ERR_ARG;
  if (d->workspace && ((uintptr_t)d->workspace % WS_ALIGN)) return LLMCACHE_ERR_ARG;
  return LLMCACHE_OK;
}

size_t layer_ws_bytes(const llmcache_layer_desc& d) {
  const size_t T = (size_t)d.max_seqs * d.seq_len;
  const size_t vt = (size_t)d.max_seqs * d.d_model * attention_vt_pitch(d.seq_len) * 2;      // per-head transposes of V
  return up256(T * 3 * d.d_model * 2) + 3 * up256(T * d.d_model * 2) + up256(T * d.ffn * 2) + up256(vt) + WS_ALIGN;
}
}  // namespace

extern "C" {

int llmcache_layer_bytes(const llmcache_layer_desc* desc, size_t* bytes_out) {
  if (!bytes_out) return LLMCACHE_ERR_ARG;
  int rc = check_layer_desc(desc);
  if (rc != LLMCACHE_OK) return rc;
  *bytes_out = layer_ws_bytes(*desc);
  return LLMCACHE_OK;
}

int llmcache_layer_create(const llmcache_layer_desc* desc, llmcache_layer_t** layer_out) {
  if (!layer_out) return LLMCACHE_ERR_ARG;
  *layer_out = nullptr;
  int rc = check_layer_desc(desc);
  if (rc != LLMCACHE_OK) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  if (desc->device < 0 || desc->device >= ndev) return LLMCACHE_ERR_ARG;
  int prev = 0;
  cudaGetDevice(&prev);
  if (cudaSetDevice(desc->device) != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  llmcache_layer* L = new (std::nothrow) llmcache_layer();
  if (!L) { cudaSetDevice(prev); return LLMCACHE_ERR_NOMEM; }
  L->desc = *desc;
  if (L->desc.eps <= 0.f) L->desc.eps = 1e-5f;
  const size_t need = layer_ws_bytes(*desc);
  cudaError_t e = cudaDeviceGetAttribute(&L->sm_count, cudaDevAttrMultiProcessorCount, desc->device);
  if (e == cudaSuccess) {
    if (desc->workspace) {
      if (desc->workspace_bytes < need) { delete L; cudaSetDevice(prev); return LLMCACHE_ERR_NOMEM; }
      L->ws = (char*)desc->workspace;
    } else {
      if (cudaMalloc((void**)&L->ws, need) != cudaSuccess) { cudaGetLastError(); delete L; cudaSetDevice(prev); return LLMCACHE_ERR_NOMEM; }
      L->owns_ws = true;
    }
  }
  if (e == cudaSuccess) {
    const size_t T = (size_t)desc->max_seqs * desc->seq_len, d = desc->d_model;
    char* p = L->ws;
    L->status = (uint32_t*)p; p += WS_ALIGN;
    L->qkv = (__nv_bfloat16*)p; p += up256(T * 3 * d * 2);
    L->a = (__nv_bfloat16*)p; p += up256(T * d * 2);
    L->t = (__nv_bfloat16*)p; p += up256(T * d * 2);
    L->y = (__nv_bfloat16*)p; p += up256(T * d * 2);
    L->f = (__nv_bfloat16*)p; p += up256(T * desc->ffn * 2);
    L->vt = (__nv_bfloat16*)p;
    e = cudaMemset(L->status, 0, WS_ALIGN);
  }
  if (e == cudaSuccess) e = setup_gemm_kernel();
  if (e == cudaSuccess) e = setup_attention_kernel();
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    cudaGetLastError();
    if (L->owns_ws) cudaFree(L->ws);
    delete L;
    return LLMCACHE_ERR_CUDA;
  }
  *layer_out = L;
  return LLMCACHE_OK;
}

int llmcache_layer_destroy(llmcache_layer_t* L) {
  if (!L) return LLMCACHE_ERR_ARG;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(L->desc.device);
  cudaError_t e = cudaDeviceSynchronize();
  if (L->owns_ws) cudaFree(L->ws);
  cudaSetDevice(prev);
  delete L;
  return e == cudaSuccess ? LLMCACHE_OK : LLMCACHE_ERR_CUDA;
}

int llmcache_layer_forward(llmcache_layer_t* L, const void* x, uint32_t n_seqs, const uint32_t* n_seqs_dev,
                           void* out, void* stream) {
  if (!L || (n_seqs && (!x || !out))) return LLMCACHE_ERR_ARG;
  if (n_seqs > L->desc.max_seqs) return LLMCACHE_ERR_SHAPE;
  if (((uintptr_t)x | (uintptr_t)out) & 15u) return LLMCACHE_ERR_ARG;
  if (n_seqs == 0) return LLMCACHE_OK;
  int prev = 0;
  cudaGetDevice(&prev);
  if (prev != L->desc.device && cudaSetDevice(L->desc.device) != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  const llmcache_layer_desc& D = L->desc;
  const uint32_t n = D.seq_len, d = D.d_model, T = n_seqs * n;
  const uint32_t act = D.tanh_gelu ? LAYER_ACT_GELU_TANH : LAYER_ACT_GELU_ERF;
  cudaStream_t st = (cudaStream_t)stream;
  const __nv_bfloat16* X = (const __nv_bfloat16*)x;
  __nv_bfloat16* O = (__nv_bfloat16*)out;
  const int sm = L->sm_count;
  cudaError_t e;
  auto gemm = [&](const __nv_bfloat16* a, const void* w, const float* bias, const __nv_bfloat16* res,
                  __nv_bfloat16* o, uint32_t N, uint32_t K, uint32_t a_, VtOut vt = VtOut{nullptr, 0, 0, 0}) {
    return launch_gemm(a, (const __nv_bfloat16*)w, bias, res, o, L->status, T, N, K, n_seqs_dev, n, a_, sm, st, vt);
  };
  // the V third of the q|k|v product is written transposed per head (what the attention kernel reads)
  const VtOut vt_out{L->vt, 2 * d, attention_vt_pitch(n), D.heads};
  auto ln = [&](const __nv_bfloat16* in, const float* g, const float* b, __nv_bfloat16* o) {
    return launch_layernorm(in, g, b, o, T, d, n_seqs_dev, n, D.eps, sm, st);
  };
  if (!D.pre_ln) {
    e = gemm(X, D.w_qkv, D.b_qkv, nullptr, L->qkv, 3 * d, d, LAYER_ACT_NONE, vt_out);
    if (e == cudaSuccess) e = launch_attention_tc(L->qkv, L->vt, L->a, L->status, n, d, D.heads, n_seqs, n_seqs_dev, D.causal, st);
    if (e == cudaSuccess) e = gemm(L->a, D.w_o, D.b_o, X, L->t, d, d, LAYER_ACT_NONE);
    if (e == cudaSuccess) e = ln(L->t, D.ln1_g, D.ln1_b, L->y);
    if (e == cudaSuccess) e = gemm(L->y, D.w_1, D.b_1, nullptr, L->f, D.ffn, d, act);
    if (e == cudaSuccess) e = gemm(L->f, D.w_2, D.b_2, L->y, L->t, d, D.ffn, LAYER_ACT_NONE);
    if (e == cudaSuccess) e = ln(L->t, D.ln2_g, D.ln2_b, O);
  } else {
    e = ln(X, D.ln1_g, D.ln1_b, L->y);
    if (e == cudaSuccess) e = gemm(L->y, D.w_qkv, D.b_qkv, nullptr, L->qkv, 3 * d, d, LAYER_ACT_NONE, vt_out);
    if (e == cudaSuccess) e = launch_attention_tc(L->qkv, L->vt, L->a, L->status, n, d, D.heads, n_seqs, n_seqs_dev, D.causal, st);
    if (e == cudaSuccess) e = gemm(L->a, D.w_o, D.b_o, X, L->t, d, d, LAYER_ACT_NONE);
    if (e == cudaSuccess) e = ln(L->t, D.ln2_g, D.ln2_b, L->y);
    if (e == cudaSuccess) e = gemm(L->y, D.w_1, D.b_1, nullptr, L->f, D.ffn, d, act);
    if (e == cudaSuccess) e = gemm(L->f, D.w_2, D.b_2, L->t, O, d, D.ffn, LAYER_ACT_NONE);
  }
  if (prev != L->desc.device) cudaSetDevice(prev);
  if (e != cudaSuccess) { cudaGetLastError(); return LLMCACHE_ERR_CUDA; }
  return LLMCACHE_OK;
}

int llmcache_layer_status(llmcache_layer_t* L) {
  if (!L) return LLMCACHE_ERR_ARG;
  uint32_t s = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(&s, L->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  return s ? LLMCACHE_ERR_TIMEOUT : LLMCACHE_OK;
}

int llmcache_layer_debug_knobs(llmcache_layer_t* L, uint64_t wait_limit_ns, uint32_t flags) {
  if (!L) return LLMCACHE_ERR_ARG;
  uint32_t w[3] = {flags, (uint32_t)(wait_limit_ns & 0xFFFFFFFFull), (uint32_t)(wait_limit_ns >> 32)};
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(L->status + 1, w, sizeof(w), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return LLMCACHE_ERR_CUDA;
  }
  return LLMCACHE_OK;
}

// Algorithm 1 with fingerprint-on-write: only layer 1 pools its input; every later probe takes the position means
// that the previous layer's row movers produced.  pooled == nullptr: each bank's own buffer carries them.
static int infer_fused(llmcache_bank_t** banks, llmcache_layer_t** layers, uint32_t n_layers, const void* h0,
                       uint32_t B, float tau, void* buf_a, void* buf_b, void* h_miss, void* miss_out,
                       llmcache_probe_io* io, float* pooled, void** h_final, void* stream) {
  const void* cur = h0;
  void* bufs[2] = {buf_a, buf_b};
  const float* prev_means = nullptr;
  int rc = LLMCACHE_OK;
  for (uint32_t l = 0; l < n_layers && rc == LLMCACHE_OK; ++l) {
    void* next = bufs[l & 1u];
    const uint32_t ld = banks[l]->desc.d_model;
    float* means_out = pooled ? pooled : banks[l]->a.pooled_own;
    io->h_miss = h_miss;
    // the rows this layer writes are summed on the way: means_out then holds the next layer's position means.
    // (With one shared buffer the probe has consumed its previous contents before the commit overwrites them.)
    rc = llmcache_bank_pool_out(banks[l], l + 1 < n_layers ? means_out : nullptr, ld);
    if (rc != LLMCACHE_OK) break;
    if (l == 0) rc = llmcache_probe(banks[l], cur, B, tau, next, io, stream);
    else        rc = llmcache_probe_pooled(banks[l], prev_means, ld, cur, B, tau, next, io, stream);
    if (rc == LLMCACHE_OK) rc = llmcache_layer_forward(layers[l], h_miss, B, io->counts + 1, miss_out, stream);
    if (rc == LLMCACHE_OK) rc = llmcache_commit(banks[l], miss_out, io, next, nullptr, stream);
    if (rc == LLMCACHE_OK) rc = llmcache_bank_pool_out(banks[l], nullptr, 0);
    prev_means = means_out;
    cur = next;
  }
  if (rc != LLMCACHE_OK) return rc;
  *h_final = const_cast<void*>(cur);
  return LLMCACHE_OK;
}

int llmcache_infer(llmcache_bank_t** banks, llmcache_layer_t** layers, uint32_t n_layers, const void* h0, uint32_t B,
                   float tau, void* buf_a, void* buf_b, void* h_miss, void* miss_out, llmcache_probe_io* io,
                   void** h_final, void* stream) {
  if (!layers || !h0 || !buf_a || !buf_b || !h_final || n_layers == 0) return LLMCACHE_ERR_ARG;
  if (banks && (!io || !h_miss || !miss_out)) return LLMCACHE_ERR_ARG;
  if (banks) {
    // banks created with fused_pool (all of them, same width) take the fingerprint-on-write path by themselves
    bool fused = true;
    for (uint32_t l = 0; l < n_layers; ++l)
      fused = fused && banks[l] && banks[l]->a.pooled_own && banks[l]->desc.d_model == banks[0]->desc.d_model &&
              B <= banks[l]->desc.max_batch;
    if (fused) return infer_fused(banks, layers, n_layers, h0, B, tau, buf_a, buf_b, h_miss, miss_out, io, nullptr,
                                  h_final, stream);
  }
  const void* cur = h0;
  void* bufs[2] = {buf_a, buf_b};
  for (uint32_t l = 0; l < n_layers; ++l) {
    void* next = bufs[l & 1u];
    int rc;
    if (banks) {
      // Algorithm 1: lookup (hits take the stored output), layer on the compacted misses, insert
      io->h_miss = h_miss;
      rc = llmcache_probe(banks[l], cur, B, tau, next, io, stream);
      if (rc == LLMCACHE_OK) rc = llmcache_layer_forward(layers[l], h_miss, B, io->counts + 1, miss_out, stream);
      if (rc == LLMCACHE_OK) rc = llmcache_commit(banks[l], miss_out, io, next, nullptr, stream);
    } else {
      rc = llmcache_layer_forward(layers[l], cur, B, nullptr, next, stream);    // no caching: every layer in full
    }
    if (rc != LLMCACHE_OK) return rc;
    cur = next;
  }
  *h_final = const_cast<void*>(cur);
  return LLMCACHE_OK;
}

int llmcache_infer_pooled(llmcache_bank_t** banks, llmcache_layer_t** layers, uint32_t n_layers, const void* h0,
                          uint32_t B, float tau, void* buf_a, void* buf_b, void* h_miss, void* miss_out,
                          llmcache_probe_io* io, float* pooled, void** h_final, void* stream) {
  if (!banks || !layers || !h0 || !buf_a || !buf_b || !h_final || n_layers == 0) return LLMCACHE_ERR_ARG;
  if (!io || !h_miss || !miss_out || !pooled) return LLMCACHE_ERR_ARG;
  return infer_fused(banks, layers, n_layers, h0, B, tau, buf_a, buf_b, h_miss, miss_out, io, pooled, h_final, stream);
}

}  // extern "C"
