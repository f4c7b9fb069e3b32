// Miss-path transformer layer: shared declarations.
#pragma once
#include "llmcache_internal.cuh"

namespace llmc {

enum { LAYER_ACT_NONE = 0, LAYER_ACT_GELU_ERF = 1, LAYER_ACT_GELU_TANH = 2 };

// Where the columns from col0 on of a dense layer's output go instead of `out`: transposed per head of 64
// columns, vt[((seq * heads + h) * 64 + c) * pitch + pos] (ptr == nullptr: nowhere, everything goes to `out`).
struct VtOut { __nv_bfloat16* ptr; uint32_t col0, pitch, heads; };

cudaError_t setup_gemm_kernel();
cudaError_t launch_gemm(const __nv_bfloat16* a, const __nv_bfloat16* w, const float* bias,
                        const __nv_bfloat16* residual, __nv_bfloat16* out, uint32_t* status, uint32_t M_max,
                        uint32_t N, uint32_t K, const uint32_t* m_seq_dev, uint32_t rows_per_seq, uint32_t act,
                        int sm_count, cudaStream_t st, VtOut vt = VtOut{nullptr, 0, 0, 0});

cudaError_t launch_layernorm(const __nv_bfloat16* x, const float* g, const float* b, __nv_bfloat16* y, uint32_t M_max,
                             uint32_t d, const uint32_t* m_seq_dev, uint32_t rows_per_seq, float eps, int sm_count,
                             cudaStream_t st);
// h0 = token embeddings + position embeddings (pos_emb may be null), optionally layer-normed (gain, bias may be null)
cudaError_t launch_embed(const long long* tokens, const __nv_bfloat16* tok_emb, const __nv_bfloat16* pos_emb,
                         const float* gain, const float* bias, __nv_bfloat16* h0, uint32_t* bad_ids,
                         unsigned long long rows, uint32_t n, uint32_t d, long long vocab, int layer_norm, float eps,
                         int sm_count, cudaStream_t st);
// Attention on the tcgen05 tensor cores; vt: scratch for the per-head transposes of V,
// seq_max * heads * 64 rows of attention_vt_pitch(n) elements.
cudaError_t setup_attention_kernel();
uint32_t attention_vt_pitch(uint32_t n);
// vt must hold the per-head transposes of V already (written by the q|k|v product, see VtOut)
cudaError_t launch_attention_tc(const __nv_bfloat16* qkv, const __nv_bfloat16* vt, __nv_bfloat16* out, uint32_t* status,
                                uint32_t n, uint32_t d, uint32_t heads, uint32_t seq_max, const uint32_t* m_seq_dev,
                                int causal, cudaStream_t st);

}  // namespace llmc
