// Internal structures of the decoder engine and the launchers of its kernels.
#pragma once

#include <cuda_bf16.h>

#include <vector>

#include "common.cuh"

namespace spec {

// One decoder (target or draft): borrowed weights, owned KV pages.
struct Model {
    spec_model_cfg cfg{};
    const void* tok_emb = nullptr;
    const void* pos_emb = nullptr;
    const float* ln_f = nullptr;
    const void* head = nullptr;  // == tok_emb when tied
    std::vector<spec_layer_weights> layers;

    // KV pool of layer l: kv + l * layer_stride bytes, laid out
    // [n_pages][2 (K, V)][n_kv_heads][page_size][d_head] in kv_elem_bytes-wide elements.
    void* kv = nullptr;
    size_t layer_stride = 0;
    int kv_elem_bytes = 4;

    int q_dim() const { return cfg.n_heads * cfg.d_head; }
    int kv_dim() const { return cfg.n_kv_heads * cfg.d_head; }
    int qkv_dim() const { return q_dim() + 2 * kv_dim(); }
    int ffn_in_dim() const { return cfg.ffn == SPEC_FFN_GELU ? cfg.d_ff : 2 * cfg.d_ff; }
    bool bf16() const { return cfg.dtype == SPEC_DTYPE_BF16; }
};

// Row descriptors of one forward pass (device arrays of `rows` entries).
// A row with pos < 0 is inactive: it is computed but writes no K,V.
struct RowMeta {
    const int32_t* token;
    const int32_t* pos;
    const int32_t* seq;
};

// ---- kernel launchers (all asynchronous on `stream`) ------------------------

// h[r] = tok_emb[token[r]] (+ pos_emb[pos[r]] for GPT), fp32.
int launch_embed(const Model& m, const RowMeta& rows, int n_rows, float* h, cudaStream_t stream);

// out[i] = in[src[i]] / sqrt(mean(in[src[i]]^2) + eps) * gain   (src == nullptr: identity)
int launch_rmsnorm(const float* in, const float* gain, const int32_t* src_rows, int n_rows, int d, float eps,
                   float* out, cudaStream_t stream);

// y[dst(r)] = x[r] . W^T (+ residual[r]);  W is [n_out, k] row-major in fp32 or bf16.
// dst(r) = dst_rows ? dst_rows[r] : r.  y and residual may alias.
int launch_gemm_rows(const float* x, const void* w, bool w_bf16, const float* residual, const int32_t* dst_rows,
                     int n_rows, int n_out, int k, float* y, cudaStream_t stream);

// Tensor-core path for bf16 weights (gemm_tc.cu): x is first split into two bf16
// terms, partial sums of the split-K grid are reduced in a fixed order.
int gemm_tc_splits(int n_out, int k, int n_rows);
size_t gemm_tc_partial_elems(int n_out, int k, int n_rows);
int launch_split_bf16(const float* x, size_t n, __nv_bfloat16* hi, __nv_bfloat16* lo, cudaStream_t stream);
int launch_gemm_tc(const __nv_bfloat16* hi, const __nv_bfloat16* lo, int hi_rows, const void* w, const float* residual,
                   const int32_t* dst_rows, int n_rows, int n_out, int k, float* partial, float* y,
                   cudaStream_t stream);
int gemm_tc_take_error();

// Rotary positions on q and k (Llama), then K,V rows of every active row into the paged cache.
int launch_rope_append(const Model& m, int layer, const RowMeta& rows, int n_rows, float* qkv,
                       const int32_t* page_table, int pages_per_seq, int page_size, cudaStream_t stream);

// att[r, h] = softmax(q_r,h . K / sqrt(d_head)) V over cached positions <= pos[r] of sequence seq[r].
int launch_attention(const Model& m, int layer, const RowMeta& rows, int n_rows, const float* qkv, float* att,
                     const int32_t* page_table, int pages_per_seq, int page_size, cudaStream_t stream);

// f = gelu(u)  |  gelu(u[:, :F]) * u[:, F:]  |  silu(u[:, :F]) * u[:, F:]
int launch_ffn_act(const float* u, int n_rows, int d_ff, int ffn, float* f, cudaStream_t stream);

// sampling.cu
int launch_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                         const float* uniforms, const float* final_uniforms, int batch, int gamma, int vocab,
                         float temperature, int32_t* n_accepted, int32_t* next_token, void* workspace,
                         cudaStream_t stream);
int launch_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature,
                  int32_t* tokens, cudaStream_t stream);
int launch_sample_strided(const float* logits, size_t logit_stride, const float* uniforms, int uniform_stride,
                          int rows, int vocab, float temperature, int32_t* tokens, int token_stride,
                          cudaStream_t stream);
size_t verify_sample_workspace_bytes(int batch, int gamma, int vocab);

}  // namespace spec
