// Internal structures of the decoder engine and the launchers of its kernels.
#pragma once

#include <cuda.h>
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
    // Tensor-core path: the library's own tile-major copies of the block matrices
    // and of the LM head (ln1 / ln2 of these entries are unused).
    std::vector<spec_layer_weights> packed;
    const void* packed_head = nullptr;

    // KV pool of layer l: kv + l * layer_stride bytes, laid out
    // [n_pages][2 (K, V)][n_kv_heads][page_size][d_head] in kv_elem_bytes-wide elements.
    void* kv = nullptr;
    size_t layer_stride = 0;
    int kv_elem_bytes = 4;
    int kv_dtype = SPEC_DTYPE_FP32;  // SPEC_DTYPE_FP32 / FP16 / BF16
    const float2* rope_table = nullptr;  // Llama: (cos, sin) [positions][d_head / 2], owned

    // Encoder-decoder (T5) only.  The bias tables are the bucket tables expanded by
    // relative position: [n_heads][span], entry (key pos - query pos) + zero.
    std::vector<spec_layer_weights> enc_layers, enc_packed;
    const float* enc_ln_f = nullptr;
    const float* enc_bias = nullptr;  // span 2 * max_src_len - 1, zero max_src_len - 1, owned
    const float* dec_bias = nullptr;  // span max_len, zero max_len - 1 (only keys at or before the query), owned
    void* enc_kv = nullptr;           // K,V of the encoder block being computed (one layer's pool), owned
    void* cross_kv = nullptr;         // cross-attention K,V of decoder layer l: cross_kv + l * cross_stride, owned
    size_t cross_stride = 0;
    bool t5() const { return cfg.arch == SPEC_ARCH_T5; }

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

// A table model's logits: logits[dst(i)] = table[token[src(i)]] (table [vocab, vocab], fp32 or bf16).
int launch_table_logits(const void* table, bool bf16, int vocab, const int32_t* token, const int32_t* src_rows,
                        const int32_t* dst_rows, int n_rows, float* logits, cudaStream_t stream);

// Row i of the output = RMSNorm(h[src(i)]) * gain, as fp32 (`out`) and/or as two
// bf16 terms (`out_hi`, `out_lo`).  If `partial` is given (split-K results of
// the GEMM before, [splits][rows_total][d]) it is first added into h.
// Copy-from-context draft: one-hot logits at the token that followed the last `ngram` tokens before.
int launch_copy_logits(const int32_t* tokens, int max_len, const int32_t* length, const int32_t* draft_tokens, int gamma,
                       const RowMeta& rows, const int32_t* src_rows, const int32_t* dst_rows, int n_rows, int ngram,
                       int vocab, float* logits, cudaStream_t stream);
int launch_norm(float* h, const float* partial, int splits, int rows_total, const float* gain, const int32_t* src_rows,
                int n_rows, int d, float eps, float* out, __nv_bfloat16* out_hi, __nv_bfloat16* out_lo,
                cudaStream_t stream);

// y[dst(r)] = x[r] . W^T (+ residual[r]) on the FMA pipes;  W is [n_out, k] row-major in fp32 or bf16.
// dst(r) = dst_rows ? dst_rows[r] : r.  y and residual may alias.
int launch_gemm_rows(const float* x, const void* w, bool w_bf16, const float* residual, const int32_t* dst_rows,
                     int n_rows, int n_out, int k, float* y, cudaStream_t stream);

// Tensor-core path for bf16 weights (gemm_tc.cu): x arrives as two bf16 terms;
// launch_gemm_tc_partials leaves the split-K partial sums [splits][n_rows][n_out]
// for the next kernel to add up, launch_gemm_tc adds them up itself.
int gemm_tc_splits(int n_out, int k, int n_rows);
size_t gemm_tc_partial_elems(int n_out, int k, int n_rows);
int launch_split_bf16(const float* x, size_t n, __nv_bfloat16* hi, __nv_bfloat16* lo, cudaStream_t stream);
// `packed`: w is the tile-major copy made by launch_pack_weight (every [128 x 64]
// tile contiguous, so a CTA's weight stream is one sequential run of HBM).
size_t packed_weight_elems(int n_out, int k);
int launch_pack_weight(const void* w, int n_out, int k, void* out, cudaStream_t stream);
int launch_gemm_tc_partials(const __nv_bfloat16* hi, const __nv_bfloat16* lo, int hi_rows, const void* w, bool packed,
                            int n_rows, int n_out, int k, float* partial, cudaStream_t stream);
int launch_gemm_tc(const __nv_bfloat16* hi, const __nv_bfloat16* lo, int hi_rows, const void* w, bool packed,
                   const float* residual, const int32_t* dst_rows, int n_rows, int n_out, int k, float* partial,
                   float* y, cudaStream_t stream);
int gemm_tc_take_error();

// Where the K,V rows of a pass go / come from: one layer's pool
// [n_pages][2 (K, V)][n_kv_heads][page_size][d_head] and the table that maps
// (sequence slot, position / page_size) to a pool page.
struct KvPool {
    void* kv;
    int elem_bytes;  // 4 (fp32) or 2 (fp16, bf16)
    int dtype;       // SPEC_DTYPE_*
    const int32_t* page_table;
    int pages_per_seq;
    int page_size;
    int n_pages;  // pages in the pool (of one layer)
};

// Finishes a projection GEMM whose output row is [n_heads q heads | n_kv_heads k
// heads | n_kv_heads v heads] (optional split-K partial sums): rotary positions
// on q and k when `rope` is given, q heads left in `qkv`, K,V heads of every
// active row appended to the pool.  n_kv_heads = 0: queries only; n_heads = 0:
// K,V only.
int launch_qkv(int n_heads, int n_kv_heads, int d_head, const float2* rope, const KvPool& pool, const RowMeta& rows,
               int n_rows, float* qkv, const float* partial, int splits, cudaStream_t stream);
void fill_rope_table(std::vector<float2>& table, int positions, int d_head, double base);

// One attention call: head h of query row r is at q + r * q_stride + h * d_head.
// kv_len == nullptr: causal over the pool (row at position p sees keys 0..p);
// otherwise every active row of sequence slot s sees keys 0..kv_len[s]-1.
// bias (optional): score of (row at position p, key at position k, head h) gets
// bias[h * bias_span + (k - p) + bias_zero] added after scaling.
struct AttnSource {
    const float* q;
    int q_stride;
    KvPool pool;
    const int32_t* kv_len;
    const float* bias;
    int bias_span;
    int bias_zero;
};

// att[r, h] = softmax(scores) V for the rows of a pass; rows of sequence b are
// rows b*m_rows .. of the pass.  Output as fp32 and/or two bf16 terms.
int attention_slices(const Model& m, int batch, int m_rows, int max_len);
struct AttentionPlan {
    int tensor_cores, slices, cluster_merge, in_turn;
};
AttentionPlan attention_plan(const Model& m, int batch, int m_rows, int max_keys);
size_t attention_partial_elems(int rows, int n_heads, int d_head, int slices);
// (slices from attention_slices with the same batch, m_rows and max_keys, the capacity of the key set)
int launch_attention(const Model& m, const AttnSource& src, const RowMeta& rows, int batch, int m_rows, int slices,
                     int max_keys, float* part, float* att, __nv_bfloat16* att_hi, __nv_bfloat16* att_lo, cudaStream_t stream);

// f = gelu(u)  |  gelu(u[:, :F]) * u[:, F:]  |  silu(u[:, :F]) * u[:, F:], u given in full or as partial sums.
int launch_ffn_act(const float* u, const float* partial, int splits, int n_rows, int d_ff, int ffn, float* f,
                   __nv_bfloat16* f_hi, __nv_bfloat16* f_lo, cudaStream_t stream);

// mega.cu: one forward pass over at most 16 rows as one persistent cooperative kernel
// (bf16 decoder-only models).
struct PassScratch {
    float *h = nullptr, *ssq[2] = {nullptr, nullptr}, *part[2] = {nullptr, nullptr};
    float *out = nullptr, *att = nullptr, *attn_part = nullptr;
    unsigned *sync = nullptr, *ticket[2] = {nullptr, nullptr};
    int ticket_count = 0;
    void* layers[2] = {nullptr, nullptr};  // per model: device array of its blocks' pointers (nullptr: not served)
    void* tile_counts[2] = {nullptr, nullptr};  // per model: parts per tile of every GEMM kind (bytes)
    int count_offset[2][7] = {};
    int count_total[2] = {0, 0};
    int ctas = 0;                          // 0: the kernel is not available
};
struct PassTables {
    const int32_t* page_table;
    int pages_per_seq, page_size;
    const int32_t* src_page_table;
    int src_pages_per_seq;
    const int32_t* src_len;
    int bias_span, bias_zero;
};
int pass_scratch_init(PassScratch& s, const Model* models, int n_models, std::vector<void*>& allocations);
bool pass_kernel_serves(const PassScratch& s, const Model& m, int which, int n_rows, int n_logit_rows);
int launch_pass(const PassScratch& s, const Model& m, int which, const RowMeta& rows, const PassTables& t, int batch, int m_rows,
                int n_logit_rows, const int32_t* logit_src, const int32_t* logit_dst, float* logits, cudaStream_t stream,
                unsigned long long* trace = nullptr, int trace_capacity = 0);
void pass_scratch_release(PassScratch& s);
int pass_take_error();

// A tensor map over `rows` rows of `cols` (64 or 128) fp16 elements starting at `base`, fetched in boxes of 64 elements
// by 32 rows with the 128-byte swizzle; maps are cached by (base, rows, cols).  gemm_tc.cu
int cached_f16_rows_map(const void* base, unsigned long long rows, int cols, CUtensorMap* out);
// Non-zero (and cleared) if the f16 attention kernel gave up on a bounded wait for a tile.  attention.cu
int attention_take_error();

// sampling.cu
int launch_verify_sample(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                         const float* uniforms, const float* final_uniforms, int batch, int gamma, int vocab,
                         float temperature, float lenience, int top_k, float top_p, int32_t* n_accepted,
                         int32_t* next_token, void* workspace, cudaStream_t stream, int* nonfinite = nullptr);
// (`nonfinite`, optional device word: set to 1 if a row holds a NaN or +inf logit, or no finite logit at all)
// top_k = 0 and top_p = 1: the whole vocabulary; otherwise floor_scratch holds one float per row.
int launch_sample(const float* logits, const float* uniforms, int rows, int vocab, float temperature, int top_k,
                  float top_p, float* floor_scratch, int32_t* tokens, cudaStream_t stream);
int launch_sample_strided(const float* logits, size_t logit_stride, const float* uniforms, int uniform_stride,
                          int rows, int vocab, float temperature, int top_k, float top_p, float* floor_scratch,
                          int32_t* tokens, int token_stride, cudaStream_t stream, int* nonfinite = nullptr);
size_t verify_sample_workspace_bytes(int batch, int gamma, int vocab);

}  // namespace spec
