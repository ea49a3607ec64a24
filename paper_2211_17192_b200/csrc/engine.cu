// Decoder engine: context set-up, the forward pass over a set of rows, the
// device-resident generation loop of Algorithm 1 (draft steps, parallel
// verification, speculative sampling, commit + roll-back) replayed as a CUDA
// graph, and the teacher-forced diagnostics used by the parity tests.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "model.cuh"

struct spec_ctx {
    spec::Model model[2];  // 0 target, 1 draft
    bool has_draft = false;
    spec_runtime_cfg rt{};
    cudaStream_t stream = nullptr;
    cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};
    int max_rows = 0;       // rows of any pass (activations)
    int max_logit_rows = 0;  // rows of the generation loop's logits buffers
    int pages_per_seq = 0;
    // encoder-decoder contexts: the sources' own page table and lengths
    int src_pages_per_seq = 0;
    int32_t *src_page_table = nullptr, *src_len = nullptr;
    bool encoded = false;
    int encoded_batch = 0;

    // activations (sized for the wider model)
    float *h = nullptr, *a = nullptr, *qkv = nullptr, *att = nullptr, *u = nullptr, *f = nullptr;
    float *target_logits = nullptr, *draft_logits = nullptr;
    // tensor-core GEMM path: bf16 hi/lo copies of the GEMM input, split-K partial sums
    __nv_bfloat16 *x_hi = nullptr, *x_lo = nullptr;
    float* partials = nullptr;
    unsigned long long* pass_trace = nullptr;  // set while spec_pass_trace runs
    int pass_trace_capacity = 0;
    float* attn_part = nullptr;  // per key slice: (max, sum, accumulator) of every (row, head)
    int hi_rows = 0;
    spec::PassScratch pass;  // the persistent pass kernel's scratch (passes of at most 16 rows of a bf16 model)
    int32_t *row_token = nullptr, *row_pos = nullptr, *row_seq = nullptr, *logit_src = nullptr, *logit_dst = nullptr;
    int32_t* page_table = nullptr;

    // generation state (device)
    int32_t *tokens = nullptr, *length = nullptr, *prompt_len = nullptr, *draft_tokens = nullptr;
    int32_t *n_accepted = nullptr, *next_token = nullptr;
    float *draft_u = nullptr, *accept_u = nullptr, *final_u = nullptr;
    unsigned long long* counters = nullptr;  // iterations, tokens, tests evaluated, tests passed, then iterations by n = 0 .. 64
    int* nonfinite = nullptr;                // set by the sampling kernels when a row holds a NaN or +inf logit
    void* sampler_ws = nullptr;
    struct Params { unsigned long long seed; int n_new; float imposed_alpha; }* params = nullptr;
    float imposed_alpha = -1.0f;  // >= 0: timing instrument, see spec_set_imposed_acceptance
    float lenience = 1.0f;        // Appendix A.5; 1 = Algorithm 1 as printed
    int iteration_gamma = 0;      // gamma of the iteration being enqueued (the copy draft indexes the guesses by it)
    int top_k = 0;                // Section 2.2: both models standardised over their k largest logits; 0 = all
    float top_p = 1.0f;           // and then over the nucleus of mass top_p; 1 = all
    float* sample_floors = nullptr;  // the draft rows' k-th largest logits, one per sequence

    // cached iteration graphs, one per gamma, all for the same batch and sampling settings
    std::vector<cudaGraphExec_t> graphs;  // indexed by gamma; nullptr = not captured yet
    cudaGraphExec_t graph = nullptr;      // the one in use (an element of `graphs`)
    int graph_batch = -1, graph_gamma = -1;
    float graph_temperature = -1.0f, graph_lenience = 1.0f;
    int graph_top_k = 0;
    float graph_top_p = 1.0f;

    // generation in progress (spec_begin / spec_generate)
    int session_batch = 0, session_gamma = 0, session_n_new = 0;
    float session_temperature = 0.0f;
    int session_gamma_cap = 0;  // the gamma the session's capacity was checked for (spec_set_gamma stays below it)
    long long session_replays = 0, session_draft_passes = 0;
    float session_prefill_ms = 0.0f;
    std::vector<int32_t> session_prompt_len;

    // host-side cached lengths for the diagnostics
    std::vector<int32_t> cached[2];
    std::vector<void*> allocations;
};

namespace spec {
namespace {

constexpr int kCounters = 4 + 65;  // see spec_ctx::counters

int check_cfg(const spec_model_cfg& c, const char* which) {
    if (c.arch == SPEC_ARCH_BIGRAM) {
        if (c.vocab < 1 || (c.dtype != SPEC_DTYPE_FP32 && c.dtype != SPEC_DTYPE_BF16))
            return fail(SPEC_ERR_BAD_CONFIG, "%s: a table model needs vocab >= 1 and a known dtype", which);
        return SPEC_OK;
    }
    if (c.arch == SPEC_ARCH_COPY) {
        if (c.vocab < 1 || c.ngram < 1 || c.ngram > 64)
            return fail(SPEC_ERR_BAD_CONFIG, "%s: a copy model needs vocab >= 1 and 1 <= ngram <= 64", which);
        return SPEC_OK;
    }
    if (c.arch != SPEC_ARCH_GPT && c.arch != SPEC_ARCH_LLAMA && c.arch != SPEC_ARCH_T5)
        return fail(SPEC_ERR_BAD_CONFIG, "%s: unknown arch %d", which, c.arch);
    if (c.arch == SPEC_ARCH_T5) {
        if (c.n_enc_layers < 1 || c.n_kv_heads != c.n_heads || c.tied_embeddings)
            return fail(SPEC_ERR_BAD_CONFIG, "%s: encoder-decoder needs n_enc_layers >= 1, n_kv_heads == n_heads, an untied head", which);
        if (c.rel_buckets < 4 || c.rel_buckets > 256 || c.rel_buckets % 4 || c.rel_max_distance <= c.rel_buckets / 2)
            return fail(SPEC_ERR_BAD_CONFIG, "%s: rel_buckets %d (multiple of 4, 4..256) / rel_max_distance %d", which, c.rel_buckets, c.rel_max_distance);
    }
    if (c.n_layers < 1 || c.d_model < 8 || c.n_heads < 1 || c.n_kv_heads < 1 || c.d_ff < 8 || c.vocab < 1 || c.max_positions < 1)
        return fail(SPEC_ERR_BAD_CONFIG, "%s: non-positive dimension", which);
    if (c.d_head != 64 && c.d_head != 128) return fail(SPEC_ERR_BAD_CONFIG, "%s: d_head %d (64 or 128 supported)", which, c.d_head);
    if (c.n_heads % c.n_kv_heads) return fail(SPEC_ERR_BAD_CONFIG, "%s: n_kv_heads must divide n_heads", which);
    if (c.d_model % 8 || c.d_ff % 8) return fail(SPEC_ERR_BAD_CONFIG, "%s: d_model and d_ff must be multiples of 8", which);
    if (c.ffn < SPEC_FFN_GELU || c.ffn > SPEC_FFN_SWIGLU) return fail(SPEC_ERR_BAD_CONFIG, "%s: unknown ffn %d", which, c.ffn);
    if (c.dtype != SPEC_DTYPE_FP32 && c.dtype != SPEC_DTYPE_BF16) return fail(SPEC_ERR_BAD_CONFIG, "%s: unknown dtype %d", which, c.dtype);
    if (!(c.rms_eps >= 0.0f)) return fail(SPEC_ERR_BAD_CONFIG, "%s: rms_eps", which);
    return SPEC_OK;
}

template <typename T>
int dev_alloc(spec_ctx* ctx, T** out, size_t count) {
    void* p = nullptr;
    const cudaError_t err = cudaMalloc(&p, std::max<size_t>(count, 1) * sizeof(T));
    if (err != cudaSuccess) {
        cudaGetLastError();
        return fail(SPEC_ERR_OOM, "cudaMalloc of %zu bytes failed: %s", count * sizeof(T), cudaGetErrorString(err));
    }
    ctx->allocations.push_back(p);
    *out = static_cast<T*>(p);
    return SPEC_OK;
}

#define SPEC_TRY(expr)                    \
    do {                                  \
        const int status__ = (expr);      \
        if (status__ != SPEC_OK) return status__; \
    } while (0)

// The GEMMs and hand-offs of a pass on either path.  bf16 models take the
// tensor-core path: every GEMM leaves split-K partial sums that the next small
// kernel adds up (a GEMM that closes a residual branch leaves them pending until
// the next norm adds them into h), and every GEMM input is produced directly as
// two bf16 terms.  fp32 models run the same kernels with fp32 hand-offs and the
// FMA-pipe GEMM.
struct Pass {
    spec_ctx* ctx;
    const Model& m;
    int n_rows;
    bool tc;
    cudaStream_t st;
    int pending = 0;      // split count of partial sums not yet added into h
    int last_splits = 0;  // split count of the last projection

    __nv_bfloat16* hi() const { return ctx->x_hi; }
    __nv_bfloat16* lo() const { return ctx->x_lo; }

    // a (fp32) or hi/lo = rmsnorm(h[src(i)]) * gain for i < n
    int norm(const float* gain, const int32_t* src_rows, int n) {
        const int d = m.cfg.d_model;
        const int status = tc ? launch_norm(ctx->h, pending ? ctx->partials : nullptr, pending, n_rows, gain, src_rows, n, d,
                                            m.cfg.rms_eps, nullptr, hi(), lo(), st)
                              : launch_norm(ctx->h, nullptr, 0, n_rows, gain, src_rows, n, d, m.cfg.rms_eps, ctx->a, nullptr,
                                            nullptr, st);
        pending = 0;
        return status;
    }
    // y = x . W^T for a consumer that is not the residual stream: partial sums (tc) or `y` (fp32 path, input `x`)
    int proj(const void* w, const void* pw, int n_out, int k, const float* x, float* y) {
        if (tc) {
            last_splits = gemm_tc_splits(n_out, k, n_rows);
            return launch_gemm_tc_partials(hi(), lo(), ctx->hi_rows, pw, true, n_rows, n_out, k, ctx->partials, st);
        }
        return launch_gemm_rows(x, w, m.bf16(), nullptr, nullptr, n_rows, n_out, k, y, st);
    }
    // h += x . W^T
    int residual(const void* w, const void* pw, int k, const float* x) {
        const int d = m.cfg.d_model;
        if (tc) {
            pending = gemm_tc_splits(d, k, n_rows);
            return launch_gemm_tc_partials(hi(), lo(), ctx->hi_rows, pw, true, n_rows, d, k, ctx->partials, st);
        }
        return launch_gemm_rows(x, w, m.bf16(), ctx->h, nullptr, n_rows, d, k, ctx->h, st);
    }
    const float* partials() const { return tc ? ctx->partials : nullptr; }
    // h += FFN(rmsnorm(h) * gain)
    int ffn(const spec_layer_weights& w, const spec_layer_weights& pw) {
        const spec_model_cfg& c = m.cfg;
        SPEC_TRY(norm(w.ln2, nullptr, n_rows));
        SPEC_TRY(proj(w.w_in, pw.w_in, m.ffn_in_dim(), c.d_model, ctx->a, ctx->u));
        SPEC_TRY(launch_ffn_act(tc ? nullptr : ctx->u, partials(), last_splits, n_rows, c.d_ff, c.ffn, tc ? nullptr : ctx->f,
                                tc ? hi() : nullptr, tc ? lo() : nullptr, st));
        return residual(w.w_out, pw.w_out, c.d_ff, ctx->f);
    }
    // h += Wo . attention(projection of rmsnorm(h) * gain) over `pool`
    int self_attention(const spec_layer_weights& w, const spec_layer_weights& pw, const RowMeta& rows, int batch, int m_rows,
                       const KvPool& pool, const int32_t* kv_len, const float* bias, int bias_span, int bias_zero,
                       int max_keys) {
        const spec_model_cfg& c = m.cfg;
        SPEC_TRY(norm(w.ln1, nullptr, n_rows));
        SPEC_TRY(proj(w.wqkv, pw.wqkv, m.qkv_dim(), c.d_model, ctx->a, ctx->qkv));
        SPEC_TRY(launch_qkv(c.n_heads, c.n_kv_heads, c.d_head, c.arch == SPEC_ARCH_LLAMA ? m.rope_table : nullptr, pool, rows,
                            n_rows, ctx->qkv, partials(), last_splits, st));
        const int slices = attention_slices(m, batch, m_rows, max_keys);
        const AttnSource src{ctx->qkv, m.qkv_dim(), pool, kv_len, bias, bias_span, bias_zero};
        SPEC_TRY(launch_attention(m, src, rows, batch, m_rows, slices, max_keys, ctx->attn_part, tc ? nullptr : ctx->att,
                                  tc ? hi() : nullptr, tc ? lo() : nullptr, st));
        return residual(w.wo, pw.wo, m.q_dim(), ctx->att);
    }
};

// Non-zero (and cleared) if a tensor-core GEMM or the persistent pass kernel gave up on a bounded wait.
int device_gave_up(spec_ctx* ctx) {
    const int gemm = gemm_tc_take_error(), pass = pass_take_error(), attn = attention_take_error();
    return gemm ? gemm : pass ? pass : attn;
}

KvPool layer_pool(const spec_ctx* ctx, const Model& m, int layer) {
    return KvPool{static_cast<char*>(m.kv) + static_cast<size_t>(layer) * m.layer_stride, m.kv_elem_bytes, m.kv_dtype, ctx->page_table,
                  ctx->pages_per_seq, ctx->rt.page_size, ctx->rt.max_batch * ctx->pages_per_seq};
}

KvPool source_pool(const spec_ctx* ctx, const Model& m, void* base) {
    return KvPool{base, m.kv_elem_bytes, m.kv_dtype, ctx->src_page_table, ctx->src_pages_per_seq, ctx->rt.page_size,
                  ctx->rt.max_batch * ctx->src_pages_per_seq};
}

// One forward pass of `m` over batch * m_rows rows (rows of sequence b are rows
// b*m_rows .. of ctx->row_*); K,V rows of active rows are appended to the cache.
// If n_logit_rows > 0 the final norm and LM head run on rows logit_src[i] and
// write logits rows logit_dst[i] (all rows in order if both are null).
int forward(spec_ctx* ctx, const Model& m, int batch, int m_rows, int n_logit_rows, const int32_t* logit_src,
            const int32_t* logit_dst, float* logits) {
    const spec_model_cfg& c = m.cfg;
    const int n_rows = batch * m_rows;
    const RowMeta rows{ctx->row_token, ctx->row_pos, ctx->row_seq};
    if (c.arch == SPEC_ARCH_BIGRAM)  // logits = table[last token]: one gather
        return n_logit_rows > 0 ? launch_table_logits(m.tok_emb, m.bf16(), c.vocab, rows.token, logit_src, logit_dst, n_logit_rows,
                                                       logits, ctx->stream)
                                : SPEC_OK;
    if (c.arch == SPEC_ARCH_COPY)  // one-hot at the token that followed the same suffix before: one search
        return n_logit_rows > 0 ? launch_copy_logits(ctx->tokens, ctx->rt.max_len, ctx->length, ctx->draft_tokens,
                                                      std::max(ctx->iteration_gamma, 1), rows, logit_src, logit_dst,
                                                      n_logit_rows, c.ngram, c.vocab, logits, ctx->stream)
                                : SPEC_OK;
    const int which = &m == &ctx->model[1] ? 1 : 0;
    if (ctx->rt.pass_kernel && pass_kernel_serves(ctx->pass, m, which, n_rows, n_logit_rows)) {
        // a few rows: the whole pass is one persistent kernel
        const PassTables tables{ctx->page_table, ctx->pages_per_seq, ctx->rt.page_size, ctx->src_page_table,
                                ctx->src_pages_per_seq, ctx->src_len, ctx->rt.max_len, ctx->rt.max_len - 1};
        return launch_pass(ctx->pass, m, which, rows, tables, batch, m_rows, n_logit_rows, logit_src, logit_dst, logits, ctx->stream,
                           ctx->pass_trace, ctx->pass_trace_capacity);
    }
    Pass pass{ctx, m, n_rows, m.bf16(), ctx->stream};
    const int d = c.d_model;
    const float* bias = m.t5() ? m.dec_bias : nullptr;

    SPEC_TRY(launch_embed(m, rows, n_rows, ctx->h, ctx->stream));
    for (int l = 0; l < c.n_layers; ++l) {
        const spec_layer_weights& w = m.layers[l];
        const spec_layer_weights& pw = pass.tc ? m.packed[l] : w;
        SPEC_TRY(pass.self_attention(w, pw, rows, batch, m_rows, layer_pool(ctx, m, l), nullptr, bias, ctx->rt.max_len,
                                     ctx->rt.max_len - 1, ctx->rt.max_len));
        if (m.t5()) {  // cross-attention over the source's K,V (every row sees every source position)
            SPEC_TRY(pass.norm(w.lnx, nullptr, n_rows));
            SPEC_TRY(pass.proj(w.wq_x, pw.wq_x, m.q_dim(), d, ctx->a, ctx->qkv));
            if (pass.tc)  // the partial sums become the query rows
                SPEC_TRY(launch_qkv(c.n_heads, 0, c.d_head, nullptr, KvPool{}, rows, n_rows, ctx->qkv, ctx->partials,
                                    pass.last_splits, ctx->stream));
            const KvPool pool = source_pool(ctx, m, static_cast<char*>(m.cross_kv) + static_cast<size_t>(l) * m.cross_stride);
            const int slices = attention_slices(m, batch, m_rows, ctx->rt.max_src_len);
            const AttnSource src{ctx->qkv, m.q_dim(), pool, ctx->src_len, nullptr, 0, 0};
            SPEC_TRY(launch_attention(m, src, rows, batch, m_rows, slices, ctx->rt.max_src_len, ctx->attn_part, pass.tc ? nullptr : ctx->att,
                                      pass.tc ? pass.hi() : nullptr, pass.tc ? pass.lo() : nullptr, ctx->stream));
            SPEC_TRY(pass.residual(w.wo_x, pw.wo_x, m.q_dim(), ctx->att));
        }
        SPEC_TRY(pass.ffn(w, pw));
    }
    if (n_logit_rows > 0) {
        SPEC_TRY(pass.norm(m.ln_f, logit_src, n_logit_rows));
        if (pass.tc)
            SPEC_TRY(launch_gemm_tc(pass.hi(), pass.lo(), ctx->hi_rows, m.packed_head, true, nullptr, logit_dst, n_logit_rows,
                                    c.vocab, d, ctx->partials, logits, ctx->stream));
        else
            SPEC_TRY(launch_gemm_rows(ctx->a, m.head, m.bf16(), nullptr, logit_dst, n_logit_rows, c.vocab, d, logits, ctx->stream));
    }
    return SPEC_OK;
}

// The encoder of `m` over batch * m_rows source rows described by ctx->row_*
// (inactive rows pad short sources), then the cross-attention K,V of every
// decoder block from its output.
int encode(spec_ctx* ctx, const Model& m, int batch, int m_rows) {
    const spec_model_cfg& c = m.cfg;
    const int n_rows = batch * m_rows;
    const RowMeta rows{ctx->row_token, ctx->row_pos, ctx->row_seq};
    Pass pass{ctx, m, n_rows, m.bf16(), ctx->stream};
    const int S = ctx->rt.max_src_len;
    SPEC_TRY(launch_embed(m, rows, n_rows, ctx->h, ctx->stream));
    for (int l = 0; l < c.n_enc_layers; ++l) {
        const spec_layer_weights& w = m.enc_layers[l];
        const spec_layer_weights& pw = pass.tc ? m.enc_packed[l] : w;
        SPEC_TRY(pass.self_attention(w, pw, rows, batch, m_rows, source_pool(ctx, m, m.enc_kv), ctx->src_len, m.enc_bias,
                                     2 * S - 1, S - 1, S));
        SPEC_TRY(pass.ffn(w, pw));
    }
    SPEC_TRY(pass.norm(m.enc_ln_f, nullptr, n_rows));  // the encoder output, input of every Wkv_x
    for (int l = 0; l < c.n_layers; ++l) {
        const spec_layer_weights& w = m.layers[l];
        const spec_layer_weights& pw = pass.tc ? m.packed[l] : w;
        SPEC_TRY(pass.proj(w.wkv_x, pw.wkv_x, 2 * m.kv_dim(), c.d_model, ctx->a, ctx->qkv));
        const KvPool pool = source_pool(ctx, m, static_cast<char*>(m.cross_kv) + static_cast<size_t>(l) * m.cross_stride);
        SPEC_TRY(launch_qkv(0, c.n_kv_heads, c.d_head, nullptr, pool, rows, n_rows, ctx->qkv, pass.partials(),
                            pass.last_splits, ctx->stream));
    }
    return SPEC_OK;
}

// ---- generation-loop kernels (one thread per sequence; tiny) ----------------

// Uniforms of one iteration (the paper leaves the consumption of randomness
// open; here every draw is keyed by the position it decides):
//   draft_u[b, i]  draw of x_{i+1} at position L+i           (purpose 0)
//   accept_u[b, i] accept test of x_{i+1} at position L+i     (purpose 1)
//   final_u[b, n]  final draw t at position L+n, n = 0..gamma (purpose 2)
__global__ void iteration_uniforms_kernel(const spec_ctx::Params* __restrict__ params,
                                          const int32_t* __restrict__ length, int batch, int gamma,
                                          float* __restrict__ draft_u, float* __restrict__ accept_u,
                                          float* __restrict__ final_u) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch * (gamma + 1)) return;
    const int b = i / (gamma + 1), j = i % (gamma + 1);
    const uint32_t pos = static_cast<uint32_t>(length[b] + j);
    const unsigned long long seed = params->seed;
    final_u[i] = method_uniform(seed, pos, b, kPurposeFinal);
    accept_u[i] = method_uniform(seed, pos, b, kPurposeAccept);  // entry j = gamma is unused
    if (j < gamma) draft_u[b * gamma + j] = method_uniform(seed, pos, b, kPurposeDraft);
}

// First draft step of an iteration: two rows per sequence, positions L-2 and
// L-1.  Position L-2 is already cached unless the previous iteration accepted
// every guess (x_gamma was never fed to the draft); feeding it again rewrites
// the same K,V row, so the shape of the step never changes.
__global__ void prep_draft_first_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ length,
                                        int batch, int gamma, int max_len, int32_t* row_token, int32_t* row_pos,
                                        int32_t* row_seq, int32_t* logit_src, int32_t* logit_dst) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int L = length[b];
    const int p0 = max(L - 2, 0), p1 = L - 1;
    row_token[2 * b] = tokens[static_cast<size_t>(b) * max_len + p0];
    row_token[2 * b + 1] = tokens[static_cast<size_t>(b) * max_len + p1];
    row_pos[2 * b] = p0;
    row_pos[2 * b + 1] = p1;
    row_seq[2 * b] = row_seq[2 * b + 1] = b;
    logit_src[b] = 2 * b + 1;
    logit_dst[b] = b * gamma;  // q_1
}

// Draft step i (2..gamma): one row per sequence, the previous guess x_{i-1} at position L+i-2.
__global__ void prep_draft_step_kernel(const int32_t* __restrict__ draft_tokens, const int32_t* __restrict__ length,
                                       int batch, int gamma, int step, int32_t* row_token, int32_t* row_pos,
                                       int32_t* row_seq, int32_t* logit_src, int32_t* logit_dst) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    row_token[b] = draft_tokens[b * gamma + step - 2];
    row_pos[b] = length[b] + step - 2;
    row_seq[b] = b;
    logit_src[b] = b;
    logit_dst[b] = b * gamma + step - 1;
}

// The target's parallel pass: rows [last committed token, x_1..x_gamma] at positions L-1..L-1+gamma.
__global__ void prep_verify_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ draft_tokens,
                                   const int32_t* __restrict__ length, int batch, int gamma, int max_len,
                                   int32_t* row_token, int32_t* row_pos, int32_t* row_seq) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch * (gamma + 1)) return;
    const int b = i / (gamma + 1), j = i % (gamma + 1);
    const int L = length[b];
    row_token[i] = j == 0 ? tokens[static_cast<size_t>(b) * max_len + L - 1] : draft_tokens[b * gamma + j - 1];
    row_pos[i] = L - 1 + j;
    row_seq[i] = b;
}

// Commit x_1..x_n and t, advance L.  Rolling the caches back needs no data
// movement: both caches are valid up to position L_new - 2 by construction and
// whatever lies beyond is overwritten by the next iteration.  A sequence that
// already has its n_new tokens is frozen.
__global__ void commit_kernel(const spec_ctx::Params* __restrict__ params, const int32_t* __restrict__ draft_tokens,
                              const int32_t* __restrict__ n_accepted, const int32_t* __restrict__ next_token,
                              const float* __restrict__ accept_u, const int32_t* __restrict__ prompt_len, int batch,
                              int gamma, int max_len, int32_t* tokens, int32_t* length, unsigned long long* counters) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int L = length[b];
    if (L - prompt_len[b] >= params->n_new) return;
    int n = n_accepted[b];
    const float imposed = params->imposed_alpha;
    if (imposed >= 0.0f) {  // timing instrument: accept x_i iff r_i < alpha, whatever p and q say
        n = 0;
        while (n < gamma && accept_u[b * (gamma + 1) + n] < imposed) ++n;
    }
    int32_t* seq_tokens = tokens + static_cast<size_t>(b) * max_len;
    for (int i = 0; i < n; ++i) seq_tokens[L + i] = draft_tokens[b * gamma + i];
    seq_tokens[L + n] = next_token[b];
    length[b] = L + n + 1;
    atomicAdd(&counters[0], 1ull);
    atomicAdd(&counters[1], static_cast<unsigned long long>(n + 1));
    atomicAdd(&counters[2], static_cast<unsigned long long>(min(n + 1, gamma)));
    atomicAdd(&counters[3], static_cast<unsigned long long>(n));
    atomicAdd(&counters[4 + n], 1ull);  // how often an iteration accepted n guesses (Eq. 1's capped geometric law)
}

// Enqueues one iteration of Algorithm 1 for the whole batch on ctx->stream.
int enqueue_iteration(spec_ctx* ctx, int batch, int gamma, float temperature) {
    cudaStream_t st = ctx->stream;
    ctx->iteration_gamma = gamma;
    const int vocab = ctx->model[0].cfg.vocab;
    const int threads = 128;
    const int blocks_b = (batch + threads - 1) / threads;
    const int blocks_bg = (batch * (gamma + 1) + threads - 1) / threads;
    SPEC_TRY(launch_pdl(iteration_uniforms_kernel, dim3(blocks_bg), dim3(threads), 0, st, ctx->params, ctx->length,
                        batch, gamma, ctx->draft_u, ctx->accept_u, ctx->final_u));
    for (int step = 1; step <= gamma; ++step) {
        int rows;
        if (step == 1) {
            SPEC_TRY(launch_pdl(prep_draft_first_kernel, dim3(blocks_b), dim3(threads), 0, st, ctx->tokens, ctx->length,
                                batch, gamma, ctx->rt.max_len, ctx->row_token, ctx->row_pos, ctx->row_seq,
                                ctx->logit_src, ctx->logit_dst));
            rows = 2 * batch;
        } else {
            SPEC_TRY(launch_pdl(prep_draft_step_kernel, dim3(blocks_b), dim3(threads), 0, st, ctx->draft_tokens,
                                ctx->length, batch, gamma, step, ctx->row_token, ctx->row_pos, ctx->row_seq,
                                ctx->logit_src, ctx->logit_dst));
            rows = batch;
        }
        SPEC_TRY(forward(ctx, ctx->model[1], batch, rows / batch, batch, ctx->logit_src, ctx->logit_dst, ctx->draft_logits));
        // x_step ~ q_step for every sequence
        SPEC_TRY(launch_sample_strided(ctx->draft_logits + static_cast<size_t>(step - 1) * vocab,
                                       static_cast<size_t>(gamma) * vocab, ctx->draft_u + (step - 1), gamma, batch,
                                       vocab, temperature, ctx->top_k, ctx->top_p, ctx->sample_floors,
                                       ctx->draft_tokens + (step - 1), gamma, st, ctx->nonfinite));
    }
    SPEC_TRY(launch_pdl(prep_verify_kernel, dim3(blocks_bg), dim3(threads), 0, st, ctx->tokens, ctx->draft_tokens,
                        ctx->length, batch, gamma, ctx->rt.max_len, ctx->row_token, ctx->row_pos, ctx->row_seq));
    SPEC_TRY(forward(ctx, ctx->model[0], batch, gamma + 1, batch * (gamma + 1), nullptr, nullptr, ctx->target_logits));
    SPEC_TRY(launch_verify_sample(ctx->target_logits, ctx->draft_logits, ctx->draft_tokens, ctx->accept_u, ctx->final_u,
                                  batch, gamma, vocab, temperature, ctx->lenience, ctx->top_k, ctx->top_p, ctx->n_accepted,
                                  ctx->next_token, ctx->sampler_ws, st, ctx->nonfinite));
    return launch_pdl(commit_kernel, dim3(blocks_b), dim3(threads), 0, st, ctx->params, ctx->draft_tokens,
                      ctx->n_accepted, ctx->next_token, ctx->accept_u, ctx->prompt_len, batch, gamma, ctx->rt.max_len,
                      ctx->tokens, ctx->length, ctx->counters);
}

void drop_graphs(spec_ctx* ctx) {
    for (cudaGraphExec_t g : ctx->graphs)
        if (g) cudaGraphExecDestroy(g);
    ctx->graphs.assign(ctx->graphs.size(), nullptr);
    ctx->graph = nullptr;
}

// Makes ctx->graph the iteration graph for (batch, gamma) under the current
// sampling settings.  Graphs of other gammas captured under the same settings
// are kept, so that a generation can move between gammas without re-capturing.
int build_graph(spec_ctx* ctx, int batch, int gamma, float temperature) {
    if (ctx->graphs.size() < static_cast<size_t>(ctx->rt.max_gamma) + 1) ctx->graphs.resize(ctx->rt.max_gamma + 1, nullptr);
    const bool same_settings = ctx->graph_batch == batch && ctx->graph_temperature == temperature &&
                               ctx->graph_lenience == ctx->lenience && ctx->graph_top_k == ctx->top_k &&
                               ctx->graph_top_p == ctx->top_p;
    if (!same_settings) drop_graphs(ctx);
    if (!ctx->graphs[gamma]) {
        SPEC_CUDA_TRY(cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
        const int status = enqueue_iteration(ctx, batch, gamma, temperature);
        cudaGraph_t g = nullptr;
        const cudaError_t err = cudaStreamEndCapture(ctx->stream, &g);
        if (status != SPEC_OK) {
            if (g) cudaGraphDestroy(g);
            return status;
        }
        SPEC_CUDA_TRY(err);
        const cudaError_t ierr = cudaGraphInstantiate(&ctx->graphs[gamma], g, 0);
        cudaGraphDestroy(g);
        if (ierr != cudaSuccess) ctx->graphs[gamma] = nullptr;
        SPEC_CUDA_TRY(ierr);
    }
    ctx->graph = ctx->graphs[gamma];
    ctx->graph_batch = batch;
    ctx->graph_gamma = gamma;
    ctx->graph_temperature = temperature;
    ctx->graph_lenience = ctx->lenience;
    ctx->graph_top_k = ctx->top_k;
    ctx->graph_top_p = ctx->top_p;
    return SPEC_OK;
}

// Feeds, for every sequence, positions [from[b], to[b]) of host tokens through
// model `which` in chunks (no logits): the prompt pass.
int feed_host_tokens(spec_ctx* ctx, int which, const int32_t* tokens, int stride, const std::vector<int>& from,
                     const std::vector<int>& to, int batch) {
    const int chunk = std::max(1, ctx->max_rows / batch);
    int longest = 0;
    for (int b = 0; b < batch; ++b) longest = std::max(longest, to[b] - from[b]);
    std::vector<int32_t> tok(static_cast<size_t>(batch) * chunk), pos(tok.size()), seq(tok.size());
    for (int c0 = 0; c0 < longest; c0 += chunk) {
        for (int b = 0; b < batch; ++b)
            for (int j = 0; j < chunk; ++j) {
                const int p = from[b] + c0 + j;
                const size_t r = static_cast<size_t>(b) * chunk + j;
                const bool active = p < to[b];
                tok[r] = active ? tokens[static_cast<size_t>(b) * stride + p] : 0;
                pos[r] = active ? p : -1;
                seq[r] = b;
            }
        const size_t bytes = tok.size() * sizeof(int32_t);
        SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_token, tok.data(), bytes, cudaMemcpyHostToDevice, ctx->stream));
        SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_pos, pos.data(), bytes, cudaMemcpyHostToDevice, ctx->stream));
        SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_seq, seq.data(), bytes, cudaMemcpyHostToDevice, ctx->stream));
        SPEC_TRY(forward(ctx, ctx->model[which], batch, chunk, 0, nullptr, nullptr, nullptr));
        SPEC_CUDA_TRY(cudaStreamSynchronize(ctx->stream));  // the host vectors are reused
    }
    return SPEC_OK;
}

// Tile-major copies of every matrix the tensor-core GEMM streams.
int pack_model(spec_ctx* ctx, Model& m) {
    const spec_model_cfg& c = m.cfg;
    auto pack = [&](const void* w, int n_out, int k, const void** out) -> int {
        __nv_bfloat16* dst = nullptr;
        SPEC_TRY(dev_alloc(ctx, &dst, packed_weight_elems(n_out, k)));
        SPEC_TRY(launch_pack_weight(w, n_out, k, dst, ctx->stream));
        *out = dst;
        return SPEC_OK;
    };
    auto pack_block = [&](const spec_layer_weights& w, spec_layer_weights& out) -> int {
        SPEC_TRY(pack(w.wqkv, m.qkv_dim(), c.d_model, &out.wqkv));
        SPEC_TRY(pack(w.wo, c.d_model, m.q_dim(), &out.wo));
        SPEC_TRY(pack(w.w_in, m.ffn_in_dim(), c.d_model, &out.w_in));
        SPEC_TRY(pack(w.w_out, c.d_model, c.d_ff, &out.w_out));
        return SPEC_OK;
    };
    m.packed.assign(c.n_layers, spec_layer_weights{});
    for (int l = 0; l < c.n_layers; ++l) {
        SPEC_TRY(pack_block(m.layers[l], m.packed[l]));
        if (m.t5()) {
            SPEC_TRY(pack(m.layers[l].wq_x, m.q_dim(), c.d_model, &m.packed[l].wq_x));
            SPEC_TRY(pack(m.layers[l].wkv_x, 2 * m.kv_dim(), c.d_model, &m.packed[l].wkv_x));
            SPEC_TRY(pack(m.layers[l].wo_x, c.d_model, m.q_dim(), &m.packed[l].wo_x));
        }
    }
    m.enc_packed.assign(m.enc_layers.size(), spec_layer_weights{});
    for (size_t l = 0; l < m.enc_layers.size(); ++l) SPEC_TRY(pack_block(m.enc_layers[l], m.enc_packed[l]));
    SPEC_TRY(pack(m.head, c.vocab, c.d_model, &m.packed_head));
    SPEC_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    return SPEC_OK;
}

int init_model(spec_ctx* ctx, int which, const spec_model_cfg& cfg, const spec_weights& w) {
    Model& m = ctx->model[which];
    m.cfg = cfg;
    if (cfg.arch == SPEC_ARCH_BIGRAM || cfg.arch == SPEC_ARCH_COPY) {
        // a table or a search: no blocks, no cache; the sizes below only keep the buffer arithmetic valid
        if (which != 1) return fail(SPEC_ERR_BAD_CONFIG, "spec_init: a table or copy model can only be the draft");
        if (cfg.arch == SPEC_ARCH_BIGRAM && !w.tok_emb) return fail(SPEC_ERR_BAD_ARG, "spec_init: missing table pointer");
        m.tok_emb = w.tok_emb;
        m.cfg.dtype = cfg.arch == SPEC_ARCH_COPY ? SPEC_DTYPE_FP32 : cfg.dtype;
        m.cfg.n_layers = 0;
        m.cfg.d_model = m.cfg.d_ff = 8;
        m.cfg.n_heads = m.cfg.n_kv_heads = 1;
        m.cfg.d_head = 64;
        m.cfg.ffn = SPEC_FFN_GELU;
        m.cfg.max_positions = 1 << 30;
        m.cfg.tied_embeddings = 1;
        return SPEC_OK;
    }
    if (!w.tok_emb || !w.ln_f || !w.layers || (cfg.arch == SPEC_ARCH_GPT && !w.pos_emb) || (!cfg.tied_embeddings && !w.head))
        return fail(SPEC_ERR_BAD_ARG, "spec_init: missing weight pointer");
    m.tok_emb = w.tok_emb;
    m.pos_emb = w.pos_emb;
    m.ln_f = w.ln_f;
    m.head = cfg.tied_embeddings ? w.tok_emb : w.head;
    m.layers.assign(w.layers, w.layers + cfg.n_layers);
    for (const spec_layer_weights& l : m.layers)
        if (!l.ln1 || !l.wqkv || !l.wo || !l.ln2 || !l.w_in || !l.w_out)
            return fail(SPEC_ERR_BAD_ARG, "spec_init: missing layer weight pointer");
    if (m.t5()) {
        if (!w.enc_layers || !w.enc_ln_f || !w.enc_rel_bias || !w.rel_bias)
            return fail(SPEC_ERR_BAD_ARG, "spec_init: missing encoder weight pointer");
        m.enc_layers.assign(w.enc_layers, w.enc_layers + cfg.n_enc_layers);
        m.enc_ln_f = w.enc_ln_f;
        for (const spec_layer_weights& l : m.enc_layers)
            if (!l.ln1 || !l.wqkv || !l.wo || !l.ln2 || !l.w_in || !l.w_out)
                return fail(SPEC_ERR_BAD_ARG, "spec_init: missing encoder layer weight pointer");
        for (const spec_layer_weights& l : m.layers)
            if (!l.lnx || !l.wq_x || !l.wkv_x || !l.wo_x)
                return fail(SPEC_ERR_BAD_ARG, "spec_init: missing cross-attention weight pointer");
    }
    m.kv_dtype = ctx->rt.kv_dtype;
    m.kv_elem_bytes = ctx->rt.kv_dtype == SPEC_DTYPE_FP32 ? 4 : 2;
    const size_t n_pages = static_cast<size_t>(ctx->rt.max_batch) * ctx->pages_per_seq;
    m.layer_stride = n_pages * 2 * cfg.n_kv_heads * ctx->rt.page_size * cfg.d_head * m.kv_elem_bytes;
    char* kv = nullptr;
    SPEC_TRY(dev_alloc(ctx, &kv, m.layer_stride * cfg.n_layers));
    // (rows that no sequence has written yet are read, and masked, by the attention kernels that fetch whole tiles:
    // they must hold numbers, not whatever the allocation held)
    SPEC_CUDA_TRY(cudaMemset(kv, 0, m.layer_stride * cfg.n_layers));
    m.kv = kv;
    if (cfg.arch == SPEC_ARCH_LLAMA) {
        std::vector<float2> table;
        fill_rope_table(table, std::min(ctx->rt.max_len, cfg.max_positions), cfg.d_head, cfg.rope_base);
        float2* dev = nullptr;
        SPEC_TRY(dev_alloc(ctx, &dev, table.size()));
        SPEC_CUDA_TRY(cudaMemcpy(dev, table.data(), table.size() * sizeof(float2), cudaMemcpyHostToDevice));
        m.rope_table = dev;
    }
    if (m.t5()) {
        // pools of the source positions: the encoder block in flight and every decoder block's cross K,V
        const size_t src_pages = static_cast<size_t>(ctx->rt.max_batch) * ctx->src_pages_per_seq;
        m.cross_stride = src_pages * 2 * cfg.n_kv_heads * ctx->rt.page_size * cfg.d_head * m.kv_elem_bytes;
        char *enc_kv = nullptr, *cross = nullptr;
        SPEC_TRY(dev_alloc(ctx, &enc_kv, m.cross_stride));
        SPEC_TRY(dev_alloc(ctx, &cross, m.cross_stride * cfg.n_layers));
        SPEC_CUDA_TRY(cudaMemset(enc_kv, 0, m.cross_stride));
        SPEC_CUDA_TRY(cudaMemset(cross, 0, m.cross_stride * cfg.n_layers));
        m.enc_kv = enc_kv;
        m.cross_kv = cross;
        // bias tables by relative position, from the bucket tables
        const int H = cfg.n_heads, B = cfg.rel_buckets, S = ctx->rt.max_src_len, L = ctx->rt.max_len;
        std::vector<float> enc_table(static_cast<size_t>(B) * H), dec_table(enc_table.size());
        SPEC_CUDA_TRY(cudaMemcpy(enc_table.data(), w.enc_rel_bias, enc_table.size() * sizeof(float), cudaMemcpyDeviceToHost));
        SPEC_CUDA_TRY(cudaMemcpy(dec_table.data(), w.rel_bias, dec_table.size() * sizeof(float), cudaMemcpyDeviceToHost));
        std::vector<float> enc_bias(static_cast<size_t>(H) * (2 * S - 1)), dec_bias(static_cast<size_t>(H) * L);
        for (int h = 0; h < H; ++h) {
            for (int delta = -(S - 1); delta <= S - 1; ++delta)
                enc_bias[static_cast<size_t>(h) * (2 * S - 1) + delta + S - 1] =
                    enc_table[static_cast<size_t>(spec_rel_bucket(delta, 1, B, cfg.rel_max_distance)) * H + h];
            for (int delta = -(L - 1); delta <= 0; ++delta)
                dec_bias[static_cast<size_t>(h) * L + delta + L - 1] =
                    dec_table[static_cast<size_t>(spec_rel_bucket(delta, 0, B, cfg.rel_max_distance)) * H + h];
        }
        float *enc_dev = nullptr, *dec_dev = nullptr;
        SPEC_TRY(dev_alloc(ctx, &enc_dev, enc_bias.size()));
        SPEC_TRY(dev_alloc(ctx, &dec_dev, dec_bias.size()));
        SPEC_CUDA_TRY(cudaMemcpy(enc_dev, enc_bias.data(), enc_bias.size() * sizeof(float), cudaMemcpyHostToDevice));
        SPEC_CUDA_TRY(cudaMemcpy(dec_dev, dec_bias.data(), dec_bias.size() * sizeof(float), cudaMemcpyHostToDevice));
        m.enc_bias = enc_dev;
        m.dec_bias = dec_dev;
    }
    return SPEC_OK;
}

}  // namespace
}  // namespace spec

using namespace spec;

extern "C" int spec_rel_bucket(int delta, int bidirectional, int n_buckets, int max_distance) {
    if (n_buckets < 4 || n_buckets % 4 || max_distance <= n_buckets / 2) return fail(SPEC_ERR_BAD_ARG, "spec_rel_bucket: bad table shape");
    int n = n_buckets, base = 0, dist;
    if (bidirectional) {
        n /= 2;
        base = delta > 0 ? n : 0;  // keys after the query use the upper half
        dist = std::abs(delta);
    } else {
        dist = std::max(-delta, 0);  // only keys at or before the query matter
    }
    const int exact = n / 2;  // distances below this have a bucket each
    if (dist < exact) return base + dist;
    const double spread = std::log(static_cast<double>(dist) / exact) / std::log(static_cast<double>(max_distance) / exact) * (n - exact);
    return base + std::min(exact + static_cast<int>(std::floor(spread)), n - 1);
}

extern "C" int spec_init(const spec_model_cfg* target_cfg, const spec_model_cfg* draft_cfg,
                         const spec_weights* target_weights, const spec_weights* draft_weights,
                         const spec_runtime_cfg* runtime, spec_ctx** out) {
    if (!target_cfg || !target_weights || !runtime || !out) return fail(SPEC_ERR_BAD_ARG, "spec_init: null pointer");
    if (draft_cfg && !draft_weights) return fail(SPEC_ERR_BAD_ARG, "spec_init: draft config without weights");
    *out = nullptr;
    SPEC_TRY(check_cfg(*target_cfg, "target"));
    if (draft_cfg) {
        SPEC_TRY(check_cfg(*draft_cfg, "draft"));
        if (draft_cfg->vocab != target_cfg->vocab) return fail(SPEC_ERR_BAD_CONFIG, "spec_init: vocabularies differ");
        if (draft_cfg->arch != SPEC_ARCH_BIGRAM && draft_cfg->arch != SPEC_ARCH_COPY &&
            (draft_cfg->arch == SPEC_ARCH_T5) != (target_cfg->arch == SPEC_ARCH_T5))
            return fail(SPEC_ERR_BAD_CONFIG, "spec_init: an encoder-decoder target needs an encoder-decoder draft and vice versa");
    }
    const bool t5 = target_cfg->arch == SPEC_ARCH_T5;
    if (t5 && (runtime->max_src_len < 1 || runtime->max_src_len > (1 << 16) ||
               static_cast<long long>(runtime->max_src_len) * runtime->max_batch > (1 << 20)))
        return fail(SPEC_ERR_BAD_CONFIG, "spec_init: max_src_len %d out of range for an encoder-decoder context", runtime->max_src_len);
    const spec_runtime_cfg& rt = *runtime;
    if (rt.max_batch < 1 || rt.max_batch > 4096 || rt.max_len < 2 || rt.max_gamma < 0 || rt.max_gamma > 64 ||
        rt.page_size < 32 || rt.page_size > 256 || (rt.page_size & (rt.page_size - 1)) ||
        (rt.kv_dtype != SPEC_DTYPE_FP32 && rt.kv_dtype != SPEC_DTYPE_BF16 && rt.kv_dtype != SPEC_DTYPE_FP16) || (rt.pass_kernel != 0 && rt.pass_kernel != 1))
        return fail(SPEC_ERR_BAD_CONFIG, "spec_init: runtime config out of range");
    int device_count = 0;
    if (cudaGetDeviceCount(&device_count) != cudaSuccess || device_count == 0) {
        cudaGetLastError();
        return fail(SPEC_ERR_CUDA, "spec_init: no CUDA device (this library has no CPU path)");
    }
    spec_ctx* ctx = new (std::nothrow) spec_ctx();
    if (!ctx) return fail(SPEC_ERR_OOM, "spec_init: host allocation failed");
    ctx->rt = rt;
    ctx->has_draft = draft_cfg != nullptr;
    ctx->pages_per_seq = (rt.max_len + rt.page_size - 1) / rt.page_size;
    ctx->max_logit_rows = std::max(rt.max_batch * std::max(rt.max_gamma + 1, 2), 64);
    // The prompt pass takes up to 256 rows at a time (weights streamed once per chunk).
    ctx->max_rows = std::max(ctx->max_logit_rows, std::min(256, rt.max_batch * rt.max_len));
    if (t5) {  // an encoder pass takes every source row of the batch at once
        ctx->src_pages_per_seq = (rt.max_src_len + rt.page_size - 1) / rt.page_size;
        ctx->max_rows = std::max(ctx->max_rows, rt.max_batch * rt.max_src_len);
    }
    auto cleanup = [&](int status) {
        spec_free(ctx);
        return status;
    };
    cudaError_t err = cudaStreamCreateWithFlags(&ctx->stream, cudaStreamNonBlocking);
    if (err != cudaSuccess) return cleanup(fail(SPEC_ERR_CUDA, "cudaStreamCreate: %s", cudaGetErrorString(err)));
    for (auto& e : ctx->ev)
        if (cudaEventCreate(&e) != cudaSuccess) return cleanup(fail(SPEC_ERR_CUDA, "cudaEventCreate failed"));

    int status = init_model(ctx, 0, *target_cfg, *target_weights);
    if (status == SPEC_OK && draft_cfg) status = init_model(ctx, 1, *draft_cfg, *draft_weights);
    if (status != SPEC_OK) return cleanup(status);

    size_t d = 0, qkv = 0, att = 0, fin = 0, ff = 0;
    for (int i = 0; i < (ctx->has_draft ? 2 : 1); ++i) {
        const Model& m = ctx->model[i];
        d = std::max<size_t>(d, m.cfg.d_model);
        qkv = std::max<size_t>(qkv, m.qkv_dim());
        att = std::max<size_t>(att, m.q_dim());
        fin = std::max<size_t>(fin, m.ffn_in_dim());
        ff = std::max<size_t>(ff, m.cfg.d_ff);
    }
    const size_t R = ctx->max_rows, B = rt.max_batch, G = rt.max_gamma, V = target_cfg->vocab;
    const size_t RL = ctx->max_logit_rows;
#define SPEC_ALLOC(ptr, count) \
    if ((status = dev_alloc(ctx, &ctx->ptr, (count))) != SPEC_OK) return cleanup(status)
    SPEC_ALLOC(h, R * d);
    SPEC_ALLOC(a, R * d);
    SPEC_ALLOC(qkv, R * std::max(qkv, 2 * att));
    SPEC_ALLOC(att, R * att);
    SPEC_ALLOC(u, R * fin);
    SPEC_ALLOC(f, R * ff);
    {
        size_t attn = 0;
        for (int i = 0; i < (ctx->has_draft ? 2 : 1); ++i) {
            const Model& m = ctx->model[i];
            for (int b = 1; b <= rt.max_batch; ++b)
                for (int mr = 1; b * mr <= ctx->max_rows; ++mr)
                    for (int keys : {rt.max_len, rt.max_src_len})
                        if (keys > 0)
                            attn = std::max(attn, attention_partial_elems(b * mr, m.cfg.n_heads, m.cfg.d_head,
                                                                          attention_slices(m, b, mr, keys)));
        }
        SPEC_ALLOC(attn_part, attn);
    }
    SPEC_ALLOC(target_logits, RL * V);
    SPEC_ALLOC(draft_logits, std::max<size_t>(B * G, 1) * V);
    {
        // Tensor-core path (any bf16 model): inputs as two bf16 terms, split-K partial sums.
        size_t max_k = 0, partial = 0;
        bool any_bf16 = false;
        for (int i = 0; i < (ctx->has_draft ? 2 : 1); ++i) {
            const Model& m = ctx->model[i];
            if (!m.bf16() || m.cfg.arch == SPEC_ARCH_BIGRAM || m.cfg.arch == SPEC_ARCH_COPY) continue;
            any_bf16 = true;
            max_k = std::max<size_t>({max_k, static_cast<size_t>(m.cfg.d_model), static_cast<size_t>(m.q_dim()), static_cast<size_t>(m.cfg.d_ff)});
            const int shapes[7][2] = {{m.qkv_dim(), m.cfg.d_model}, {m.cfg.d_model, m.q_dim()}, {m.ffn_in_dim(), m.cfg.d_model},
                                      {m.cfg.d_model, m.cfg.d_ff}, {m.q_dim(), m.cfg.d_model}, {2 * m.kv_dim(), m.cfg.d_model},
                                      {m.cfg.vocab, m.cfg.d_model}};
            for (int s = 0; s < 7; ++s) {
                if (!m.t5() && (s == 4 || s == 5)) continue;  // cross-attention projections
                const int most = s == 6 ? ctx->max_logit_rows : ctx->max_rows;  // the head only sees decode rows
                for (int rows = 1; rows <= most; ++rows)
                    partial = std::max(partial, gemm_tc_partial_elems(shapes[s][0], shapes[s][1], rows));
            }
        }
        if (any_bf16) {
            for (int i = 0; i < (ctx->has_draft ? 2 : 1); ++i)
                if (ctx->model[i].bf16() && ctx->model[i].cfg.arch != SPEC_ARCH_BIGRAM &&
                    (status = pack_model(ctx, ctx->model[i])) != SPEC_OK)
                    return cleanup(status);
            ctx->hi_rows = (ctx->max_rows + 255) / 256 * 256;  // whole token tiles of the widest GEMM variant
            SPEC_ALLOC(x_hi, static_cast<size_t>(ctx->hi_rows) * max_k);
            SPEC_ALLOC(x_lo, static_cast<size_t>(ctx->hi_rows) * max_k);
            SPEC_ALLOC(partials, partial);
            cudaMemset(ctx->x_hi, 0, static_cast<size_t>(ctx->hi_rows) * max_k * 2);
            cudaMemset(ctx->x_lo, 0, static_cast<size_t>(ctx->hi_rows) * max_k * 2);
            if (rt.pass_kernel && (status = pass_scratch_init(ctx->pass, ctx->model, ctx->has_draft ? 2 : 1, ctx->allocations)) != SPEC_OK)
                return cleanup(status);
        }
    }
    SPEC_ALLOC(row_token, R);
    SPEC_ALLOC(row_pos, R);
    SPEC_ALLOC(row_seq, R);
    SPEC_ALLOC(logit_src, R);
    SPEC_ALLOC(logit_dst, R);
    SPEC_ALLOC(page_table, B * ctx->pages_per_seq);
    if (t5) {
        SPEC_ALLOC(src_page_table, B * ctx->src_pages_per_seq);
        SPEC_ALLOC(src_len, B);
    }
    SPEC_ALLOC(tokens, B * rt.max_len);
    SPEC_ALLOC(length, B);
    SPEC_ALLOC(prompt_len, B);
    SPEC_ALLOC(draft_tokens, std::max<size_t>(B * G, 1));
    SPEC_ALLOC(n_accepted, B);
    SPEC_ALLOC(next_token, B);
    SPEC_ALLOC(draft_u, std::max<size_t>(B * G, 1));
    SPEC_ALLOC(accept_u, B * (G + 1));
    SPEC_ALLOC(final_u, B * (G + 1));
    SPEC_ALLOC(counters, kCounters);
    SPEC_ALLOC(nonfinite, 1);
    SPEC_ALLOC(params, 1);
    SPEC_ALLOC(sample_floors, B);
    {
        char* ws = nullptr;
        if ((status = dev_alloc(ctx, &ws, verify_sample_workspace_bytes(static_cast<int>(B), static_cast<int>(G), static_cast<int>(V)))) != SPEC_OK)
            return cleanup(status);
        ctx->sampler_ws = ws;
    }
#undef SPEC_ALLOC
    // Page j of sequence b is pool page j * max_batch + b: consecutive pages of a
    // sequence are not adjacent in memory, so every access goes through the table.
    std::vector<int32_t> table(B * ctx->pages_per_seq);
    for (size_t b = 0; b < B; ++b)
        for (int j = 0; j < ctx->pages_per_seq; ++j) table[b * ctx->pages_per_seq + j] = static_cast<int32_t>(j * B + b);
    err = cudaMemcpy(ctx->page_table, table.data(), table.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (err != cudaSuccess) return cleanup(fail(SPEC_ERR_CUDA, "page table upload: %s", cudaGetErrorString(err)));
    if (t5) {
        std::vector<int32_t> src_table(B * ctx->src_pages_per_seq);
        for (size_t b = 0; b < B; ++b)
            for (int j = 0; j < ctx->src_pages_per_seq; ++j) src_table[b * ctx->src_pages_per_seq + j] = static_cast<int32_t>(j * B + b);
        err = cudaMemcpy(ctx->src_page_table, src_table.data(), src_table.size() * sizeof(int32_t), cudaMemcpyHostToDevice);
        if (err != cudaSuccess) return cleanup(fail(SPEC_ERR_CUDA, "source page table upload: %s", cudaGetErrorString(err)));
    }
    ctx->cached[0].assign(B, 0);
    ctx->cached[1].assign(B, 0);
    *out = ctx;
    return SPEC_OK;
}

extern "C" void spec_free(spec_ctx* ctx) {
    if (!ctx) return;
    if (ctx->stream) cudaStreamSynchronize(ctx->stream);
    drop_graphs(ctx);
    pass_scratch_release(ctx->pass);
    for (void* p : ctx->allocations) cudaFree(p);
    for (auto& e : ctx->ev)
        if (e) cudaEventDestroy(e);
    if (ctx->stream) cudaStreamDestroy(ctx->stream);
    delete ctx;
}

namespace {

// Encoder pass of the first n_models models over the sources of `batch` sequences.
int encode_sources(spec_ctx* ctx, const int32_t* source, const int32_t* source_len, int stride, int batch, int n_models) {
    if (!ctx->model[0].t5()) return fail(SPEC_ERR_BAD_CONFIG, "encode: not an encoder-decoder context");
    if (!source || !source_len || stride < 1 || batch < 1) return fail(SPEC_ERR_BAD_ARG, "encode: bad argument");
    if (batch > ctx->rt.max_batch) return fail(SPEC_ERR_CAPACITY, "encode: batch %d exceeds max_batch %d", batch, ctx->rt.max_batch);
    int longest = 0;
    for (int b = 0; b < batch; ++b) {
        if (source_len[b] < 1 || source_len[b] > stride) return fail(SPEC_ERR_BAD_ARG, "encode: source_len[%d]=%d", b, source_len[b]);
        if (source_len[b] > ctx->rt.max_src_len)
            return fail(SPEC_ERR_CAPACITY, "encode: source %d has %d tokens, max_src_len is %d", b, source_len[b], ctx->rt.max_src_len);
        for (int i = 0; i < source_len[b]; ++i) {
            const int32_t t = source[static_cast<size_t>(b) * stride + i];
            if (t < 0 || t >= ctx->model[0].cfg.vocab) return fail(SPEC_ERR_BAD_ARG, "encode: token %d out of range", t);
        }
        longest = std::max(longest, source_len[b]);
    }
    const size_t n = static_cast<size_t>(batch) * longest;
    std::vector<int32_t> tok(n), pos(n), seq(n);
    for (int b = 0; b < batch; ++b)
        for (int j = 0; j < longest; ++j) {
            const bool active = j < source_len[b];
            tok[static_cast<size_t>(b) * longest + j] = active ? source[static_cast<size_t>(b) * stride + j] : 0;
            pos[static_cast<size_t>(b) * longest + j] = active ? j : -1;
            seq[static_cast<size_t>(b) * longest + j] = b;
        }
    cudaStream_t st = ctx->stream;
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_token, tok.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_pos, pos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_seq, seq.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->src_len, source_len, batch * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    for (int which = 0; which < n_models; ++which)
        if (ctx->model[which].t5()) SPEC_TRY(encode(ctx, ctx->model[which], batch, longest));  // (a table draft has no encoder)
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));  // the host vectors go out of scope
    if (const int gave_up = device_gave_up(ctx)) return fail(SPEC_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (code %d)", gave_up);
    ctx->encoded = true;
    ctx->encoded_batch = batch;
    return SPEC_OK;
}

// Validates a generation request, uploads the prompts, runs the prompt pass of
// both models and prepares the iteration graph.
int begin_session(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride, int batch,
                  int n_new, int gamma, float temperature, uint64_t seed) {
    if (!ctx || !prompt || !prompt_len) return fail(SPEC_ERR_BAD_ARG, "generation: null pointer");
    if (batch < 1 || n_new < 1 || gamma < 0 || prompt_stride < 1 || !(temperature >= 0.0f) || !std::isfinite(temperature))
        return fail(SPEC_ERR_BAD_ARG, "generation: batch=%d n_new=%d gamma=%d temperature=%g", batch, n_new, gamma, temperature);
    if (batch > ctx->rt.max_batch || gamma > ctx->rt.max_gamma)
        return fail(SPEC_ERR_CAPACITY, "generation: batch %d / gamma %d exceed the context's limits (%d / %d)", batch, gamma, ctx->rt.max_batch, ctx->rt.max_gamma);
    if (gamma > 0 && !ctx->has_draft) return fail(SPEC_ERR_BAD_CONFIG, "generation: gamma > 0 needs a draft model");
    int limit = std::min(ctx->rt.max_len, ctx->model[0].cfg.max_positions);
    if (gamma > 0) limit = std::min(limit, ctx->model[1].cfg.max_positions);
    // Encoder-decoder: `prompt` is the source; the decoder's own prompt is the start token.
    const bool t5 = ctx->model[0].t5();
    const int32_t *source = prompt, *source_len = prompt_len;
    const int source_stride = prompt_stride;
    std::vector<int32_t> start_tokens(batch, 0), start_len(batch, 1);
    if (t5) {
        prompt = start_tokens.data();
        prompt_len = start_len.data();
        prompt_stride = 1;
    }
    for (int b = 0; b < batch; ++b) {
        if (prompt_len[b] < 1 || prompt_len[b] > prompt_stride) return fail(SPEC_ERR_BAD_ARG, "generation: prompt_len[%d]=%d", b, prompt_len[b]);
        if (prompt_len[b] + n_new + gamma + 1 > limit)
            return fail(SPEC_ERR_CAPACITY, "generation: sequence %d needs %d positions, limit %d", b, prompt_len[b] + n_new + gamma + 1, limit);
        for (int i = 0; i < prompt_len[b]; ++i) {
            const int32_t t = prompt[static_cast<size_t>(b) * prompt_stride + i];
            if (t < 0 || t >= ctx->model[0].cfg.vocab) return fail(SPEC_ERR_BAD_ARG, "generation: token %d out of range", t);
        }
    }
    cudaStream_t st = ctx->stream;
    const int max_len = ctx->rt.max_len;
    ctx->session_batch = 0;

    // upload prompts and state
    std::vector<int32_t> host_tokens(static_cast<size_t>(batch) * max_len, 0);
    for (int b = 0; b < batch; ++b)
        std::memcpy(&host_tokens[static_cast<size_t>(b) * max_len], prompt + static_cast<size_t>(b) * prompt_stride, prompt_len[b] * sizeof(int32_t));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->tokens, host_tokens.data(), host_tokens.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->length, prompt_len, batch * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->prompt_len, prompt_len, batch * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemsetAsync(ctx->counters, 0, kCounters * sizeof(unsigned long long), st));
    SPEC_CUDA_TRY(cudaMemsetAsync(ctx->nonfinite, 0, sizeof(int), st));
    const spec_ctx::Params params{seed, n_new, ctx->imposed_alpha};
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->params, &params, sizeof(params), cudaMemcpyHostToDevice, st));

    // prompt pass: positions 0..prompt_len-2 (the last prompt token is fed by the first iteration)
    SPEC_CUDA_TRY(cudaEventRecord(ctx->ev[0], st));
    if (t5) SPEC_TRY(encode_sources(ctx, source, source_len, source_stride, batch, gamma > 0 ? 2 : 1));
    std::vector<int> from(batch, 0), to(batch);
    for (int b = 0; b < batch; ++b) to[b] = prompt_len[b] - 1;
    SPEC_TRY(feed_host_tokens(ctx, 0, prompt, prompt_stride, from, to, batch));
    if (gamma > 0) SPEC_TRY(feed_host_tokens(ctx, 1, prompt, prompt_stride, from, to, batch));
    SPEC_CUDA_TRY(cudaEventRecord(ctx->ev[1], st));
    SPEC_TRY(build_graph(ctx, batch, gamma, temperature));
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));  // host_tokens goes out of scope
    float pre = 0.0f;
    cudaEventElapsedTime(&pre, ctx->ev[0], ctx->ev[1]);
    ctx->session_prefill_ms = pre;
    ctx->session_batch = batch;
    ctx->session_gamma = gamma;
    ctx->session_gamma_cap = gamma;
    ctx->session_temperature = temperature;
    ctx->session_draft_passes = 0;
    ctx->session_n_new = n_new;
    ctx->session_replays = 0;
    ctx->session_prompt_len.assign(prompt_len, prompt_len + batch);
    // the diagnostics' view of the caches is stale now
    std::fill(ctx->cached[0].begin(), ctx->cached[0].end(), 0);
    std::fill(ctx->cached[1].begin(), ctx->cached[1].end(), 0);
    return SPEC_OK;
}

// Replays the iteration graph `iterations` times; returns the device time and
// the largest number of tokens any sequence still lacks.
int run_iterations(spec_ctx* ctx, int iterations, float* elapsed_ms, int* remaining) {
    cudaStream_t st = ctx->stream;
    const int batch = ctx->session_batch;
    std::vector<int32_t> lengths(batch);
    SPEC_CUDA_TRY(cudaEventRecord(ctx->ev[1], st));
    for (int i = 0; i < iterations; ++i) SPEC_CUDA_TRY(cudaGraphLaunch(ctx->graph, st));
    SPEC_CUDA_TRY(cudaEventRecord(ctx->ev[2], st));
    ctx->session_replays += iterations;
    ctx->session_draft_passes += static_cast<long long>(iterations) * ctx->session_gamma;
    SPEC_CUDA_TRY(cudaMemcpyAsync(lengths.data(), ctx->length, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    int nonfinite = 0;
    SPEC_CUDA_TRY(cudaMemcpyAsync(&nonfinite, ctx->nonfinite, sizeof(int), cudaMemcpyDeviceToHost, st));
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    if (nonfinite) {
        SPEC_CUDA_TRY(cudaMemsetAsync(ctx->nonfinite, 0, sizeof(int), st));
        return fail(SPEC_ERR_NONFINITE, "a model produced a NaN or +inf logit, or a row without a finite logit (the tokens of these "
                                        "iterations are not valid)");
    }
    if (const int gave_up = device_gave_up(ctx)) return fail(SPEC_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (code %d)", gave_up);
    SPEC_CUDA_TRY(cudaEventElapsedTime(elapsed_ms, ctx->ev[1], ctx->ev[2]));
    *remaining = 0;
    for (int b = 0; b < batch; ++b)
        *remaining = std::max(*remaining, ctx->session_n_new - (lengths[b] - ctx->session_prompt_len[b]));
    return SPEC_OK;
}

int fill_stats(spec_ctx* ctx, double decode_ms, spec_stats* stats) {
    unsigned long long counters[kCounters];
    SPEC_CUDA_TRY(cudaMemcpy(counters, ctx->counters, sizeof(counters), cudaMemcpyDeviceToHost));
    for (int n = 0; n <= 64; ++n) stats->accepted_histogram[n] = static_cast<int64_t>(counters[4 + n]);
    stats->iterations = static_cast<int64_t>(counters[0]);
    stats->tokens = static_cast<int64_t>(counters[1]);
    stats->tests_evaluated = static_cast<int64_t>(counters[2]);
    stats->tests_passed = static_cast<int64_t>(counters[3]);
    stats->target_passes = ctx->session_replays;
    stats->draft_passes = ctx->session_draft_passes;
    stats->prefill_ms = ctx->session_prefill_ms;
    stats->decode_ms = decode_ms;
    return SPEC_OK;
}

}  // namespace

extern "C" int spec_generate(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride,
                             int batch, int n_new, int gamma, float temperature, uint64_t seed, int32_t* out_tokens,
                             spec_stats* stats) {
    if (!out_tokens) return fail(SPEC_ERR_BAD_ARG, "spec_generate: null pointer");
    SPEC_TRY(begin_session(ctx, prompt, prompt_len, prompt_stride, batch, n_new, gamma, temperature, seed));
    // decode loop: the iteration graph is replayed in bursts; after each burst the
    // host reads the committed lengths.  A burst is as long as the iterations that
    // are certainly needed (every iteration emits at most gamma + 1 tokens).
    double decode_ms = 0.0;
    int remaining = n_new;
    while (remaining > 0) {
        float ms = 0.0f;
        SPEC_TRY(run_iterations(ctx, (remaining + gamma) / (gamma + 1), &ms, &remaining));
        decode_ms += ms;
    }
    SPEC_TRY(spec_read_tokens(ctx, out_tokens));
    if (stats) SPEC_TRY(fill_stats(ctx, decode_ms, stats));
    return SPEC_OK;
}

extern "C" int spec_begin(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride,
                          int batch, int n_new, int gamma, float temperature, uint64_t seed) {
    return begin_session(ctx, prompt, prompt_len, prompt_stride, batch, n_new, gamma, temperature, seed);
}

extern "C" int spec_step(spec_ctx* ctx, int iterations, int* remaining, spec_stats* stats) {
    if (!ctx || iterations < 1) return fail(SPEC_ERR_BAD_ARG, "spec_step: bad argument");
    if (ctx->session_batch < 1) return fail(SPEC_ERR_BAD_ARG, "spec_step: no generation in progress (call spec_begin)");
    float ms = 0.0f;
    int left = 0;
    SPEC_TRY(run_iterations(ctx, iterations, &ms, &left));
    if (remaining) *remaining = left;
    if (stats) SPEC_TRY(fill_stats(ctx, ms, stats));
    return SPEC_OK;
}

extern "C" int spec_read_tokens(spec_ctx* ctx, int32_t* out_tokens) {
    if (!ctx || !out_tokens) return fail(SPEC_ERR_BAD_ARG, "spec_read_tokens: null pointer");
    if (ctx->session_batch < 1) return fail(SPEC_ERR_BAD_ARG, "spec_read_tokens: no generation in progress");
    const int batch = ctx->session_batch, n_new = ctx->session_n_new, max_len = ctx->rt.max_len;
    std::vector<int32_t> host_tokens(static_cast<size_t>(batch) * max_len);
    SPEC_CUDA_TRY(cudaMemcpyAsync(host_tokens.data(), ctx->tokens, host_tokens.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    SPEC_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    for (int b = 0; b < batch; ++b)
        std::memcpy(out_tokens + static_cast<size_t>(b) * n_new, &host_tokens[static_cast<size_t>(b) * max_len + ctx->session_prompt_len[b]], n_new * sizeof(int32_t));
    return SPEC_OK;
}

extern "C" int spec_set_gamma(spec_ctx* ctx, int gamma) {
    if (!ctx) return fail(SPEC_ERR_BAD_ARG, "spec_set_gamma: null context");
    if (ctx->session_batch < 1) return fail(SPEC_ERR_BAD_ARG, "spec_set_gamma: no generation in progress (call spec_begin)");
    // gamma = 0 iterations do not feed the draft, whose cache would then lag behind the committed tokens
    if (ctx->session_gamma_cap < 1 || gamma < 1 || gamma > ctx->session_gamma_cap)
        return fail(SPEC_ERR_BAD_ARG, "spec_set_gamma: gamma %d outside [1, %d] (the gamma given to spec_begin)", gamma,
                    ctx->session_gamma_cap);
    SPEC_TRY(build_graph(ctx, ctx->session_batch, gamma, ctx->session_temperature));
    ctx->session_gamma = gamma;
    return SPEC_OK;
}

extern "C" int spec_choose_gamma(double alpha, double base_cost, double cost_per_guess, int gamma_max) {
    if (!(alpha >= 0.0) || !(alpha <= 1.0) || !(base_cost > 0.0) || !(cost_per_guess >= 0.0) || gamma_max < 1) return -1;
    int best = 1;
    double best_rate = -1.0;
    for (int g = 1; g <= gamma_max; ++g) {
        // Eq. 1: expected tokens per iteration, 1 + alpha + ... + alpha^g
        double tokens = 0.0, term = 1.0;
        for (int i = 0; i <= g; ++i) {
            tokens += term;
            term *= alpha;
        }
        const double rate = tokens / (base_cost + cost_per_guess * g);
        if (rate > best_rate) {
            best_rate = rate;
            best = g;
        }
    }
    return best;
}

extern "C" int spec_generate_adaptive(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride,
                                      int batch, int n_new, int gamma_max, float temperature, uint64_t seed, int burst,
                                      int32_t* out_tokens, spec_stats* stats, int32_t* trace, int trace_capacity,
                                      int* n_bursts) {
    if (!out_tokens || burst < 1 || gamma_max < 1 || trace_capacity < 0 || (trace_capacity > 0 && !trace))
        return fail(SPEC_ERR_BAD_ARG, "spec_generate_adaptive: bad argument");
    SPEC_TRY(begin_session(ctx, prompt, prompt_len, prompt_stride, batch, n_new, gamma_max, temperature, seed));
    // Iteration time is modelled as base + per_guess * gamma (one target pass and the
    // sampler; one draft pass and one more target row per guess) and fitted to the
    // bursts run so far; alpha is the running estimate of Definition 3.1's E(beta).
    std::vector<double> time_sum(gamma_max + 1, 0.0), iters(gamma_max + 1, 0.0);
    double alpha = 0.5, decode_ms = 0.0;
    double recent_evaluated = 0.0, recent_passed = 0.0;  // counts that fade by kFade per burst
    constexpr double kFade = 0.8;
    long long seen_evaluated = 0, seen_passed = 0;
    int remaining = n_new, bursts = 0;
    while (remaining > 0) {
        int gamma;
        if (bursts == 0) gamma = 1;                            // two calibration bursts span the range
        else if (bursts == 1) gamma = gamma_max;
        else {
            // least squares through the mean iteration time of every gamma tried so far
            double n = 0, sx = 0, sy = 0, sxx = 0, sxy = 0;
            for (int g = 1; g <= gamma_max; ++g)
                if (iters[g] > 0) {
                    const double y = time_sum[g] / iters[g];
                    n += 1; sx += g; sy += y; sxx += double(g) * g; sxy += g * y;
                }
            double per = 0.0, base = sy / n;
            const double det = n * sxx - sx * sx;
            if (det > 0) {
                per = std::max(0.0, (n * sxy - sx * sy) / det);
                base = std::max(1e-9, (sy - per * sx) / n);
            }
            gamma = spec_choose_gamma(alpha, base, per, gamma_max);
        }
        SPEC_TRY(spec_set_gamma(ctx, gamma));
        const int count = std::min(burst, (remaining + gamma) / (gamma + 1));
        float ms = 0.0f;
        SPEC_TRY(run_iterations(ctx, count, &ms, &remaining));
        decode_ms += ms;
        time_sum[gamma] += ms;
        iters[gamma] += count;
        if (2 * bursts + 1 < trace_capacity) {
            trace[2 * bursts] = gamma;
            trace[2 * bursts + 1] = count;
        }
        ++bursts;
        unsigned long long counters[4];
        SPEC_CUDA_TRY(cudaMemcpy(counters, ctx->counters, sizeof(counters), cudaMemcpyDeviceToHost));
        const long long evaluated = static_cast<long long>(counters[2]) - seen_evaluated;
        const long long passed = static_cast<long long>(counters[3]) - seen_passed;
        seen_evaluated += evaluated;
        seen_passed += passed;
        recent_evaluated = kFade * recent_evaluated + static_cast<double>(evaluated);
        recent_passed = kFade * recent_passed + static_cast<double>(passed);
        if (recent_evaluated > 0.0) alpha = recent_passed / recent_evaluated;
    }
    if (n_bursts) *n_bursts = bursts;
    SPEC_TRY(spec_read_tokens(ctx, out_tokens));
    if (stats) SPEC_TRY(fill_stats(ctx, decode_ms, stats));
    return SPEC_OK;
}

extern "C" int spec_set_lenience(spec_ctx* ctx, float lenience) {
    if (!ctx || !(lenience > 0.0f) || !(lenience <= 1.0f)) return fail(SPEC_ERR_BAD_ARG, "spec_set_lenience: lenience must be in (0, 1]");
    ctx->lenience = lenience;
    return SPEC_OK;
}

extern "C" int spec_set_truncation(spec_ctx* ctx, int top_k, float top_p) {
    if (!ctx || top_k < 0 || !(top_p == top_p))
        return fail(SPEC_ERR_BAD_ARG, "spec_set_truncation: top_k must be >= 0 (0: off) and top_p a number (>= 1: off)");
    ctx->top_k = top_k;
    ctx->top_p = top_p;
    return SPEC_OK;
}

extern "C" int spec_set_imposed_acceptance(spec_ctx* ctx, float alpha) {
    if (!ctx || !(alpha <= 1.0f)) return fail(SPEC_ERR_BAD_ARG, "spec_set_imposed_acceptance: alpha must be <= 1 (negative: off)");
    ctx->imposed_alpha = alpha < 0.0f ? -1.0f : alpha;
    return SPEC_OK;
}

extern "C" int spec_encode(spec_ctx* ctx, const int32_t* source, const int32_t* source_len, int source_stride, int batch) {
    if (!ctx) return fail(SPEC_ERR_BAD_ARG, "spec_encode: null context");
    ctx->session_batch = 0;
    SPEC_TRY(encode_sources(ctx, source, source_len, source_stride, batch, ctx->has_draft ? 2 : 1));
    std::fill(ctx->cached[0].begin(), ctx->cached[0].end(), 0);
    std::fill(ctx->cached[1].begin(), ctx->cached[1].end(), 0);
    return SPEC_OK;
}

extern "C" int spec_reset(spec_ctx* ctx) {
    if (!ctx) return fail(SPEC_ERR_BAD_ARG, "spec_reset: null context");
    std::fill(ctx->cached[0].begin(), ctx->cached[0].end(), 0);
    std::fill(ctx->cached[1].begin(), ctx->cached[1].end(), 0);
    ctx->session_batch = 0;  // the diagnostics reuse the caches
    SPEC_CUDA_TRY(cudaStreamSynchronize(ctx->stream));
    return SPEC_OK;
}

extern "C" int spec_truncate(spec_ctx* ctx, int which, const int32_t* lengths, int batch) {
    if (!ctx || !lengths || which < 0 || which > 1 || batch < 1 || batch > ctx->rt.max_batch)
        return fail(SPEC_ERR_BAD_ARG, "spec_truncate: bad argument");
    for (int b = 0; b < batch; ++b) {
        if (lengths[b] < 0 || lengths[b] > ctx->cached[which][b])
            return fail(SPEC_ERR_BAD_ARG, "spec_truncate: length %d of sequence %d is not within the cached %d", lengths[b], b, ctx->cached[which][b]);
    }
    for (int b = 0; b < batch; ++b) ctx->cached[which][b] = lengths[b];
    return SPEC_OK;
}

extern "C" int spec_attention_plan(spec_ctx* ctx, int which, int batch, int rows, int cross, int* plan) {
    if (!ctx || !plan || which < 0 || which > 1 || batch < 1 || rows < 1)
        return fail(SPEC_ERR_BAD_ARG, "spec_attention_plan: bad argument");
    if (which == 1 && !ctx->has_draft) return fail(SPEC_ERR_BAD_CONFIG, "spec_attention_plan: no draft model");
    const Model& m = ctx->model[which];
    if (m.cfg.arch == SPEC_ARCH_BIGRAM || m.cfg.arch == SPEC_ARCH_COPY)
        return fail(SPEC_ERR_BAD_CONFIG, "spec_attention_plan: a table or copy model has no attention");
    if (cross && !m.t5()) return fail(SPEC_ERR_BAD_CONFIG, "spec_attention_plan: only encoder-decoder models have cross-attention");
    const AttentionPlan p = attention_plan(m, batch, rows, cross ? ctx->rt.max_src_len : ctx->rt.max_len);
    plan[0] = p.tensor_cores;
    plan[1] = p.slices;
    plan[2] = p.cluster_merge;
    plan[3] = p.in_turn;
    return SPEC_OK;
}

extern "C" int spec_pass_trace(spec_ctx* ctx, int which, int batch, int rows, unsigned long long* stamps_ns, int capacity,
                               int* count) {
    if (!ctx || !stamps_ns || !count || capacity < 2 || which < 0 || which > 1 || batch < 1 || rows < 1)
        return fail(SPEC_ERR_BAD_ARG, "spec_pass_trace: bad argument");
    if (which == 1 && !ctx->has_draft) return fail(SPEC_ERR_BAD_CONFIG, "spec_pass_trace: no draft model");
    const Model& m = ctx->model[which];
    const int n = batch * rows;
    if (batch > ctx->rt.max_batch || n > ctx->max_logit_rows)
        return fail(SPEC_ERR_CAPACITY, "spec_pass_trace: %d x %d rows exceed the workspace (%d rows)", batch, rows, ctx->max_logit_rows);
    if (!ctx->rt.pass_kernel || !pass_kernel_serves(ctx->pass, m, which, n, n))
        return fail(SPEC_ERR_BAD_CONFIG, "spec_pass_trace: a pass of %d x %d rows of this model does not run as the persistent kernel", batch, rows);
    ctx->session_batch = 0;
    std::vector<int32_t> tok(n, 0), pos(n), seq(n);
    for (int b = 0; b < batch; ++b) {
        if (ctx->cached[which][b] + rows > std::min(ctx->rt.max_len, m.cfg.max_positions))
            return fail(SPEC_ERR_CAPACITY, "spec_pass_trace: sequence %d would exceed the cache", b);
        for (int j = 0; j < rows; ++j) {
            pos[b * rows + j] = ctx->cached[which][b] + j;
            seq[b * rows + j] = b;
        }
    }
    cudaStream_t st = ctx->stream;
    unsigned long long* dev = nullptr;
    SPEC_CUDA_TRY(cudaMalloc(&dev, static_cast<size_t>(capacity) * sizeof(unsigned long long)));
    cudaError_t err = cudaMemsetAsync(dev, 0, static_cast<size_t>(capacity) * sizeof(unsigned long long), st);
    if (err == cudaSuccess) err = cudaMemcpyAsync(ctx->row_token, tok.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st);
    if (err == cudaSuccess) err = cudaMemcpyAsync(ctx->row_pos, pos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st);
    if (err == cudaSuccess) err = cudaMemcpyAsync(ctx->row_seq, seq.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st);
    int status = SPEC_OK;
    if (err == cudaSuccess) {
        status = forward(ctx, m, batch, rows, n, nullptr, nullptr, ctx->target_logits);  // untimed: warms the caches
        ctx->pass_trace = dev;
        ctx->pass_trace_capacity = capacity;
        if (status == SPEC_OK) status = forward(ctx, m, batch, rows, n, nullptr, nullptr, ctx->target_logits);
        ctx->pass_trace = nullptr;
        ctx->pass_trace_capacity = 0;
    }
    if (err == cudaSuccess) err = cudaMemcpyAsync(stamps_ns, dev, static_cast<size_t>(capacity) * sizeof(unsigned long long), cudaMemcpyDeviceToHost, st);
    if (err == cudaSuccess) err = cudaStreamSynchronize(st);
    cudaFree(dev);
    SPEC_CUDA_TRY(err);
    if (status != SPEC_OK) return status;
    if (const int gave_up = device_gave_up(ctx)) return fail(SPEC_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (code %d)", gave_up);
    int used = 0;
    for (int i = 0; i < capacity; ++i)
        if (stamps_ns[i]) used = i + 1;
    *count = used;
    return SPEC_OK;
}

extern "C" int spec_time_forward(spec_ctx* ctx, int which, int batch, int rows, int repeats, float* ms_per_pass) {
    if (!ctx || !ms_per_pass || which < 0 || which > 1 || batch < 1 || rows < 1 || repeats < 1)
        return fail(SPEC_ERR_BAD_ARG, "spec_time_forward: bad argument");
    if (which == 1 && !ctx->has_draft) return fail(SPEC_ERR_BAD_CONFIG, "spec_time_forward: no draft model");
    if (batch > ctx->rt.max_batch || batch * rows > ctx->max_logit_rows)
        return fail(SPEC_ERR_CAPACITY, "spec_time_forward: %d x %d rows exceed the workspace (%d rows)", batch, rows, ctx->max_logit_rows);
    const Model& m = ctx->model[which];
    if (m.t5() && (!ctx->encoded || batch > ctx->encoded_batch))
        return fail(SPEC_ERR_BAD_ARG, "spec_time_forward: call spec_encode for these sequences first");
    const int n = batch * rows;
    ctx->session_batch = 0;
    std::vector<int32_t> tok(n, 0), pos(n), seq(n);
    for (int b = 0; b < batch; ++b) {
        if (ctx->cached[which][b] + rows > std::min(ctx->rt.max_len, m.cfg.max_positions))
            return fail(SPEC_ERR_CAPACITY, "spec_time_forward: sequence %d would exceed the cache", b);
        for (int j = 0; j < rows; ++j) {
            pos[b * rows + j] = ctx->cached[which][b] + j;
            seq[b * rows + j] = b;
        }
    }
    cudaStream_t st = ctx->stream;
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_token, tok.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_pos, pos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_seq, seq.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    SPEC_CUDA_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    const int status = forward(ctx, m, batch, rows, n, nullptr, nullptr, ctx->target_logits);
    cudaGraph_t g = nullptr;
    const cudaError_t end = cudaStreamEndCapture(st, &g);
    if (status != SPEC_OK) {
        if (g) cudaGraphDestroy(g);
        return status;
    }
    SPEC_CUDA_TRY(end);
    cudaGraphExec_t exec = nullptr;
    const cudaError_t inst = cudaGraphInstantiate(&exec, g, 0);
    cudaGraphDestroy(g);
    SPEC_CUDA_TRY(inst);
    cudaError_t err = cudaGraphLaunch(exec, st);  // untimed: uploads the graph, warms the caches
    if (err == cudaSuccess) err = cudaEventRecord(ctx->ev[1], st);
    for (int i = 0; i < repeats && err == cudaSuccess; ++i) err = cudaGraphLaunch(exec, st);
    if (err == cudaSuccess) err = cudaEventRecord(ctx->ev[2], st);
    if (err == cudaSuccess) err = cudaStreamSynchronize(st);
    cudaGraphExecDestroy(exec);
    SPEC_CUDA_TRY(err);
    if (const int gave_up = device_gave_up(ctx)) return fail(SPEC_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (code %d)", gave_up);
    float ms = 0.0f;
    SPEC_CUDA_TRY(cudaEventElapsedTime(&ms, ctx->ev[1], ctx->ev[2]));
    *ms_per_pass = ms / static_cast<float>(repeats);
    return SPEC_OK;
}

extern "C" int spec_forward_logits(spec_ctx* ctx, int which, const int32_t* tokens, int batch, int rows, float* logits) {
    if (!ctx || !tokens || !logits || which < 0 || which > 1 || batch < 1 || rows < 1)
        return fail(SPEC_ERR_BAD_ARG, "spec_forward_logits: bad argument");
    if (which == 1 && !ctx->has_draft) return fail(SPEC_ERR_BAD_CONFIG, "spec_forward_logits: no draft model");
    if (ctx->model[which].cfg.arch == SPEC_ARCH_COPY)
        return fail(SPEC_ERR_BAD_CONFIG, "spec_forward_logits: a copy model reads the generation's own tokens and has no teacher-forced pass");
    if (batch > ctx->rt.max_batch || batch * rows > ctx->max_logit_rows)
        return fail(SPEC_ERR_CAPACITY, "spec_forward_logits: %d x %d rows exceed the workspace (%d rows)", batch, rows, ctx->max_logit_rows);
    if (ctx->model[which].t5() && (!ctx->encoded || batch > ctx->encoded_batch))
        return fail(SPEC_ERR_BAD_ARG, "spec_forward_logits: call spec_encode for these sequences first");
    const Model& m = ctx->model[which];
    const int n = batch * rows;
    ctx->session_batch = 0;  // the diagnostics reuse the caches
    std::vector<int32_t> tok(n), pos(n), seq(n);
    for (int b = 0; b < batch; ++b) {
        if (ctx->cached[which][b] + rows > std::min(ctx->rt.max_len, m.cfg.max_positions))
            return fail(SPEC_ERR_CAPACITY, "spec_forward_logits: sequence %d would exceed the cache", b);
        for (int j = 0; j < rows; ++j) {
            const int32_t t = tokens[b * rows + j];
            if (t < 0 || t >= m.cfg.vocab) return fail(SPEC_ERR_BAD_ARG, "spec_forward_logits: token %d out of range", t);
            tok[b * rows + j] = t;
            pos[b * rows + j] = ctx->cached[which][b] + j;
            seq[b * rows + j] = b;
        }
    }
    cudaStream_t st = ctx->stream;
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_token, tok.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_pos, pos.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_CUDA_TRY(cudaMemcpyAsync(ctx->row_seq, seq.data(), n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SPEC_TRY(forward(ctx, m, batch, rows, n, nullptr, nullptr, logits));
    SPEC_CUDA_TRY(cudaStreamSynchronize(st));
    if (const int gave_up = device_gave_up(ctx)) return fail(SPEC_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (code %d)", gave_up);
    for (int b = 0; b < batch; ++b) ctx->cached[which][b] += rows;
    return SPEC_OK;
}
