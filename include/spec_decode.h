/*
 * spec_decode.h -- C ABI of the B200 (sm_100a) speculative-decoding library.
 *
 * Method: Leviathan, Kalman, Matias, "Fast Inference from Transformers via
 * Speculative Decoding" (ICML 2023).  The library implements the hot path of
 * Algorithm 1: the draft model's gamma serial steps, the target model's single
 * parallel pass over gamma+1 rows, the speculative-sampling rule of
 * Section 2.3, and the roll-back of both KV caches to the accepted length.
 *
 * Conventions
 *   - Every function returns SPEC_OK (0) or a negative spec_status.  Nothing
 *     throws or aborts across this boundary.  spec_last_error() gives a
 *     human-readable message for the calling thread's last failure.
 *   - "device" pointers are CUDA device addresses on the current device;
 *     "host" pointers are ordinary host memory.  The library never takes
 *     ownership of caller memory and never frees it.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Functions that take a stream only enqueue work on it and do
 *     not synchronise unless stated.
 *   - There is no CPU fallback: without a CUDA device every compute entry
 *     point fails with SPEC_ERR_CUDA.
 *   - The library reads one environment variable, once per process:
 *     SPEC_NO_PDL=1 launches every kernel fully serialised instead of with
 *     programmatic dependent launch (same kernels, same results, slower; for
 *     debugging launch-order problems).  Nothing else in the environment
 *     changes what runs.
 */
#ifndef SPEC_DECODE_H
#define SPEC_DECODE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum spec_status {
    SPEC_OK = 0,
    SPEC_ERR_BAD_ARG = -1,        /* null pointer, negative size, value out of range */
    SPEC_ERR_BAD_CONFIG = -2,     /* model/runtime configuration not supported */
    SPEC_ERR_OOM = -3,            /* device allocation failed */
    SPEC_ERR_CAPACITY = -4,       /* prompt + n_new + gamma exceeds max_len / max_positions */
    SPEC_ERR_CUDA = -5,           /* a CUDA call failed (message has the CUDA error) */
    SPEC_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait expired */
    SPEC_ERR_NONFINITE = -7       /* spec_generate / spec_step: a model produced a NaN or +inf logit (or a row with
                                     no finite logit) in the iterations just run */
} spec_status;

/* Message for the calling thread's most recent failure ("" if none).  The
 * pointer stays valid until the thread's next failing call. */
const char* spec_last_error(void);

/* ------------------------------------------------------------------------- *
 * Speculative sampling (Section 2.3; Algorithm 1 from the accept tests to the
 * returned token).
 *
 * For each of `batch` independent sequences, given the target model's logits
 * for the gamma+1 prefixes, the draft model's logits for the gamma prefixes it
 * drafted from, the drafted tokens x_1..x_gamma and gamma+1 uniforms:
 *   p_i = softmax(target_logits[i] / T), q_i = softmax(draft_logits[i] / T)
 *   (Section 2.2; T = 0 means argmax with the lowest index winning ties);
 *   x_i is rejected iff r_i * q_i(x_i) > p_i(x_i)  (r_i > p_i(x_i)/q_i(x_i));
 *   n = number of guesses before the first rejection (gamma if none);
 *   t is drawn from norm(max(0, p_{n+1} - q_{n+1})) if n < gamma, else from
 *   p_{gamma+1}, by inverse CDF in index order with the last uniform (the
 *   smallest k whose running weight sum exceeds u times the total).  If the
 *   residual sums to zero, t is drawn from p_{n+1} unmodified.
 * At T = 0 no uniform is used and draft_logits is not read: x_i is accepted
 * iff it equals argmax p_i, and t = argmax p_{n+1}.  (For a guess that is the
 * draft's own argmax, as x_i ~ q_i gives, this is Algorithm 1's test between two
 * one-hot distributions; for any other guess the printed test divides by
 * q_i(x_i) = 0 and decides nothing: the library's rule there is the same "iff it
 * is the target's argmax".)
 *
 * All pointers are DEVICE pointers, caller-owned:
 *   target_logits [batch, gamma+1, vocab] fp32, row-major, dense
 *   draft_logits  [batch, gamma,   vocab] fp32 (may be NULL if gamma == 0 or T == 0)
 *   draft_tokens  [batch, gamma] int32, each in [0, vocab)
 *   uniforms      [batch, gamma+1] fp32 in (0,1): r_1..r_gamma, then u (may be NULL at T == 0)
 *   n_accepted    [batch] int32 out, in [0, gamma]
 *   next_token    [batch] int32 out, in [0, vocab)
 *   workspace     scratch of at least spec_verify_sample_workspace_bytes()
 *                 bytes, 256-byte aligned; contents need not be initialised
 *                 or preserved.  It must not be shared by calls that may
 *                 overlap on the device.
 * Two kernel launches are enqueued on `stream` (a streaming statistics pass
 * over all logits, then one CTA per sequence that decides and draws); the
 * call does not synchronise and allocates nothing.
 * Errors: SPEC_ERR_BAD_ARG for null pointers, batch < 0, gamma < 0 or > 64,
 * vocab < 1, temperature < 0 or not finite, workspace too small or
 * misaligned; SPEC_ERR_CUDA if the launch fails.  batch == 0 is a no-op.
 * Drafted tokens outside [0, vocab) are treated as rejected.
 * ------------------------------------------------------------------------- */
size_t spec_verify_sample_workspace_bytes(int batch, int gamma, int vocab);

int spec_verify_sample(const float* target_logits, const float* draft_logits,
                       const int32_t* draft_tokens, const float* uniforms,
                       int batch, int gamma, int vocab, float temperature,
                       int32_t* n_accepted, int32_t* next_token,
                       void* workspace, size_t workspace_bytes, void* stream);

/* The same with the lenience factor of Appendix A.5, `lenience` in (0, 1]:
 * q_i(x_i) is multiplied by it before the comparison, i.e. x_i is rejected iff
 * r_i * lenience * q_i(x_i) > p_i(x_i); the adjusted distribution after a
 * rejection stays norm(max(0, p - q)) (the appendix changes only the
 * comparison).  The output is then no longer distributed as the target's, but
 * no token is emitted with probability above p(x) / lenience.  At T = 0 lenience
 * is applied before standardising: x_i is accepted iff
 * logit(x_i) >= max logit + ln(lenience) on the target's row (p(x_i) >= lenience
 * * max p for the T = 1 softmax); the appendix prints this inequality the other
 * way round, which would accept everything at lenience 1.  lenience == 1 is
 * spec_verify_sample exactly.  Errors as above, plus SPEC_ERR_BAD_ARG for a
 * lenience outside (0, 1]. */
int spec_verify_sample_lenient(const float* target_logits, const float* draft_logits,
                               const int32_t* draft_tokens, const float* uniforms,
                               int batch, int gamma, int vocab, float temperature, float lenience,
                               int32_t* n_accepted, int32_t* next_token,
                               void* workspace, size_t workspace_bytes, void* stream);

/* The same with top-k and nucleus (top-p) standardisation.  Section 2.2 lists
 * both among the sampling methods that are a draw from an adjusted
 * distribution and asks that both models be standardised the same way; it
 * defines neither.  Here, for T > 0:
 *   0 < top_k < vocab: every logit below the top_k-th largest logit of its own
 *     row reads as -inf before the temperature softmax (logits equal to the
 *     top_k-th largest all stay, so ties can keep more than top_k);
 *   0 < top_p < 1: of what top-k left, tokens are taken in order of decreasing
 *     probability until their mass first reaches top_p of the total; every
 *     logit below the last one taken reads as -inf (ties with it stay);
 * for the target's rows and the draft's alike.  top_k == 0 or >= vocab switches
 * the first off, top_p <= 0 or >= 1 the second; with both off, or at T == 0 (the
 * maximum is always kept), this is spec_verify_sample_lenient exactly.  A
 * drafted token outside the target's kept set has p_i(x_i) = 0 and is rejected
 * unless q_i(x_i) is 0 too.  Enqueues one more kernel (the per-row selection,
 * both cuts in one launch) before the other two; same workspace.  Top-k is
 * exact.  The nucleus takes fp32 weights exp((l - max) / T) from the hardware
 * exp2 and sums them in 2^-40 fixed point with integer additions, so a row
 * always gives the same cut whatever the order of summation; a cut whose mass
 * comes within the weights' rounding (about 1e-6 of the total) of top_p may
 * differ from exact arithmetic by a neighbouring token.  Logits that are
 * -inf, +inf or NaN are never counted.  Errors as above plus SPEC_ERR_BAD_ARG
 * for top_k < 0 or a NaN top_p. */
int spec_verify_sample_truncated(const float* target_logits, const float* draft_logits,
                                 const int32_t* draft_tokens, const float* uniforms,
                                 int batch, int gamma, int vocab, float temperature, float lenience,
                                 int top_k, float top_p, int32_t* n_accepted, int32_t* next_token,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* floors[r] = the lowest logit of row r that the cuts above keep, for logits
 * [rows, vocab] fp32 device and T > 0 (fp32 device out): what the truncated
 * variants apply.  With top-k alone the result is exact (comparisons only).
 * Errors: SPEC_ERR_BAD_ARG if neither cut is active or T <= 0. */
int spec_truncation_floors(const float* logits, int rows, int vocab, float temperature,
                           int top_k, float top_p, float* floors, void* stream);

/* ------------------------------------------------------------------------- *
 * spec_verify_sample for callers that cannot allocate device memory.  (The
 * paper has no counterpart: this is a property of the library, not of the
 * method.)
 *
 * Some hosts of this library may not call cudaMalloc when they need to sample:
 * a serving process that handed all device memory to its own pool at start-up,
 * a real-time loop that forbids allocation after warm-up, a plugin that is only
 * given input and output buffers.  They have nowhere to put the workspace that
 * spec_verify_sample asks for.  This entry point computes the same result with
 * the same kernels but keeps the per-chunk softmax statistics in a fixed array
 * of spec_verify_sample_static_capacity() bytes (1 MiB) that is part of the
 * library image: every GPU that loads the library holds that array until the
 * process exits, and the call itself allocates nothing (no cudaMalloc, no
 * cudaFree, no allocating library routine).
 *
 * Arguments, layouts, asynchrony and errors are those of spec_verify_sample,
 * without the workspace.  In addition:
 *   - SPEC_ERR_CAPACITY if spec_verify_sample_workspace_bytes(batch, gamma,
 *     vocab) exceeds the built-in array (for example batch 64, gamma 7, vocab
 *     32000 needs about 105 KB; batch 1024 at the same shape does not fit).
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current); make that first call
 *     before any stream capture begins.
 *   - All calls on a device share the one array, which keeps whatever the
 *     last call left in it.  Nothing in it has to start at zero: each call
 *     overwrites every entry it later reads.  Two calls that may overlap on
 *     the device (different streams, no ordering between them) race on the
 *     array and corrupt each other's results; order them, or give one of them
 *     a workspace through spec_verify_sample.
 * ------------------------------------------------------------------------- */
size_t spec_verify_sample_static_capacity(void);

int spec_verify_sample_static(const float* target_logits, const float* draft_logits,
                              const int32_t* draft_tokens, const float* uniforms,
                              int batch, int gamma, int vocab, float temperature,
                              int32_t* n_accepted, int32_t* next_token, void* stream);

/* ------------------------------------------------------------------------- *
 * Plain standardised sampling (Section 2.2): one token per row of logits,
 * tokens[r] ~ softmax(logits[r] / T) by the same inverse-CDF rule, or the
 * lowest-index argmax at T = 0.  This is the draft model's x_i ~ q_i
 * (Algorithm 1) and target-only decoding's t ~ p.
 *   logits [rows, vocab] fp32 device; uniforms [rows] fp32 device (NULL at
 *   T == 0); tokens [rows] int32 device out.
 * Enqueues one kernel on `stream`; no synchronisation, no allocation.
 * ------------------------------------------------------------------------- */
int spec_sample(const float* logits, const float* uniforms, int rows, int vocab,
                float temperature, int32_t* tokens, void* stream);

/* The same over what top-k and the nucleus keep of each row (see
 * spec_verify_sample_truncated); floors [rows] fp32 device is scratch that
 * receives the rows' thresholds (may be NULL when both cuts are off or T == 0,
 * where the call is spec_sample).  One more kernel. */
int spec_sample_truncated(const float* logits, const float* uniforms, int rows, int vocab,
                          float temperature, int top_k, float top_p, int32_t* tokens,
                          float* floors, void* stream);

/* ------------------------------------------------------------------------- *
 * Uniforms of the method's counter-based generator, on the device.
 * out[i] = uniform(seed, positions[i], sequences[i], purpose): Philox4x32-10
 * with key = seed, counter = (position, sequence, purpose, 0), first output
 * word w mapped to (2 * (w >> 9) + 1) / 2^24.  purpose: 0 draft draw, 1 accept
 * test, 2 final draw.  (The paper does not fix how randomness is consumed;
 * this is the library's rule, the same one spec_generate uses.)
 *   positions, sequences [count] int32 device; out [count] fp32 device.
 * ------------------------------------------------------------------------- */
int spec_uniforms(uint64_t seed, const int32_t* positions, const int32_t* sequences,
                  int purpose, int count, float* out, void* stream);

/* ------------------------------------------------------------------------- *
 * Models.  The paper treats M_p and M_q as black boxes that map a prefix to a
 * next-token distribution (Section 2.1) and fixes only their sizes (Section 4:
 * GPT-like decoders, T5).  This library runs decoder-only Transformers:
 * pre-RMSNorm blocks, no biases, causal attention scaled by 1/sqrt(d_head),
 * n_heads query heads over n_kv_heads key/value heads.
 *   SPEC_ARCH_GPT:   token + learned position embeddings, FFN per `ffn`.
 *   SPEC_ARCH_LLAMA: rotary positions (rotate-half pairing j, j + d_head/2,
 *                    angle position * rope_base^(-2j/d_head)) on q and k.
 *   SPEC_ARCH_T5:    encoder-decoder (the T5-shaped pairs of Section 4.1; the
 *                    paper fixes only their sizes).  No absolute positions;
 *                    self-attention scores get, after scaling, an additive
 *                    bias table[bucket(key pos - query pos)][head] with the
 *                    usual log-spaced buckets (rel_buckets of them up to
 *                    rel_max_distance; two mirrored halves in the encoder,
 *                    backwards only in the decoder), one table per stack.
 *                    The encoder (n_enc_layers blocks, every source position
 *                    sees every other, output RMS-normalised with enc_ln_f)
 *                    runs once per source.  A decoder block is causal
 *                    self-attention, cross-attention (q = Wq_x . rmsnorm(h)
 *                    with gain lnx; [K; V] = Wkv_x . encoder output, computed
 *                    once; no bias; out-projection Wo_x) and the FFN.
 *                    n_kv_heads == n_heads; decoding starts from token id 0.
 *   SPEC_ARCH_BIGRAM: a negligible-cost approximation model (the paper's
 *                    Section 4 evaluates unigram and bigram drafts): the next-token logits depend
 *                    on the last token only, logits = table[token].  Only
 *                    valid as the DRAFT.  tok_emb points at the table
 *                    [vocab, vocab] (row = last token) in `dtype`; only `arch`,
 *                    `vocab` and `dtype` of the config are read, no other
 *                    weight pointer is used, and it keeps no K,V rows.
 *   SPEC_ARCH_COPY:   a parameter-less negligible-cost approximation model
 *                    (Section 3.6 suggests one that copies tokens from the
 *                    context where a matching prefix is found; no procedure
 *                    is given).  Ours: let s be the sequence so far and n =
 *                    `ngram` >= 1.  The guess is the token that followed the
 *                    most recent earlier occurrence of the last n tokens of s,
 *                    i.e. s[j+1] for the largest j < len(s)-1 with
 *                    s[j-n+1..j] == s[len-n..len-1]; if there is none (or s has
 *                    fewer than n+1 tokens) the last token is repeated.  q is
 *                    one-hot at the guess (logit 0 there, -inf elsewhere), so
 *                    Algorithm 1 accepts it with probability p(guess) and
 *                    otherwise draws from p with the guess removed.  Only
 *                    valid as the DRAFT; only `arch`, `vocab` and `ngram` are
 *                    read; no weights, no K,V rows; no teacher-forced pass
 *                    (spec_forward_logits refuses it).
 *   FFN: SPEC_FFN_GELU (tanh approximation) with W_in [d_ff, d_model];
 *        SPEC_FFN_GATED_GELU / SPEC_FFN_SWIGLU with W_in [2*d_ff, d_model],
 *        rows 0..d_ff-1 the gate, rows d_ff..2*d_ff-1 the up projection.
 * Matrices are row-major [out_features, in_features] in `dtype` (fp32, or
 * bf16 as raw 16-bit patterns); gains are fp32.  The residual stream, softmax,
 * normalisation and logits are fp32 in every configuration.
 * ------------------------------------------------------------------------- */
enum { SPEC_ARCH_GPT = 0, SPEC_ARCH_LLAMA = 1, SPEC_ARCH_T5 = 2, SPEC_ARCH_BIGRAM = 3, SPEC_ARCH_COPY = 4 };
enum { SPEC_FFN_GELU = 0, SPEC_FFN_GATED_GELU = 1, SPEC_FFN_SWIGLU = 2 };
enum { SPEC_DTYPE_FP32 = 0, SPEC_DTYPE_BF16 = 1, SPEC_DTYPE_FP16 = 2 /* cached K,V rows only */ };

typedef struct spec_model_cfg {
    int arch;             /* SPEC_ARCH_* */
    int n_layers;
    int d_model;
    int n_heads;
    int n_kv_heads;       /* divides n_heads */
    int d_head;           /* 64 or 128 */
    int d_ff;
    int ffn;              /* SPEC_FFN_* */
    int vocab;
    int max_positions;    /* rows of pos_emb (GPT); upper bound on positions */
    int tied_embeddings;  /* 1: the LM head is tok_emb */
    int dtype;            /* SPEC_DTYPE_* of every matrix */
    float rms_eps;
    float rope_base;
    int n_enc_layers;     /* T5: encoder blocks (0 otherwise) */
    int rel_buckets;      /* T5: rows of the bias tables (even, 2..256) */
    int rel_max_distance; /* T5: distance from which the last bucket is used */
    int ngram;            /* SPEC_ARCH_COPY: length of the matched suffix (0 otherwise) */
} spec_model_cfg;

typedef struct spec_layer_weights {
    const float* ln1;     /* [d_model] */
    const void* wqkv;     /* [(n_heads + 2 n_kv_heads) d_head, d_model]: q rows, k rows, v rows */
    const void* wo;       /* [d_model, n_heads d_head] */
    const float* ln2;     /* [d_model] */
    const void* w_in;     /* [d_ff or 2 d_ff, d_model] */
    const void* w_out;    /* [d_model, d_ff] */
    /* T5 decoder blocks only (NULL otherwise): cross-attention */
    const float* lnx;     /* [d_model] */
    const void* wq_x;     /* [n_heads d_head, d_model] */
    const void* wkv_x;    /* [2 n_heads d_head, d_model]: k rows, v rows */
    const void* wo_x;     /* [d_model, n_heads d_head] */
} spec_layer_weights;

/* All pointers are DEVICE pointers that the caller keeps alive until
 * spec_free(); `layers` itself is a HOST array of n_layers entries that is
 * copied during spec_init. */
typedef struct spec_weights {
    const void* tok_emb;  /* [vocab, d_model] */
    const void* pos_emb;  /* [max_positions, d_model], GPT only */
    const float* ln_f;    /* [d_model] */
    const void* head;     /* [vocab, d_model]; ignored when tied_embeddings */
    const spec_layer_weights* layers;
    /* T5 only (NULL otherwise) */
    const spec_layer_weights* enc_layers; /* HOST array of n_enc_layers entries */
    const float* enc_ln_f;                /* [d_model] */
    const float* enc_rel_bias;            /* fp32 [rel_buckets, n_heads] */
    const float* rel_bias;                /* fp32 [rel_buckets, n_heads], decoder */
} spec_weights;

typedef struct spec_runtime_cfg {
    int max_batch;        /* sequences decoded together */
    int max_len;          /* tokens per sequence the KV caches can hold (prompt + new + gamma) */
    int page_size;        /* tokens per KV page (power of two, 32..256) */
    int max_gamma;        /* largest gamma spec_generate will be asked for */
    int kv_dtype;         /* element type of the cached K,V rows: SPEC_DTYPE_FP32, SPEC_DTYPE_FP16 or
                             SPEC_DTYPE_BF16.  The 16-bit types halve the K,V traffic.  fp16 keeps 11
                             significant bits (values beyond +-65504 are stored as +-65504) and stays
                             inside the 2e-2 logit tolerance of bf16 models; bf16 keeps 8, which on
                             wide or deep models moves logits by more than that. */
    int max_src_len;      /* T5: longest source the encoders are given (0 for decoder-only models) */
    int pass_kernel;      /* 0 (default): every pass is a chain of kernels.  1: passes of at most 16 rows of
                             a bf16 GPT- or Llama-shaped model run as one persistent cooperative kernel
                             (one CTA per SM, grid-wide barriers between the steps, weights streamed
                             ahead of the steps that wait); same results within the parity tolerances,
                             measured slower than the chain on a B200 (see spec_pass_trace). */
} spec_runtime_cfg;

typedef struct spec_ctx spec_ctx;

/* Counters of one spec_generate call (Section 3: what alpha, E[#tokens] and the
 * walltime analysis are computed from). */
typedef struct spec_stats {
    int64_t iterations;       /* runs of Algorithm 1, summed over sequences */
    int64_t tokens;           /* tokens emitted by those runs (before truncation to n_new) */
    int64_t tests_evaluated;  /* accept tests that were reached (i <= n + 1) */
    int64_t tests_passed;     /* drafted tokens accepted */
    int64_t target_passes;    /* batched forward passes of M_p inside the decode loop */
    int64_t draft_passes;     /* batched forward passes of M_q inside the decode loop */
    double prefill_ms;        /* device time of the prompt pass */
    double decode_ms;         /* device time of the decode loop */
    int64_t accepted_histogram[65]; /* [n]: runs of Algorithm 1 that accepted exactly n guesses (n <= gamma <= 64):
                                 for i.i.d. acceptance the capped geometric law behind Eq. 1 */
} spec_stats;

/* Creates a context for a target model and (optionally, draft_cfg == NULL for
 * target-only decoding) a draft model with the same vocabulary.  Allocates the
 * paged KV caches, activations and logits buffers with cudaMalloc on the
 * current device and creates a private stream.  Weights are borrowed; for bf16
 * models the library also makes its own tile-major copies of the block matrices
 * and the LM head (see spec_pack_weight), which doubles their footprint.
 * Errors: SPEC_ERR_BAD_ARG (null), SPEC_ERR_BAD_CONFIG (unsupported shapes,
 * vocabularies differ), SPEC_ERR_OOM, SPEC_ERR_CUDA. */
int spec_init(const spec_model_cfg* target_cfg, const spec_model_cfg* draft_cfg,
              const spec_weights* target_weights, const spec_weights* draft_weights,
              const spec_runtime_cfg* runtime, spec_ctx** out);

/* Releases everything spec_init allocated (not the weights). NULL is allowed. */
void spec_free(spec_ctx* ctx);

/* Generation by speculative decoding (Algorithm 1 repeated): for each of
 * `batch` sequences, emits exactly n_new tokens after its prompt.
 *   prompt      HOST int32 [batch, prompt_stride]; sequence b uses the first
 *               prompt_len[b] >= 1 entries of its row
 *   prompt_len  HOST int32 [batch]
 *   gamma       drafted tokens per iteration; 0 = plain autoregressive
 *               decoding from the target alone with the same kernels
 *   temperature 0 = greedy (argmax, lowest index on ties)
 *   seed        key of the counter-based generator (see spec_uniforms): the
 *               draft's draw of the token at position s uses purpose 0, its
 *               accept test purpose 1, the final draw of an iteration purpose
 *               2, each with counter (s, sequence index)
 *   out_tokens  HOST int32 [batch, n_new]
 *   stats       HOST, may be NULL
 * Both models first consume the prompt; then each iteration runs the draft
 * gamma times (one row per sequence; two in the first step, which re-feeds
 * the previous token so that the draft catches up after an iteration that
 * accepted every guess), the target once over gamma+1 rows per sequence, the
 * speculative-sampling rule, and the roll-back of both caches to the accepted
 * length.  The last iteration's surplus tokens are dropped.  The call blocks
 * until the tokens are on the host.
 * Errors: SPEC_ERR_BAD_ARG; SPEC_ERR_CAPACITY if prompt_len + n_new + gamma + 1
 * exceeds max_len or a model's max_positions, batch > max_batch or
 * gamma > max_gamma; SPEC_ERR_BAD_CONFIG if gamma > 0 without a draft model. */
int spec_generate(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride,
                  int batch, int n_new, int gamma, float temperature, uint64_t seed,
                  int32_t* out_tokens, spec_stats* stats);

/* Encoder-decoder models (SPEC_ARCH_T5): `prompt` holds the SOURCE of every
 * sequence.  spec_generate / spec_begin run both encoders over it once, keep
 * the cross-attention K,V of every decoder block, and then decode n_new tokens
 * from the start token 0 exactly as above (the decoder's "prompt" is that one
 * token).  SPEC_ERR_CAPACITY also if a source is longer than max_src_len. */

/* The same generation in phases, for callers that interleave other work or
 * time the decode loop: spec_begin validates the request, uploads the prompts
 * and runs the prompt pass (arguments as for spec_generate); spec_step runs
 * `iterations` iterations of Algorithm 1 for the whole batch (sequences that
 * already have n_new tokens are frozen), blocks until they are done and reports
 * in *remaining (may be NULL) the largest number of tokens any sequence still
 * lacks; *stats (may be NULL) gets the counters since spec_begin, with
 * decode_ms the device time of this call alone.  spec_read_tokens copies the
 * n_new tokens of every sequence to HOST int32 [batch, n_new] (entries not yet
 * generated are unspecified).  A teacher-forced diagnostic call ends the
 * generation in progress. */
int spec_begin(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride,
               int batch, int n_new, int gamma, float temperature, uint64_t seed);

/* Lenience factor (Appendix A.5; see spec_verify_sample_lenient) used by the
 * generations that start after this call; 1 (the default) is Algorithm 1 as
 * printed.  Errors: SPEC_ERR_BAD_ARG outside (0, 1]. */
int spec_set_lenience(spec_ctx* ctx, float lenience);

/* top-k and nucleus standardisation (see spec_verify_sample_truncated) of both
 * models in the generations that start after this call: the draft draws x_i
 * from its truncated distribution, the accept tests and the final draw use the
 * target's and the draft's truncated distributions, and gamma = 0 decodes from
 * the target's.  top_k = 0 and top_p = 1 (the defaults): the whole vocabulary.
 * Errors: SPEC_ERR_BAD_ARG for top_k < 0 or a NaN top_p. */
int spec_set_truncation(spec_ctx* ctx, int top_k, float top_p);

/* Timing instrument (no counterpart in Algorithm 1): from the next spec_begin /
 * spec_generate on, the accept decision of every drafted token is replaced by
 * "r_i < alpha" with the same uniforms r_i, i.e. an i.i.d. Bernoulli(alpha)
 * acceptance as the analysis of Section 3.1-3.2 assumes, whatever p and q say;
 * the final token is still drawn by the sampler.  The emitted tokens are then
 * NOT distributed as the target's: use it only to time iterations at a chosen
 * acceptance rate (random-init model pairs sit at one uncontrolled alpha).
 * alpha < 0 restores Algorithm 1.  Errors: SPEC_ERR_BAD_ARG (alpha > 1 or NaN). */
int spec_set_imposed_acceptance(spec_ctx* ctx, float alpha);

/* Encoder-decoder models only: runs the encoder of every model of the context
 * over the sources (HOST int32 [batch, source_stride], source_len[b] >= 1
 * entries used) and stores the cross-attention K,V; forgets every cached
 * decoder row.  spec_generate and spec_begin call it themselves; the
 * teacher-forced diagnostics below need it called first.  Blocks until done.
 * Errors: SPEC_ERR_BAD_ARG, SPEC_ERR_BAD_CONFIG (not an encoder-decoder
 * context), SPEC_ERR_CAPACITY (batch > max_batch, a source longer than
 * max_src_len). */
int spec_encode(spec_ctx* ctx, const int32_t* source, const int32_t* source_len, int source_stride, int batch);

/* The relative-position bucket of SPEC_ARCH_T5 for delta = key position - query
 * position (host arithmetic only; exported so that it can be checked without a
 * GPU).  Negative return: SPEC_ERR_BAD_ARG for a table shape spec_init would
 * reject. */
int spec_rel_bucket(int delta, int bidirectional, int n_buckets, int max_distance);
int spec_step(spec_ctx* ctx, int iterations, int* remaining, spec_stats* stats);
int spec_read_tokens(spec_ctx* ctx, int32_t* out_tokens);

/* Choosing gamma (Section 3.5: the optimal gamma is the integer that maximises
 * the walltime improvement for given alpha and c; the same section names
 * varying gamma during a run as a further refinement and leaves it open).
 *
 * spec_choose_gamma is host arithmetic, no device involved: the gamma in
 * [1, gamma_max] that maximises expected tokens per unit of time,
 *   (1 + alpha + ... + alpha^gamma) / (base_cost + cost_per_guess * gamma),
 * the numerator being Eq. 1; lowest gamma on ties.  With base_cost = 1 and
 * cost_per_guess = c this is the maximiser of Theorem 3.8's improvement factor
 * (1 - alpha^(gamma+1)) / ((1 - alpha)(gamma c + 1)).  Returns -1 for alpha
 * outside [0, 1], base_cost <= 0, cost_per_guess < 0 or gamma_max < 1.
 *
 * spec_set_gamma changes the number of guesses per iteration of the generation
 * in progress, between spec_step calls: 1 <= gamma <= the gamma given to
 * spec_begin (whose capacity check covers it).  gamma = 0 is refused: such
 * iterations would not feed the draft model.  Iteration graphs are kept per
 * gamma, so going back to an earlier gamma costs nothing.  Because the
 * randomness is keyed by position, the tokens depend on the sequence of gammas
 * but on nothing else; at T = 0 they do not depend on it at all.
 *
 * spec_generate_adaptive is spec_generate with gamma chosen by the library:
 * iterations run in bursts of at most `burst`; the first burst uses gamma = 1,
 * the second gamma_max, and from then on the gamma spec_choose_gamma returns
 * for alpha = accepted / evaluated guesses so far, with the counts of earlier
 * bursts fading by 0.8 per burst, and a straight line fitted to the measured
 * device time per iteration of every gamma tried.  trace (HOST int32, may be
 * NULL with trace_capacity 0) receives (gamma, iterations) per burst, as many
 * pairs as fit; *n_bursts (may be NULL) the number of bursts.  Replaying the
 * trace with spec_begin / spec_set_gamma / spec_step gives the same tokens.
 * Errors as spec_generate; gamma_max < 1 or burst < 1: SPEC_ERR_BAD_ARG. */
int spec_choose_gamma(double alpha, double base_cost, double cost_per_guess, int gamma_max);
int spec_set_gamma(spec_ctx* ctx, int gamma);
int spec_generate_adaptive(spec_ctx* ctx, const int32_t* prompt, const int32_t* prompt_len, int prompt_stride,
                           int batch, int n_new, int gamma_max, float temperature, uint64_t seed, int burst,
                           int32_t* out_tokens, spec_stats* stats, int32_t* trace, int trace_capacity,
                           int* n_bursts);

/* Diagnostics for parity tests: teacher-forced forward passes on the KV caches.
 * spec_reset forgets every cached row.  spec_forward_logits feeds, for each
 * of `batch` sequences, `rows` tokens at positions cached_len[b].. of model
 * `which` (0 target, 1 draft), appends their K,V rows and writes fp32 logits
 * [batch, rows, vocab] to the DEVICE buffer `logits`; tokens is HOST int32
 * [batch, rows].  spec_truncate sets the cached length of every sequence of
 * the model (HOST int32 [batch]); later passes overwrite the dropped rows.
 * All three synchronise. */
int spec_reset(spec_ctx* ctx);
int spec_forward_logits(spec_ctx* ctx, int which, const int32_t* tokens, int batch, int rows, float* logits);
int spec_truncate(spec_ctx* ctx, int which, const int32_t* lengths, int batch);

/* Diagnostic for the parity tests: how the library would run the attention of a
 * pass of model `which` over `rows` rows per sequence for `batch` sequences
 * (Algorithm 1's parallel pass has rows = gamma + 1; a draft step has 1 or 2),
 * `cross` != 0 for the cross-attention of an encoder-decoder block.  The choice
 * depends on the shapes and on the context's capacities (max_len, max_src_len)
 * only, never on the data.  plan (HOST int32 [4]) receives
 *   plan[0]  0: one warp per query on the FMA pipes; 1: the queries of a KV head
 *               are multiplied on the tensor cores in tf32 from rows converted to
 *               fp32; 2: in f16 straight from fp16 rows, all the queries of a KV
 *               head in one CTA;
 *   plan[1]  key slices (CTAs) per (sequence, KV head);
 *   plan[2]  1: the slices are merged inside a thread-block cluster, 0: by a
 *               second kernel from partial states in global memory;
 *   plan[3]  1: K and V of a key tile share one staging buffer (tensor-core
 *               kernel only).
 * No device work.  Errors: SPEC_ERR_BAD_ARG, SPEC_ERR_BAD_CONFIG. */
int spec_attention_plan(spec_ctx* ctx, int which, int batch, int rows, int cross, int* plan);

/* Diagnostic: where the time of one pass goes.  Passes of at most 16 rows of a bf16
 * decoder-only model run as one persistent kernel (one CTA per SM) whose steps (GEMMs,
 * rotary + append, attention, merge) are separated by grid-wide barriers.  This call runs
 * such a pass twice at the cached lengths (as spec_time_forward does; the second run is
 * the traced one) and returns the CTAs' clocks: stamps_ns[0] is the number of CTAs P,
 * stamps_ns[1] the start of the pass, and stamps_ns[2 + (k - 1) * P + c] the time CTA c
 * arrived at the k-th barrier (k = 1, 2, ...), in nanoseconds of the GPU's global timer;
 * a barrier opens when its last CTA has arrived.  *count entries are valid.  HOST buffer
 * of `capacity` entries.  Synchronises and, unlike every other entry point, allocates and
 * frees device memory for the stamps.
 * Errors: SPEC_ERR_BAD_CONFIG if such a pass does not take the persistent kernel. */
int spec_pass_trace(spec_ctx* ctx, int which, int batch, int rows, unsigned long long* stamps_ns, int capacity, int* count);

/* Device time of one forward pass of model `which` over `rows` rows per
 * sequence for `batch` sequences, at the cached lengths the diagnostics above
 * have built up (the quantities c and the cost of gamma+1 parallel rows in the
 * walltime analysis of Section 3.3 are ratios of such times).  The pass (token
 * 0 in every row, logits of every row computed and discarded) is captured in a
 * CUDA graph once and replayed `repeats` times between two events on the
 * context's stream; *ms_per_pass gets the mean.  The cached lengths do not
 * change (the rows are written beyond them).  Synchronises.
 * Errors as spec_forward_logits. */
int spec_time_forward(spec_ctx* ctx, int which, int batch, int rows, int repeats, float* ms_per_pass);

/* ------------------------------------------------------------------------- *
 * One linear layer y = x . W^T, the building block of the verification pass
 * (the paper's premise, Section 1 and Section 3.4: the pass is bound by
 * streaming W from memory, and gamma+1 rows share one stream of the weights).
 *   x [rows, k] fp32 device; w [n_out, k] device in w_dtype (SPEC_DTYPE_*);
 *   y [rows, n_out] fp32 device out; k a multiple of 8.
 *   path 0: tensor cores for bf16 weights, FMA pipes for fp32; 1: FMA pipes;
 *        2: tensor cores (bf16 only); 3: tensor cores with `w` in the
 *           tile-major layout that spec_pack_weight produces, which is what
 *           the engine streams: every [128 x 64] tile of W is contiguous
 *           (tiles ordered by 128-row band, then by 64-column block; rows and
 *           columns past the matrix are zero; inside a tile row the eight
 *           16-byte chunks are stored in shared-memory swizzle order, chunk c
 *           of row r at position c ^ (r & 7)), so that a CTA's weight stream
 *           is one sequential run of HBM and a tile is copied as it is.
 * The tensor-core path splits x into two bf16 terms and sums split-K partial
 * results in a fixed order; it needs `workspace` (device, 256-byte aligned, at
 * least spec_linear_workspace_bytes(rows, n_out, k) bytes, contents arbitrary,
 * not shared by overlapping calls).  The FMA path ignores the workspace.
 * Asynchronous on `stream`; allocates nothing.
 * spec_device_error() returns non-zero (and clears it) if a kernel of this
 * library gave up on a bounded device-side wait since the last call; it
 * synchronises with the device.
 * ------------------------------------------------------------------------- */
size_t spec_linear_workspace_bytes(int rows, int n_out, int k);
/* Bytes of the tile-major copy of a bf16 matrix [n_out, k], and the copy itself
 * (device pointers, asynchronous on `stream`). */
size_t spec_packed_weight_bytes(int n_out, int k);
int spec_pack_weight(const void* w, int n_out, int k, void* packed, void* stream);

/* The tensor-core weight-streaming GEMM exactly as the decoder engine launches it
 * for one matrix: tile-major weights (spec_pack_weight), the activations as two
 * bf16 terms, split-K partial sums left for the consumer (in the engine the next
 * small kernel adds them up).  With split_input != 0 the fp32 rows x [rows, k] are
 * first split into the workspace; with 0 the split made by an earlier call with
 * the same (rows, k) and workspace is reused, so that a sweep over many matrices
 * launches nothing but the GEMM kernel.  *partial (may be NULL) receives the
 * DEVICE address, inside the workspace, of the sums [*splits][rows][n_out] fp32;
 * their sum over the first index, in index order, is x . W^T.  Workspace as for
 * spec_linear.  Asynchronous on `stream`.  Errors: SPEC_ERR_BAD_ARG. */
int spec_linear_partials(const float* x, const void* w_packed, int rows, int n_out, int k, int split_input,
                         void* workspace, size_t workspace_bytes, float** partial, int* splits, void* stream);
int spec_linear(const float* x, const void* w, int w_dtype, int rows, int n_out, int k, int path,
                float* y, void* workspace, size_t workspace_bytes, void* stream);
int spec_device_error(void);

/* Failure-path drill (no counterpart in the paper).  Every wait inside the library's kernels on
 * a barrier or a flag is bounded: when it runs out the kernel records a code, frees the tensor
 * memory it holds and returns, and the next synchronising call of the library reports
 * SPEC_ERR_DEVICE_TIMEOUT instead of hanging the GPU.  This call exercises that path without
 * breaking anything: it launches the tensor-core GEMM kernel on one tile with its producer
 * switched off (nothing is requested from memory, so nothing is in flight when the CTA gives
 * up) and a limit of 4096 polls, waits for it, and returns SPEC_ERR_DEVICE_TIMEOUT if the kernel
 * reported the expired wait as it should (SPEC_ERR_CUDA if it did not).  The device error flag
 * is clear afterwards and the context stays usable.  Synchronises `stream`. */
int spec_timeout_drill(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_DECODE_H */
