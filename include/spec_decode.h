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
    SPEC_ERR_NONFINITE = -7       /* non-finite logits were seen */
} spec_status;

/* Message for the calling thread's most recent failure ("" if none).  The
 * pointer stays valid until the thread's next failing call. */
const char* spec_last_error(void);

/* ------------------------------------------------------------------------- *
 * Speculative sampling (Section 2.3; Algorithm 1 from "determine the number
 * of accepted guesses" to "return").
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
 * iff it equals argmax p_i (x_i is assumed to be the draft's own argmax), and
 * t = argmax p_{n+1}.
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

#ifdef __cplusplus
}
#endif
#endif /* SPEC_DECODE_H */
