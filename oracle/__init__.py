"""CPU oracle for the speculative-decoding hot path.

TEST INFRASTRUCTURE ONLY.  Everything under this package is a plain, slow,
obviously-correct CPU restatement of what the CUDA library computes, written
from the paper (Leviathan, Kalman, Matias, "Fast Inference from Transformers
via Speculative Decoding", ICML 2023).  It exists so that the CUDA path can be
compared against something independent of itself.  It shares no code with the
CUDA path and never imports it.  Only the test-suite, the smoke check and the
benchmark's `cpu_baseline` / reference arm may import it; the product never
does.

Modules
-------
philox    counter-based generator (Philox4x32-10) and the uniform grid used for
          every random draw of the method.
sampling  Section 2.2 standardisation, Section 2.3 speculative sampling, the
          accept/adjust/draw part of Algorithm 1.
analysis  closed forms: Definition 3.2 / Lemma 3.3 (D_LK), Theorem 3.5 (beta),
          Eq. 1, Theorem 3.8, Corollary 3.9, Theorem 3.11, Section 3.5.
decoder   the two decoder families the synthetic configs use (GPT-like with
          learned positions, Llama-like with rotary positions and grouped KV
          heads), cache-free and cached.
generate  Algorithm 1 looped to a fixed number of new tokens, plus target-only
          decoding.

Pins (what each part is checked against, other than itself) are listed in the
header of each module; a part with no such pin says "parity unpinned".
"""
