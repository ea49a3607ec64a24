"""Algorithm 1 looped to a fixed number of new tokens, and target-only decoding.

Test infrastructure (see the package docstring).

Conventions the paper leaves open, fixed here:

* L = number of committed tokens (prompt + emitted so far).  Committed tokens
  occupy positions 0..L-1.  The drafted token x_i (i = 1..gamma) is the
  candidate for position L+i-1; the final token t is the token for position
  L+n.
* Randomness: oracle.philox.uniform(seed, position, sequence, purpose) with
  purpose 0 for the draft's draw of the token at `position`, 1 for its accept
  test, 2 for the final draw of the token at `position`.  Target-only decoding
  draws the token at position L with purpose 2.
* gamma is fixed for the run; the last iteration may overshoot n_new, and the
  surplus is dropped (a prefix of a correctly distributed sequence is correctly
  distributed).  No end-of-sequence handling.
* `cached=False` recomputes every prefix from position 0 with nothing kept
  between calls, so it cannot be wrong about KV rollback; `cached=True` keeps
  KV rows and truncates them after a rejection.  The tests require the two to
  agree.

Pins (tests/test_oracle_generate.py): at T = 0 the output equals target-only
greedy decoding for every gamma (abstract; Section 2.2); with table "models"
on vocabularies <= 8 the exact law of the emitted sequence, enumerated over
the probability tree of Algorithm 1, equals prod_t p(x_t | x_<t); with the
same fixed p, q at every position the mean number of tokens per iteration
equals Eq. 1 and every iteration emits between 1 and gamma + 1 tokens.
"""

from dataclasses import dataclass, field

import numpy as np

from . import philox
from .sampling import sample_token, verify_step


@dataclass
class IterationRecord:
    start_len: int  # L at the start of the iteration
    draft_tokens: list
    n_accepted: int
    next_token: int
    accept_margin: float
    cdf_margin: float
    top2_gap: float
    draft_cdf_margins: list
    betas: list
    target_logits: np.ndarray = None  # [gamma+1, V], kept when asked for
    draft_logits: np.ndarray = None  # [gamma, V]


@dataclass
class GenerationResult:
    tokens: list  # exactly n_new emitted tokens
    iterations: list = field(default_factory=list)

    @property
    def tests_evaluated(self):
        return sum(min(it.n_accepted + 1, len(it.draft_tokens)) for it in self.iterations)

    @property
    def tests_passed(self):
        return sum(it.n_accepted for it in self.iterations)


def speculative_generate(target, draft, prompt, n_new, gamma, temperature, seed, sequence=0, cached=True, keep_logits=False,
                         lenience=1.0, top_k=0, top_p=1.0):
    """Algorithm 1 repeated until n_new tokens are emitted.

    `gamma` is an integer, or a sequence giving the number of guesses of every
    iteration in turn (Section 3.5 allows gamma to vary during a run; the last
    entry is used for any further iterations).

    `target` and `draft` are model objects with forward_rows / forward_full /
    truncate / reset (oracle.decoder.Decoder or a table model from the tests).
    """
    committed = [int(t) for t in prompt]
    prompt_len = len(committed)
    result = GenerationResult(tokens=[])
    if cached:
        target.reset()
        draft.reset()
        if prompt_len > 1:
            target.forward_rows(committed[:-1])
            draft.forward_rows(committed[:-1])

    schedule = None if np.isscalar(gamma) else [int(g) for g in gamma]
    while len(committed) - prompt_len < n_new:
        L = len(committed)
        if schedule is not None:
            gamma = schedule[min(len(result.iterations), len(schedule) - 1)]
        # Draft gamma guesses autoregressively.
        xs, q_logits, draft_margins = [], [], []
        for i in range(1, gamma + 1):
            if cached:
                # Every token the draft has not seen yet: normally one, two after
                # an iteration that accepted all gamma guesses (x_gamma was never fed).
                row = draft.forward_rows((committed + xs)[draft.cached_len :])[-1]
            else:
                row = draft.forward_full(committed + xs)[-1]
            u = philox.uniform(seed, L + i - 1, sequence, philox.PURPOSE_DRAFT)
            x, margin = sample_token(row, u, temperature, top_k, top_p)
            xs.append(x)
            q_logits.append(row)
            draft_margins.append(margin)
        # Run the target on the gamma + 1 prefixes in parallel.
        if cached:
            p_logits = target.forward_rows((committed + xs)[target.cached_len :])[-(gamma + 1) :]
        else:
            p_logits = target.forward_full(committed + xs)[L - 1 : L + gamma]
        # Accept, adjust, draw.
        uniforms = [philox.uniform(seed, L + i - 1, sequence, philox.PURPOSE_ACCEPT) for i in range(1, gamma + 1)]
        q_arr = np.stack(q_logits) if gamma else np.zeros((0, p_logits.shape[1]))
        # The final draw decides the token at position L + n, known only after
        # the accept tests: evaluate once with a placeholder to find n.
        probe = verify_step(p_logits, q_arr, xs, uniforms + [0.5], temperature, lenience, top_k, top_p)
        u_final = philox.uniform(seed, L + probe.n_accepted, sequence, philox.PURPOSE_FINAL)
        res = verify_step(p_logits, q_arr, xs, uniforms + [u_final], temperature, lenience, top_k, top_p)
        n = res.n_accepted
        committed.extend(xs[:n])
        committed.append(res.next_token)
        if cached:
            # Keep rows for positions 0..L+n-1 (the last committed token is not fed yet).
            target.truncate(L + n)
            draft.truncate(min(L + n, draft.cached_len))
        result.iterations.append(
            IterationRecord(
                L, xs, n, res.next_token, res.accept_margin, res.cdf_margin, res.top2_gap, draft_margins, res.betas,
                np.array(p_logits) if keep_logits else None, np.array(q_arr) if keep_logits else None,
            )
        )
    result.tokens = committed[prompt_len : prompt_len + n_new]
    return result


def target_only_generate(target, prompt, n_new, temperature, seed, sequence=0, cached=True, keep_logits=False, top_k=0, top_p=1.0):
    """Standard autoregressive decoding from the target alone (cost T per token)."""
    committed = [int(t) for t in prompt]
    prompt_len = len(committed)
    rows = []
    margins = []
    if cached:
        target.reset()
    for _ in range(n_new):
        L = len(committed)
        if cached:
            row = target.forward_rows(committed[target.cached_len :])[-1]
        else:
            row = target.forward_full(committed)[-1]
        u = philox.uniform(seed, L, sequence, philox.PURPOSE_FINAL)
        t, margin = sample_token(row, u, temperature, top_k, top_p)
        committed.append(t)
        margins.append(margin)
        if keep_logits:
            rows.append(np.array(row))
    return committed[prompt_len:], rows, margins
