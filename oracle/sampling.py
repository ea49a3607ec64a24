"""Standardised sampling, speculative sampling and the accept/adjust/draw part
of Algorithm 1, in fp64, one element at a time where order matters.

Test infrastructure (see the package docstring).

What follows the paper, and where it is silent:

* Section 2.2: every sampling method is a draw from an adjusted distribution.
  Temperature T > 0 gives softmax(logits / T); T = 0 (argmax) zeroes every
  non-maximal entry and normalises.  Reading for ties: the lowest index keeps
  all the mass, so the adjusted distribution is always one-hot at T = 0.
* Section 2.3 / Algorithm 1: a drafted token x_i ~ q_i is rejected iff
  r_i > p_i(x_i) / q_i(x_i).  The bare `x` printed in the algorithm's test is
  the drafted token x_i.  The test is evaluated without a division, as
  r_i * q_i(x_i) > p_i(x_i), which is the same predicate for q_i(x_i) > 0 and
  never rejects when q_i(x_i) = 0 (a token the draft could not have drawn).
* n = number of drafted tokens before the first rejection (gamma if none).
  p' = p_{n+1}; if n < gamma, p' = norm(max(0, p_{n+1} - q_{n+1})).
  Appendix A.1: the normaliser equals 1 - beta with beta = sum min(p, q).
  Reading for a vanishing normaliser (unreachable in exact arithmetic after a
  genuine rejection): draw from p_{n+1} unmodified and report it.
* How a categorical draw is made is not stated.  Reading: inverse CDF in index
  order on unnormalised weights w: the smallest k with w_0 + ... + w_k > u * W,
  W the total; if rounding leaves none, the last k with w_k > 0.

* Appendix A.5 (lenience l in (0, 1]): q(x) is multiplied by l before it is
  compared with p(x): reject iff r_i * l * q_i(x_i) > p_i(x_i).  The text
  changes only the comparison; reading: the adjusted distribution after a
  rejection stays norm(max(0, p - q)) (a rejection still implies q(x) > p(x),
  so it is well defined, and no token is then emitted with probability above
  p(x) / l).  At T = 0 the paper applies lenience before standardising; its
  printed condition "p(x) <= l * max(p)" would accept everything at l = 1, so
  the inequality is read the other way round: x_i is accepted iff
  p(x_i) >= l * max p with p the T = 1 softmax of the target's logits, i.e.
  logit(x_i) >= max logit + ln l; l = 1 keeps the strict rule (x_i accepted
  iff it is the lowest-index maximum).

* Section 2.2 names top-k among the sampling methods that reduce to a draw
  from an adjusted distribution and gives no definition.  Reading: with k > 0,
  every logit below the k-th largest logit of its row is set to -inf before
  the temperature softmax (entries equal to the k-th largest all stay, so
  ties can keep more than k); k = 0 or k >= vocabulary changes nothing.  The
  same k standardises p and q, as the section asks.  T = 0 ignores k (the
  maximum is always kept).
* Nucleus sampling is named in the same sentence, again without a definition.
  Reading (the usual one): with 0 < top_p < 1, tokens are taken in order of
  decreasing probability under the temperature softmax (of the top-k logits
  when k is set: top-k first, then the nucleus of what is left) until their
  mass first reaches top_p of the total; every logit below the last one taken
  is set to -inf (logits equal to it all stay) and the rest is renormalised.
  top_p >= 1 (or <= 0) changes nothing; T = 0 ignores it.

Pins (tests/test_oracle_sampling.py): the nucleus against a
take-the-maximum-until-the-mass-is-reached restatement, on a hand-computed
four-token example, its limits (top_p -> 0 keeps the argmax, top_p = 1 keeps
everything), its composition with top-k, and the emitted-token law under it;
top-k against a pick-the-maximum-k-times
restatement, its support size, the preserved ratios inside the support, k = 1
against argmax and k >= V against plain softmax, and the emitted-token law
under top-k against the top-k target distribution; emitted-token law equals p over 10^6
seeded trials (Appendix A.1); with lenience the acceptance frequency equals
sum min(p / l, q) (Appendix A.5), the emitted law equals min(q, p / l) +
(1 - alpha_l) * max(0, p - q) / (1 - beta) and never exceeds p / l, and
l = 1 is the strict algorithm; acceptance frequency equals sum min(p, q)
(Theorem 3.5); rejected-branch law equals max(0, p - q) / (1 - beta);
p = q always accepts, disjoint supports never accept (Corollary 3.4); exact
measures of every outcome on an (r, u) grid for vocabularies <= 8; gamma = 0
reduces to a textbook inverse-CDF draw from p; T = 0 reduces to greedy.
"""

from dataclasses import dataclass, field

import numpy as np


def top_k_floor(logits, top_k):
    """The k-th largest logit of a row (-inf when top-k is off: k = 0 or k >= V)."""
    z = np.asarray(logits, dtype=np.float64)
    if top_k <= 0 or top_k >= z.shape[0]:
        return -np.inf
    return float(np.sort(z)[z.shape[0] - top_k])


def keep_top_k(logits, top_k):
    """The row with every logit below its k-th largest replaced by -inf."""
    z = np.asarray(logits, dtype=np.float64)
    return np.where(z >= top_k_floor(z, top_k), z, -np.inf)


def nucleus_floor(logits, temperature, top_k=0, top_p=1.0):
    """(floor, margin): the smallest logit that top-k followed by the nucleus keeps.

    margin: distance, as a fraction of the total mass, between top_p and the
    nearer of the two cumulative masses around the cut (inf when the nucleus is
    off); a caller comparing with lower-precision arithmetic can tell from it
    whether the cut was a close call.
    """
    z = keep_top_k(logits, top_k)
    floor = top_k_floor(logits, top_k)
    if not 0.0 < top_p < 1.0 or temperature == 0:
        return floor, float("inf")
    w = np.exp((z - z.max()) / float(temperature))
    order = np.argsort(-z, kind="stable")  # decreasing probability
    running = np.cumsum(w[order])
    goal = top_p * running[-1]
    taken = int(np.searchsorted(running, goal, side="left")) + 1  # first prefix whose mass reaches the goal
    taken = min(taken, z.shape[0])
    margin = abs(running[taken - 1] - goal)
    if taken > 1:
        margin = min(margin, abs(running[taken - 2] - goal))
    return float(z[order[taken - 1]]), float(margin / running[-1])


def keep_nucleus(logits, temperature, top_k=0, top_p=1.0):
    """The row with everything outside top-k and the nucleus replaced by -inf."""
    z = np.asarray(logits, dtype=np.float64)
    return np.where(z >= nucleus_floor(z, temperature, top_k, top_p)[0], z, -np.inf)


def standardise(logits, temperature, top_k=0, top_p=1.0):
    """Section 2.2: logits -> the adjusted distribution that is sampled from.

    T > 0: softmax(logits / T) over the logits that top-k and then the nucleus
    keep (all of them for k = 0, top_p = 1), with the maximum subtracted first.
    T = 0: one-hot at the maximum (lowest index on ties).
    """
    z = np.asarray(logits, dtype=np.float64)
    if temperature == 0:
        out = np.zeros_like(z)
        out[int(np.argmax(z))] = 1.0  # numpy's argmax returns the first maximum
        return out
    z = keep_nucleus(z, temperature, top_k, top_p) / float(temperature)
    z = z - z.max()
    e = np.exp(z)
    return e / e.sum()


def inverse_cdf(weights, u):
    """Draw an index from unnormalised `weights` with the uniform `u`.

    Returns (k, margin): k is the smallest index whose running sum exceeds
    u * W; margin is the distance from u * W to the nearer of the two running
    sums that bracket it, divided by W (how close the draw was to picking a
    neighbour instead).
    """
    w = np.asarray(weights, dtype=np.float64)
    running = np.cumsum(w)  # sequential fp64 accumulation in index order
    total = running[-1]
    target = u * total
    k = int(np.searchsorted(running, target, side="right"))  # first running sum > target
    if k >= w.shape[0]:
        positive = np.nonzero(w > 0.0)[0]
        return (int(positive[-1]) if positive.size else w.shape[0] - 1), 0.0
    prev = running[k - 1] if k > 0 else 0.0
    margin = min(target - prev, running[k] - target) / total
    return k, float(margin)


def speculative_sampling(p, q, x, r, u, lenience=1.0):
    """Section 2.3 for one token: x was drawn from q; returns (accepted, token).

    Keeps x unless r > p(x) / (l q(x)) (l = 1: the paper's algorithm; l < 1:
    Appendix A.5); otherwise draws from norm(max(0, p - q)) with the uniform u.
    """
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    if not (r * lenience * q[x] > p[x]):
        return True, int(x)
    residual = np.maximum(0.0, p - q)
    if not residual.sum() > 0.0:
        residual = p
    k, _ = inverse_cdf(residual, u)
    return False, k


@dataclass
class VerifyResult:
    """Outcome of the accept/adjust/draw part of Algorithm 1 for one sequence."""

    n_accepted: int
    next_token: int
    accept_margin: float  # min |r_i - p_i(x_i)/q_i(x_i)| over the tests evaluated
    cdf_margin: float  # see inverse_cdf
    top2_gap: float  # smallest gap between the two largest target logits, rows used
    fallback: bool  # the residual vanished and p_{n+1} was used unmodified
    betas: list = field(default_factory=list)  # sum min(p_i, q_i), tests evaluated


def lenient_greedy_accepts(target_row, x, lenience):
    """Appendix A.5 at T = 0: (accepted, margin).  l = 1: x must be the lowest-index
    maximum; l < 1: logit(x) >= max logit + ln l (p(x) >= l max p before standardising)."""
    if lenience >= 1.0:
        return int(x) == int(np.argmax(target_row)), float("inf")
    slack = float(target_row[int(x)] - target_row.max() - np.log(lenience))
    return slack >= 0.0, abs(slack)


def verify_step(target_logits, draft_logits, draft_tokens, uniforms, temperature, lenience=1.0, top_k=0, top_p=1.0):
    """Algorithm 1 from the accept tests to the returned token (everything after the
    target's parallel pass).

    target_logits [gamma+1, V]: row i-1 gives p_i (i = 1..gamma+1).
    draft_logits  [gamma, V]:   row i-1 gives q_i, from which x_i was drawn.
    draft_tokens  [gamma]:      x_1..x_gamma.
    uniforms      [gamma+1]:    r_1..r_gamma, then the uniform for t ~ p'.
    """
    tl = np.asarray(target_logits, dtype=np.float64)
    ql = np.asarray(draft_logits, dtype=np.float64)
    gamma = tl.shape[0] - 1
    assert ql.shape[0] == gamma and len(draft_tokens) == gamma
    assert len(uniforms) == gamma + 1

    p = [standardise(tl[i], temperature, top_k, top_p) for i in range(gamma + 1)]
    q = [standardise(ql[i], temperature, top_k, top_p) for i in range(gamma)]

    accept_margin = float("inf")
    top2_gap = float("inf")
    betas = []
    n = gamma
    for i in range(gamma):
        x = int(draft_tokens[i])
        r = float(uniforms[i])
        betas.append(float(np.minimum(p[i], q[i]).sum()))
        top2_gap = min(top2_gap, _top2_gap(tl[i]))
        if temperature == 0 and lenience < 1.0:
            accepted, slack = lenient_greedy_accepts(tl[i], x, lenience)
            accept_margin = min(accept_margin, slack)
            if not accepted:
                n = i
                break
            continue
        if temperature == 0:
            # Both standardised distributions are one-hot (Section 2.2).  A guess drawn from q_i is
            # q_i's maximum, and the accept test then passes exactly when it is p_i's maximum too.
            # A guess that is NOT q_i's maximum cannot come from x ~ q_i: the printed test reads
            # r > p(x) / 0 there and decides nothing.  Reading: at T = 0 a guess is accepted iff it
            # is the target's (lowest-index) maximum, whatever the draft's logits say.
            if p[i][x] != 1.0:
                n = i
                break
            continue
        if q[i][x] > 0.0:
            accept_margin = min(accept_margin, abs(r - p[i][x] / (lenience * q[i][x])))
        if r * lenience * q[i][x] > p[i][x]:
            n = i
            break

    adjusted = p[n]
    fallback = False
    if n < gamma:
        adjusted = np.maximum(0.0, p[n] - q[n])
        if not adjusted.sum() > 0.0:
            adjusted = p[n]
            fallback = True
    else:
        top2_gap = min(top2_gap, _top2_gap(tl[gamma]))
    t, cdf_margin = inverse_cdf(adjusted, float(uniforms[gamma]))
    return VerifyResult(n, t, accept_margin, cdf_margin, top2_gap, fallback, betas)


def verify_batch(target_logits, draft_logits, draft_tokens, uniforms, temperature, lenience=1.0, top_k=0, top_p=1.0):
    """`verify_step` for every sequence of a batch: [B, ...] inputs -> list."""
    return [
        verify_step(target_logits[b], draft_logits[b], draft_tokens[b], uniforms[b], temperature, lenience, top_k, top_p)
        for b in range(len(target_logits))
    ]


def sample_token(logits, u, temperature, top_k=0, top_p=1.0):
    """A plain draw from the standardised distribution: (token, cdf margin).

    This is how the draft model draws x_i ~ q_i and how target-only decoding
    draws t ~ p.  The weights are left unnormalised, exp((l - max) / T), which
    the inverse-CDF rule allows.
    """
    z = np.asarray(logits, dtype=np.float64)
    if temperature == 0:
        return int(np.argmax(z)), float("inf")
    w = np.exp((keep_nucleus(z, temperature, top_k, top_p) - z.max()) / float(temperature))
    return inverse_cdf(w, u)


def sample_trials(logits, uniforms, temperature, top_k=0, top_p=1.0):
    """`sample_token` for many uniforms that share one row of logits -> [N]."""
    z = np.asarray(logits, dtype=np.float64)
    us = np.asarray(uniforms, dtype=np.float64)
    if temperature == 0:
        return np.full(us.shape[0], int(np.argmax(z)), dtype=np.int64)
    w = np.exp((keep_nucleus(z, temperature, top_k, top_p) - z.max()) / float(temperature))
    running = np.cumsum(w)
    k = np.searchsorted(running, us * running[-1], side="right")
    positive = np.nonzero(w > 0.0)[0]
    return np.where(k >= w.shape[0], positive[-1], k).astype(np.int64)


def verify_trials(target_logits, draft_logits, draft_tokens, uniforms, temperature, lenience=1.0, top_k=0, top_p=1.0):
    """Many independent trials of `verify_step` that share one set of logits.

    target_logits [gamma+1, V] and draft_logits [gamma, V] are fixed;
    draft_tokens [N, gamma] and uniforms [N, gamma+1] vary per trial.  Returns
    (n_accepted [N], next_token [N]).  Same rules as `verify_step`, evaluated
    for all trials at once (the statistical pins need 10^6 of them); the tests
    check it against `verify_step` trial by trial on a subset.
    """
    tl = np.asarray(target_logits, dtype=np.float64)
    ql = np.asarray(draft_logits, dtype=np.float64)
    xs = np.asarray(draft_tokens)
    us = np.asarray(uniforms, dtype=np.float64)
    gamma = tl.shape[0] - 1
    trials = us.shape[0]
    p = np.stack([standardise(tl[i], temperature, top_k, top_p) for i in range(gamma + 1)])
    q = np.stack([standardise(ql[i], temperature, top_k, top_p) for i in range(gamma)]) if gamma else np.zeros((0, tl.shape[1]))

    n = np.full(trials, gamma, dtype=np.int64)
    undecided = np.ones(trials, dtype=bool)
    for i in range(gamma):
        x = xs[:, i]
        if temperature == 0 and lenience < 1.0:
            rejected = ~(tl[i][x] - tl[i].max() - np.log(lenience) >= 0.0)
        elif temperature == 0:
            rejected = p[i][x] != 1.0  # (see verify_step: accepted iff the guess is the target's maximum)
        else:
            rejected = us[:, i] * lenience * q[i][x] > p[i][x]
        first = undecided & rejected
        n[first] = i
        undecided &= ~rejected

    tokens = np.empty(trials, dtype=np.int64)
    for row in range(gamma + 1):
        sel = np.nonzero(n == row)[0]
        if sel.size == 0:
            continue
        adjusted = p[row]
        if row < gamma:
            adjusted = np.maximum(0.0, p[row] - q[row])
            if not adjusted.sum() > 0.0:
                adjusted = p[row]
        running = np.cumsum(adjusted)
        k = np.searchsorted(running, us[sel, gamma] * running[-1], side="right")
        positive = np.nonzero(adjusted > 0.0)[0]
        k = np.where(k >= adjusted.shape[0], positive[-1], k)
        tokens[sel] = k
    return n, tokens


def _top2_gap(row):
    if row.shape[0] < 2:
        return float("inf")
    top = np.partition(row, -2)[-2:]
    return float(top[1] - top[0])
