"""Closed forms of the paper's analysis section, written out as printed.

Test infrastructure (see the package docstring).

Pins (tests/test_oracle_analysis.py, values in tests/golden/): every row of
Table 1 (operations and speed at c = c_hat = 0) to the printed digits; the
"Exp" column of Table 4 within print rounding; the bigram example of
Section 3.6 (alpha = 0.2, gamma = 3, c = 0 gives 1.25X); Corollary 3.9 as the
gamma = 1 case of Theorem 3.8; Lemma 3.3 against Definition 3.2 on random
distributions.
"""

import numpy as np


def d_lk(p, q):
    """Definition 3.2: sum |p - M| with M = (p + q) / 2."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    m = (p + q) / 2.0
    return float(np.abs(p - m).sum())


def beta(p, q):
    """Theorem 3.5: acceptance probability of x ~ q, sum_x min(p(x), q(x))."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    return float(np.minimum(p, q).sum())


def beta_lenient(p, q, lenience):
    """Appendix A.5: acceptance with q scaled by l, sum_x min(p(x) / l, q(x))."""
    p = np.asarray(p, dtype=np.float64)
    q = np.asarray(q, dtype=np.float64)
    return float(np.minimum(p / lenience, q).sum())


def expected_tokens(alpha, gamma):
    """Eq. 1: (1 - alpha^(gamma+1)) / (1 - alpha), a capped geometric mean."""
    if alpha == 1.0:
        return float(gamma + 1)
    return (1.0 - alpha ** (gamma + 1)) / (1.0 - alpha)


def walltime_improvement(alpha, gamma, c):
    """Theorem 3.8: (1 - alpha^(gamma+1)) / ((1 - alpha) (gamma c + 1))."""
    return expected_tokens(alpha, gamma) / (gamma * c + 1.0)


def walltime_improvement_lower_bound(alpha, c):
    """Corollary 3.9: (1 + alpha) / (1 + c), Theorem 3.8 at gamma = 1."""
    return (1.0 + alpha) / (1.0 + c)


def ops_increase(alpha, gamma, c_hat):
    """Theorem 3.11: (1 - alpha)(gamma c_hat + gamma + 1) / (1 - alpha^(gamma+1))."""
    return (gamma * c_hat + gamma + 1.0) / expected_tokens(alpha, gamma)


def best_gamma(alpha, c, gamma_max=64):
    """Section 3.5: the integer gamma >= 1 that maximises Theorem 3.8."""
    values = [walltime_improvement(alpha, g, c) for g in range(1, gamma_max + 1)]
    return int(np.argmax(values)) + 1


def generalised_speedup(tokens_per_iteration, t_target_one, t_target_rows, t_draft, gamma, t_sample=0.0):
    """Theorem 3.8's proof with its two idealisations removed.

    The proof charges an iteration T c gamma + T and assumes that gamma + 1
    parallel rows cost the same as one.  With measured times this becomes
    tokens * t_p(1) / (gamma t_q + t_p(gamma + 1) + t_sample).
    """
    return tokens_per_iteration * t_target_one / (gamma * t_draft + t_target_rows + t_sample)
