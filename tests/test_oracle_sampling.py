"""Pins for oracle.sampling: what Appendix A.1, Theorem 3.5 and Corollary 3.4 fix."""
import numpy as np
import pytest
from scipy import stats

from oracle import analysis, philox, sampling
from paper_2211_17192_b200 import workloads

TRIALS = 1_000_000
VOCAB = 64


def _chi_square_p(counts, probs):
    """Chi-square goodness of fit; bins with expected count < 5 are merged into one."""
    expected = probs * counts.sum()
    small = expected < 5
    if small.any():
        counts = np.append(counts[~small], counts[small].sum())
        expected = np.append(expected[~small], expected[small].sum())
        if expected[-1] == 0:
            assert counts[-1] == 0
            counts, expected = counts[:-1], expected[:-1]
    return stats.chisquare(counts, expected).pvalue


def _fixed_pair(noise, seed=11):
    t, d = workloads.make_sampler_logits(seed, 1, 1, VOCAB, noise)
    return t[0].astype(np.float64), d[0].astype(np.float64)  # [2, V], [1, V]


@pytest.mark.parametrize("noise", [0.5, 1.0, 2.0])
def test_emitted_token_follows_p_and_acceptance_equals_sum_min(noise):
    tl, ql = _fixed_pair(noise)
    p = sampling.standardise(tl[0], 1.0)
    q = sampling.standardise(ql[0], 1.0)
    idx = np.arange(TRIALS)
    x = sampling.sample_trials(ql[0], philox.uniforms_vec(5, idx, 0, philox.PURPOSE_DRAFT), 1.0)
    r = philox.uniforms_vec(5, idx, 0, philox.PURPOSE_ACCEPT)
    u = philox.uniforms_vec(5, idx, 0, philox.PURPOSE_FINAL)
    n, t = sampling.verify_trials(tl, ql, x[:, None], np.stack([r, u], axis=1), 1.0)

    # the draft's own draws follow q
    assert _chi_square_p(np.bincount(x, minlength=VOCAB), q) > 1e-3
    # Appendix A.1: the first emitted token (x if accepted, else t) follows p
    first = np.where(n == 1, x, t)
    assert _chi_square_p(np.bincount(first, minlength=VOCAB), p) > 1e-3
    # Theorem 3.5: acceptance frequency = sum min(p, q)
    beta = analysis.beta(p, q)
    assert abs((n == 1).mean() - beta) < 4 * np.sqrt(beta * (1 - beta) / TRIALS)
    # Appendix A.1: after a rejection the token follows max(0, p - q) / (1 - beta)
    residual = np.maximum(0, p - q)
    assert residual.sum() == pytest.approx(1 - beta, abs=1e-12)
    assert _chi_square_p(np.bincount(t[n == 0], minlength=VOCAB), residual / residual.sum()) > 1e-3
    # when all guesses are accepted the bonus token follows p_{gamma+1}
    p2 = sampling.standardise(tl[1], 1.0)
    assert _chi_square_p(np.bincount(t[n == 1], minlength=VOCAB), p2) > 1e-3


def test_tokens_per_iteration_match_eq_1():
    gamma = 4
    tl1, ql1 = _fixed_pair(1.0, seed=12)
    tl = np.repeat(tl1[:1], gamma + 1, axis=0)  # the same p at every position
    ql = np.repeat(ql1[:1], gamma, axis=0)  # the same q at every position
    alpha = analysis.beta(sampling.standardise(tl[0], 1.0), sampling.standardise(ql[0], 1.0))
    trials = 400_000
    idx = np.arange(trials)
    xs = np.stack([sampling.sample_trials(ql[0], philox.uniforms_vec(9, idx * gamma + i, 0, 0), 1.0)
                   for i in range(gamma)], axis=1)
    us = np.stack([philox.uniforms_vec(9, idx * (gamma + 1) + i, 1, 1) for i in range(gamma + 1)], axis=1)
    n, _ = sampling.verify_trials(tl, ql, xs, us, 1.0)
    tokens = n + 1
    assert tokens.min() >= 1 and tokens.max() <= gamma + 1
    assert abs(tokens.mean() - analysis.expected_tokens(alpha, gamma)) < 4 * tokens.std() / np.sqrt(trials)
    # the capped geometric law itself
    law = np.array([alpha**k * (1 - alpha) for k in range(gamma)] + [alpha**gamma])
    assert _chi_square_p(np.bincount(n, minlength=gamma + 1), law) > 1e-3


def test_vectorised_trials_equal_the_scalar_step():
    gamma = 3
    t, d = workloads.make_sampler_logits(21, 1, gamma, VOCAB, 1.0)
    tl, ql = t[0], d[0]
    trials = 3000
    idx = np.arange(trials)
    xs = np.stack([sampling.sample_trials(ql[i], philox.uniforms_vec(3, idx, i, 0), 1.0) for i in range(gamma)], axis=1)
    us = np.stack([philox.uniforms_vec(3, idx, i, 1) for i in range(gamma + 1)], axis=1)
    for temperature in (1.0, 0.7, 0.0):
        n, tok = sampling.verify_trials(tl, ql, xs, us, temperature)
        for k in range(trials):
            res = sampling.verify_step(tl, ql, xs[k], us[k], temperature)
            assert (res.n_accepted, res.next_token) == (n[k], tok[k])


def test_identical_distributions_always_accept():
    t, _ = workloads.make_sampler_logits(31, 4, 3, 50, 1.0)
    us = workloads.make_uniform_grid(31, (4, 4))
    xs = np.array([[sampling.sample_token(t[b, i], 0.3 + 0.1 * i, 1.0)[0] for i in range(3)] for b in range(4)])
    for b in range(4):
        res = sampling.verify_step(t[b], t[b, :3], xs[b], us[b], 1.0)
        assert res.n_accepted == 3
        assert res.next_token == sampling.sample_token(t[b, 3], us[b, 3], 1.0)[0]
        assert all(beta == pytest.approx(1.0, abs=1e-12) for beta in res.betas)


def test_disjoint_supports_never_accept_and_resample_from_p():
    V = 10
    big = 800.0  # exp(-800) underflows to exactly 0 in fp64
    tl = np.full((2, V), -big)
    ql = np.full((1, V), -big)
    tl[:, :5] = np.linspace(0, 1, 5)
    ql[:, 5:] = np.linspace(0, 1, 5)
    p = sampling.standardise(tl[0], 1.0)
    for u in (0.01, 0.37, 0.99):
        res = sampling.verify_step(tl, ql, [7], [1 / 2**24, u], 1.0)  # smallest possible r still rejects
        assert res.n_accepted == 0 and res.betas == [0.0]
        assert res.next_token == sampling.inverse_cdf(p, u)[0] and res.next_token < 5


def test_uniform_draft_acceptance():
    V = 32
    tl, _ = _fixed_pair(1.0, seed=5)
    p = sampling.standardise(tl[0, :V], 1.0)
    res = sampling.verify_step(tl[:, :V], np.zeros((1, V)), [3], [0.5, 0.5], 1.0)
    assert res.betas[0] == pytest.approx(np.minimum(p, 1.0 / V).sum(), abs=1e-14)


def test_gamma_zero_is_a_plain_inverse_cdf_draw():
    w = np.array([1.0, 2.0, 0.0, 1.0])
    logits = np.log(np.maximum(w, 1e-300))
    logits[2] = -1e4
    # boundaries of the CDF at 0.25, 0.75, 0.75, 1: smallest k with running sum > u
    for u, expect in [(0.1, 0), (0.2499, 0), (0.25, 1), (0.5, 1), (0.7499, 1), (0.75, 3), (0.99, 3)]:
        assert sampling.inverse_cdf(w, u)[0] == expect
        res = sampling.verify_step(logits[None, :], np.zeros((0, 4)), [], [u], 1.0)
        assert (res.n_accepted, res.next_token) == (0, expect)
    # against numpy's own inverse-CDF categorical draw on the same uniforms
    rng = np.random.default_rng(0)
    weights = rng.random(17)
    us = rng.random(1000)
    ref = np.searchsorted(np.cumsum(weights) / weights.sum(), us, side="right")
    got = [sampling.inverse_cdf(weights, u)[0] for u in us]
    assert np.array_equal(ref, got)


def test_inverse_cdf_margin_and_last_positive_fallback():
    k, margin = sampling.inverse_cdf([1.0, 1.0, 2.0], 0.3)
    assert k == 1 and margin == pytest.approx(0.05)
    assert sampling.inverse_cdf([0.5, 0.5, 0.0], 1.0)[0] == 1  # u = 1 is off the grid: last positive weight


def test_temperature_zero_is_greedy():
    gamma = 4
    t, d = workloads.make_sampler_logits(41, 6, gamma, 100, 1.0)
    for b in range(6):
        xs = [int(np.argmax(d[b, i])) for i in range(gamma)]  # the draft's own greedy draws
        res = sampling.verify_step(t[b], d[b], xs, [0.9] * (gamma + 1), 0.0)
        greedy = [int(np.argmax(t[b, i])) for i in range(gamma + 1)]
        n = 0
        while n < gamma and xs[n] == greedy[n]:
            n += 1
        assert (res.n_accepted, res.next_token) == (n, greedy[n])
    # ties go to the lowest index
    assert sampling.standardise([1.0, 3.0, 3.0, 0.0], 0.0).tolist() == [0, 1, 0, 0]
    assert sampling.sample_token([1.0, 3.0, 3.0], 0.5, 0.0)[0] == 1


def test_temperature_scales_logits():
    logits = np.array([0.3, -1.2, 2.0, 0.0])
    for T in (0.5, 2.0):
        assert np.allclose(sampling.standardise(logits, T), sampling.standardise(logits / T, 1.0), atol=1e-15)
    p = sampling.standardise(logits, 1.0)
    assert p.sum() == pytest.approx(1.0) and np.allclose(p, np.exp(logits) / np.exp(logits).sum())


def _threshold(fn, lo=0.0, hi=1.0, iters=60):
    """Largest v in [lo, hi] with fn(v) true, for fn true on [lo, v] and false above."""
    if fn(hi):
        return hi
    if not fn(lo):
        return lo
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if fn(mid):
            lo = mid
        else:
            hi = mid
    return lo


@pytest.mark.parametrize("V,gamma,seed", [(3, 1, 0), (5, 2, 1), (8, 2, 2), (4, 3, 3)])
def test_exact_outcome_measures_on_small_vocabularies(V, gamma, seed):
    """Brute force: drive verify_step over every drafted sequence and locate, by
    bisection on each uniform, the exact measure of every outcome.  The law of
    (n, t) must be prod beta-terms times the adjusted distribution, and the law
    of the first emitted token must be p_1 (Appendix A.1)."""
    rng = np.random.default_rng(seed)
    tl = rng.normal(0, 1.5, (gamma + 1, V))
    ql = rng.normal(0, 1.5, (gamma, V))
    p = [sampling.standardise(r, 1.0) for r in tl]
    q = [sampling.standardise(r, 1.0) for r in ql]
    first_token_law = np.zeros(V)
    total = 0.0
    for xs in np.ndindex(*([V] * gamma)):
        prob_x = np.prod([q[i][xs[i]] for i in range(gamma)])
        # accept thresholds tau_i: test i passes iff r_i <= tau_i (others forced to pass)
        taus = []
        for i in range(gamma):
            def passes(r, i=i):
                us = [0.0] * gamma + [0.5]
                us[i] = r
                return sampling.verify_step(tl, ql, xs, us, 1.0).n_accepted > i
            taus.append(_threshold(passes))
            assert taus[-1] == pytest.approx(min(1.0, p[i][xs[i]] / q[i][xs[i]]), abs=1e-12)
        for n in range(gamma + 1):
            prob_n = np.prod(taus[:n]) * ((1 - taus[n]) if n < gamma else 1.0)
            if prob_n == 0:
                continue
            us = [0.0] * n + [1.0] * (gamma - n)
            # measure of u that yields each token: breakpoints of a step function in u
            edges = [0.0]
            for k in range(V - 1):
                edges.append(_threshold(
                    lambda u, k=k: sampling.verify_step(tl, ql, xs, us + [u], 1.0).next_token <= k, lo=edges[-1]))
            edges.append(1.0)
            law_t = np.diff(edges)
            expect = p[n] if n == gamma else np.maximum(0, p[n] - q[n]) / np.maximum(0, p[n] - q[n]).sum()
            assert np.allclose(law_t, expect, atol=1e-10)
            total += prob_x * prob_n
            if n >= 1:
                first_token_law[xs[0]] += prob_x * prob_n
            else:
                first_token_law += prob_x * prob_n * law_t
    assert total == pytest.approx(1.0, abs=1e-10)
    assert np.allclose(first_token_law, p[0], atol=1e-10)


def test_speculative_sampling_single_token_rule():
    p = np.array([0.5, 0.3, 0.2])
    q = np.array([0.2, 0.2, 0.6])
    # q(x) <= p(x): always kept
    assert sampling.speculative_sampling(p, q, 0, 0.999, 0.5) == (True, 0)
    # q(x) > p(x): kept iff r <= p/q = 1/3
    assert sampling.speculative_sampling(p, q, 2, 0.33, 0.5) == (True, 2)
    # rejected: residual = [0.3, 0.1, 0] / 0.4 -> boundary at 0.75
    assert sampling.speculative_sampling(p, q, 2, 0.34, 0.74) == (False, 0)
    assert sampling.speculative_sampling(p, q, 2, 0.34, 0.76) == (False, 1)


@pytest.mark.parametrize("lenience", [0.5, 0.3, 0.1])
def test_lenience_acceptance_and_emitted_law(lenience):
    """Appendix A.5: alpha_l = sum min(p / l, q); no token is emitted with probability above p / l."""
    tl, ql = _fixed_pair(2.0)
    p = sampling.standardise(tl[0], 1.0)
    q = sampling.standardise(ql[0], 1.0)
    idx = np.arange(TRIALS)
    x = sampling.sample_trials(ql[0], philox.uniforms_vec(6, idx, 0, philox.PURPOSE_DRAFT), 1.0)
    r = philox.uniforms_vec(6, idx, 0, philox.PURPOSE_ACCEPT)
    u = philox.uniforms_vec(6, idx, 0, philox.PURPOSE_FINAL)
    n, t = sampling.verify_trials(tl, ql, x[:, None], np.stack([r, u], axis=1), 1.0, lenience)
    alpha_l = analysis.beta_lenient(p, q, lenience)
    assert alpha_l > analysis.beta(p, q)
    assert abs((n == 1).mean() - alpha_l) <= 4 * np.sqrt(alpha_l * (1 - alpha_l) / TRIALS)
    # exact law of the first emitted token under the reading taken for the adjusted distribution
    residual = np.maximum(0, p - q)
    law = np.minimum(q, p / lenience) + (1 - alpha_l) * residual / residual.sum()
    assert law.sum() == pytest.approx(1.0, abs=1e-12)
    assert np.all(law <= p / lenience + 1e-15)
    first = np.where(n == 1, x, t)
    assert _chi_square_p(np.bincount(first, minlength=VOCAB), law) > 1e-3
    # and it is no longer p
    assert _chi_square_p(np.bincount(first, minlength=VOCAB), p) < 1e-6


def test_lenience_one_is_the_strict_algorithm_and_scalar_equals_vectorised():
    tl, ql = _fixed_pair(2.0)
    idx = np.arange(2000)
    x = sampling.sample_trials(ql[0], philox.uniforms_vec(7, idx, 0, philox.PURPOSE_DRAFT), 1.0)
    us = np.stack([philox.uniforms_vec(7, idx, 0, philox.PURPOSE_ACCEPT), philox.uniforms_vec(7, idx, 0, philox.PURPOSE_FINAL)], axis=1)
    strict = sampling.verify_trials(tl, ql, x[:, None], us, 1.0)
    same = sampling.verify_trials(tl, ql, x[:, None], us, 1.0, 1.0)
    assert np.array_equal(strict[0], same[0]) and np.array_equal(strict[1], same[1])
    for temperature in (1.0, 0.0):
        n, t = sampling.verify_trials(tl, ql, x[:, None], us, temperature, 0.3)
        for k in range(0, 2000, 37):
            ref = sampling.verify_step(tl, ql, x[k : k + 1], us[k], temperature, 0.3)
            assert (ref.n_accepted, ref.next_token) == (n[k], t[k])


def test_lenience_at_temperature_zero():
    """Accept x iff p(x) >= l * max p with p the T = 1 softmax of the target row; a rejected slot gets argmax p."""
    rng = np.random.default_rng(3)
    tl = rng.standard_normal((2, 16)) * 2.0
    ql = rng.standard_normal((1, 16))
    p = sampling.standardise(tl[0], 1.0)
    best = int(np.argmax(tl[0]))
    for lenience in (0.5, 0.3, 0.1, 1e-9):
        for x in range(16):
            res = sampling.verify_step(tl, ql, [x], [0.5, 0.5], 0.0, lenience)
            assert (res.n_accepted == 1) == bool(p[x] >= lenience * p.max() * (1 - 1e-12))
            if res.n_accepted == 0:
                assert res.next_token == best
            else:
                assert res.next_token == int(np.argmax(tl[1]))
    # strict rule at l = 1: the draft's own argmax x is accepted only if it is the target's argmax
    accepted = []
    for x in range(16):
        draft = np.zeros((1, 16))
        draft[0, x] = 5.0
        accepted.append(sampling.verify_step(tl, draft, [x], [0.5, 0.5], 0.0, 1.0).n_accepted)
    assert accepted == [1 if x == best else 0 for x in range(16)]


def _top_k_by_repeated_argmax(row, k):
    """Indices of a top-k set found by taking the maximum k times (no sort, no threshold)."""
    left = np.array(row, dtype=np.float64)
    chosen = []
    for _ in range(k):
        i = int(np.argmax(left))
        chosen.append(i)
        left[i] = -np.inf
    return chosen


@pytest.mark.parametrize("k", [1, 2, 7, 63])
def test_top_k_support_and_ratios(k):
    tl, _ = _fixed_pair(1.0)
    row = tl[0]  # drawn from a continuous law: no ties
    for T in (1.0, 0.6):
        p_all = sampling.standardise(row, T)
        p_k = sampling.standardise(row, T, top_k=k)
        chosen = _top_k_by_repeated_argmax(row, k)
        assert sorted(np.nonzero(p_k)[0].tolist()) == sorted(chosen)
        assert p_k.sum() == pytest.approx(1.0, abs=1e-12)
        # inside the support the ratios of the plain softmax survive
        assert np.allclose(p_k[chosen] / p_k[chosen[0]], p_all[chosen] / p_all[chosen[0]], rtol=1e-12)
    assert sampling.top_k_floor(row, k) == row[chosen[-1]]


def test_top_k_edge_cases():
    tl, _ = _fixed_pair(1.0)
    row = tl[0]
    plain = sampling.standardise(row, 0.8)
    for k in (0, VOCAB, VOCAB + 5):
        assert np.array_equal(sampling.standardise(row, 0.8, top_k=k), plain)
    one = sampling.standardise(row, 0.8, top_k=1)
    assert np.array_equal(one, sampling.standardise(row, 0.0))
    # entries tied with the k-th largest all stay
    tied = np.array([0.0, 2.0, 1.0, 1.0, -1.0, 1.0])
    assert np.nonzero(sampling.standardise(tied, 1.0, top_k=2))[0].tolist() == [1, 2, 3, 5]
    assert np.nonzero(sampling.standardise(tied, 1.0, top_k=1))[0].tolist() == [1]
    # T = 0 ignores k
    assert np.array_equal(sampling.standardise(tied, 0.0, top_k=3), sampling.standardise(tied, 0.0))
    # a plain draw never leaves the support
    us = philox.uniforms_vec(9, np.arange(20000), 0, philox.PURPOSE_DRAFT)
    drawn = sampling.sample_trials(row, us, 1.0, top_k=5)
    assert set(drawn.tolist()) <= set(_top_k_by_repeated_argmax(row, 5))
    assert [sampling.sample_token(row, float(u), 1.0, top_k=5)[0] for u in us[:200]] == drawn[:200].tolist()


@pytest.mark.parametrize("k", [3, 12])
def test_emitted_law_under_top_k_is_the_top_k_target_distribution(k):
    """Section 2.2 with Appendix A.1: both models standardised the same way, output law = adjusted p."""
    trials = 400_000
    tl, ql = _fixed_pair(1.0)
    p = sampling.standardise(tl[0], 1.0, top_k=k)
    q = sampling.standardise(ql[0], 1.0, top_k=k)
    idx = np.arange(trials)
    x = sampling.sample_trials(ql[0], philox.uniforms_vec(6, idx, 0, philox.PURPOSE_DRAFT), 1.0, top_k=k)
    r = philox.uniforms_vec(6, idx, 0, philox.PURPOSE_ACCEPT)
    u = philox.uniforms_vec(6, idx, 0, philox.PURPOSE_FINAL)
    n, t = sampling.verify_trials(tl, ql, x[:, None], np.stack([r, u], axis=1), 1.0, top_k=k)
    assert _chi_square_p(np.bincount(x, minlength=VOCAB), q) > 1e-3
    first = np.where(n == 1, x, t)
    assert np.all(p[first] > 0)
    assert _chi_square_p(np.bincount(first, minlength=VOCAB), p) > 1e-3
    beta = analysis.beta(p, q)
    assert abs((n == 1).mean() - beta) < 4 * np.sqrt(beta * (1 - beta) / trials)
    # the vectorised trials are the scalar step
    for i in range(300):
        res = sampling.verify_step(tl, ql, x[i : i + 1], [r[i], u[i]], 1.0, top_k=k)
        assert (res.n_accepted, res.next_token) == (n[i], t[i])


def _nucleus_by_repeated_argmax(probs, top_p):
    """Indices taken by picking the most probable remaining token until the mass reaches top_p."""
    left = np.array(probs, dtype=np.float64)
    chosen, mass = [], 0.0
    while mass < top_p * probs.sum() and len(chosen) < len(probs):
        i = int(np.argmax(left))
        chosen.append(i)
        mass += probs[i]
        left[i] = -1.0
    return chosen


def test_nucleus_on_a_hand_computed_example():
    probs = np.array([0.05, 0.5, 0.15, 0.3])
    logits = np.log(probs)
    for top_p, kept in [(0.4, [1]), (0.6, [1, 3]), (0.75, [1, 3]), (0.85, [1, 2, 3]), (0.97, [0, 1, 2, 3])]:
        got = sampling.standardise(logits, 1.0, top_p=top_p)
        assert np.nonzero(got)[0].tolist() == kept
        assert np.allclose(got[kept], probs[kept] / probs[kept].sum(), rtol=1e-12)
    # the margin reports how close top_p came to a cumulative mass (0.5, 0.8, 0.95, 1.0)
    assert sampling.nucleus_floor(logits, 1.0, 0, 0.6)[1] == pytest.approx(0.1, abs=1e-12)
    assert sampling.nucleus_floor(logits, 1.0, 0, 0.94)[1] == pytest.approx(0.01, abs=1e-12)
    # temperature enters before the cut: at T = 0.5 the probabilities are proportional to p^2
    sharper = probs**2 / (probs**2).sum()  # 0.0068 0.68 0.061 0.245
    assert np.nonzero(sampling.standardise(logits, 0.5, top_p=0.7))[0].tolist() == [1, 3]
    assert np.allclose(sampling.standardise(logits, 0.5, top_p=0.7)[[1, 3]], sharper[[1, 3]] / sharper[[1, 3]].sum())


@pytest.mark.parametrize("top_p", [0.05, 0.5, 0.9, 0.999])
@pytest.mark.parametrize("temperature", [1.0, 0.6])
def test_nucleus_equals_the_greedy_restatement(top_p, temperature):
    tl, _ = _fixed_pair(2.0)
    row = tl[0]
    plain = sampling.standardise(row, temperature)
    got = sampling.standardise(row, temperature, top_p=top_p)
    chosen = _nucleus_by_repeated_argmax(plain, top_p)
    assert sorted(np.nonzero(got)[0].tolist()) == sorted(chosen)
    assert got.sum() == pytest.approx(1.0, abs=1e-12)
    assert plain[chosen].sum() >= top_p and plain[chosen[:-1]].sum() < top_p  # the smallest such prefix
    assert np.allclose(got[chosen] / got[chosen[0]], plain[chosen] / plain[chosen[0]], rtol=1e-12)
    # with top-k first, the nucleus is taken of the renormalised top-k distribution
    k = 9
    top = sampling.standardise(row, temperature, top_k=k)
    both = sampling.standardise(row, temperature, top_k=k, top_p=top_p)
    assert sorted(np.nonzero(both)[0].tolist()) == sorted(_nucleus_by_repeated_argmax(top, top_p))


def test_nucleus_limits_and_ties():
    tl, _ = _fixed_pair(1.0)
    row = tl[0]
    plain = sampling.standardise(row, 0.8)
    for off in (1.0, 1.5, 0.0, -0.1):
        assert np.array_equal(sampling.standardise(row, 0.8, top_p=off), plain)
    assert np.array_equal(sampling.standardise(row, 0.8, top_p=1e-9), sampling.standardise(row, 0.0))
    assert np.array_equal(sampling.standardise(row, 0.0, top_p=0.3), sampling.standardise(row, 0.0))
    # a tie at the cut stays whole: probabilities 0.4 0.2 0.2 0.2, top_p 0.5 reaches its mass inside the tie
    tied = np.log(np.array([0.2, 0.4, 0.2, 0.2]))
    assert np.nonzero(sampling.standardise(tied, 1.0, top_p=0.5))[0].tolist() == [0, 1, 2, 3]
    assert np.nonzero(sampling.standardise(tied, 1.0, top_p=0.4 - 1e-9))[0].tolist() == [1]
    us = philox.uniforms_vec(9, np.arange(20000), 0, philox.PURPOSE_DRAFT)
    support = set(np.nonzero(sampling.standardise(row, 1.0, top_p=0.5))[0].tolist())
    drawn = sampling.sample_trials(row, us, 1.0, top_p=0.5)
    assert set(drawn.tolist()) <= support
    assert [sampling.sample_token(row, float(u), 1.0, top_p=0.5)[0] for u in us[:200]] == drawn[:200].tolist()


def test_emitted_law_under_the_nucleus_is_the_nucleus_target_distribution():
    trials = 400_000
    tl, ql = _fixed_pair(1.0)
    kw = dict(top_k=20, top_p=0.8)
    p = sampling.standardise(tl[0], 1.0, **kw)
    q = sampling.standardise(ql[0], 1.0, **kw)
    assert 1 < np.count_nonzero(p) < 20 and 1 < np.count_nonzero(q) < 20
    idx = np.arange(trials)
    x = sampling.sample_trials(ql[0], philox.uniforms_vec(8, idx, 0, philox.PURPOSE_DRAFT), 1.0, **kw)
    r = philox.uniforms_vec(8, idx, 0, philox.PURPOSE_ACCEPT)
    u = philox.uniforms_vec(8, idx, 0, philox.PURPOSE_FINAL)
    n, t = sampling.verify_trials(tl, ql, x[:, None], np.stack([r, u], axis=1), 1.0, **kw)
    first = np.where(n == 1, x, t)
    assert np.all(p[first] > 0)
    assert _chi_square_p(np.bincount(first, minlength=VOCAB), p) > 1e-3
    beta = analysis.beta(p, q)
    assert abs((n == 1).mean() - beta) < 4 * np.sqrt(beta * (1 - beta) / trials)
    for i in range(300):
        res = sampling.verify_step(tl, ql, x[i : i + 1], [r[i], u[i]], 1.0, **kw)
        assert (res.n_accepted, res.next_token) == (n[i], t[i])


def test_greedy_rule_for_a_guess_off_the_drafts_support():
    """T = 0: a guess that is not the draft's maximum has q(x) = 0, where Algorithm 1's ratio test
    decides nothing; the reading taken is "accepted iff it is the target's maximum", so that the
    emitted tokens are the target's greedy continuation whatever was guessed (the abstract's claim
    that the outputs do not change)."""
    tl = np.array([[0.1, 2.0, 0.3, 0.0], [1.5, 0.2, 0.1, 0.0], [0.0, 0.1, 0.2, 3.0]])
    ql = np.array([[5.0, 0.0, 0.0, 0.0], [0.0, 0.0, 4.0, 0.0]])   # the draft's maxima: tokens 0 and 2
    us = [0.99, 0.99, 0.5]
    both = sampling.verify_step(tl, ql, [1, 0], us, 0.0)           # the target's maxima, neither is the draft's
    assert (both.n_accepted, both.next_token) == (2, 3)
    second = sampling.verify_step(tl, ql, [1, 2], us, 0.0)         # the draft's own maximum, not the target's
    assert (second.n_accepted, second.next_token) == (1, 0)
    first = sampling.verify_step(tl, ql, [3, 0], us, 0.0)          # neither model's maximum
    assert (first.n_accepted, first.next_token) == (0, 1)
    n, t = sampling.verify_trials(tl, ql, np.array([[1, 0], [1, 2], [3, 0]]), np.tile(us, (3, 1)), 0.0)
    assert n.tolist() == [2, 1, 0] and t.tolist() == [3, 0, 1]
