"""Pins for oracle.generate: Algorithm 1 looped, against what the paper fixes."""
import itertools

import numpy as np
import pytest
from scipy import stats

from oracle import analysis, generate, sampling
from oracle.decoder import Decoder
from paper_2211_17192_b200 import workloads


class TableModel:
    """A "model" whose next-token logits are a fixed table of the last `order`
    tokens (order 0: the same distribution everywhere).  Same interface as
    oracle.decoder.Decoder, including a row cache that must be rolled back."""

    def __init__(self, vocab, order, seed, scale=1.0):
        rng = np.random.default_rng(seed)
        self.vocab, self.order = vocab, order
        self.table = rng.normal(0, scale, (vocab,) * order + (vocab,))
        self.fed = []

    def reset(self):
        self.fed = []

    @property
    def cached_len(self):
        return len(self.fed)

    def truncate(self, length):
        self.fed = self.fed[:length]

    def _row(self, prefix):
        ctx = tuple(prefix[-self.order:]) if self.order else ()
        if len(ctx) < self.order:
            ctx = (0,) * (self.order - len(ctx)) + ctx
        return self.table[ctx]

    def forward_rows(self, tokens):
        rows = []
        for t in tokens:
            self.fed.append(int(t))
            rows.append(self._row(self.fed))
        return np.stack(rows)

    def forward_full(self, tokens):
        tokens = [int(t) for t in tokens]
        return np.stack([self._row(tokens[: i + 1]) for i in range(len(tokens))])

    def prob(self, prefix):
        return sampling.standardise(self._row(list(prefix)), 1.0)


@pytest.mark.parametrize("gamma", [1, 2, 3, 5, 8])
def test_temperature_zero_equals_target_only_greedy(gamma):
    tcfg = workloads.scaled_config(workloads.model_config("tiny_target"), n_layers=2, vocab=211, max_positions=64)
    dcfg = workloads.scaled_config(workloads.model_config("tiny_draft"), n_layers=1, vocab=211, max_positions=64)
    target, draft = Decoder(tcfg, workloads.make_weights(tcfg, 1)), Decoder(dcfg, workloads.make_weights(dcfg, 2))
    prompt = workloads.make_prompt(3, 6, 211)
    greedy, _, _ = generate.target_only_generate(target, prompt, 20, 0.0, seed=0)
    spec = generate.speculative_generate(target, draft, prompt, 20, gamma, 0.0, seed=0)
    assert spec.tokens == greedy
    # and with a draft that agrees with the target (itself): every guess accepted
    twin = Decoder(tcfg, workloads.make_weights(tcfg, 1))
    spec = generate.speculative_generate(target, twin, prompt, 20, gamma, 0.0, seed=0)
    assert spec.tokens == greedy and all(it.n_accepted == gamma for it in spec.iterations)


@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_cached_equals_cache_free(temperature):
    tcfg = workloads.scaled_config(workloads.model_config("llama_test_target"), vocab=150, max_positions=64)
    dcfg = workloads.scaled_config(workloads.model_config("llama_test_draft"), vocab=150, max_positions=64)
    target, draft = Decoder(tcfg, workloads.make_weights(tcfg, 1)), Decoder(dcfg, workloads.make_weights(dcfg, 2))
    prompt = workloads.make_prompt(5, 5, 150)
    a = generate.speculative_generate(target, draft, prompt, 24, 3, temperature, seed=77, cached=True, keep_logits=True)
    b = generate.speculative_generate(target, draft, prompt, 24, 3, temperature, seed=77, cached=False, keep_logits=True)
    assert a.tokens == b.tokens and len(a.iterations) == len(b.iterations)
    for x, y in zip(a.iterations, b.iterations):
        assert np.allclose(x.target_logits, y.target_logits, atol=1e-10)
        assert np.allclose(x.draft_logits, y.draft_logits, atol=1e-10)
    ns = [it.n_accepted for it in a.iterations]
    if temperature == 1.0:
        assert 0 in ns and max(ns) > 0  # both rollback and acceptance were exercised


def test_emitted_sequence_law_equals_the_target_law():
    """Monte Carlo through the real loop with context-dependent table models
    (vocabulary 3, three new tokens, gamma = 2): the law of the emitted
    sequence equals prod_t p(x_t | x_<t)."""
    V, n_new, runs = 3, 3, 30000
    target, draft = TableModel(V, 2, seed=1), TableModel(V, 1, seed=2)
    prompt = [1]
    counts = np.zeros((V,) * n_new)
    iters = 0
    for seed in range(runs):
        res = generate.speculative_generate(target, draft, prompt, n_new, 2, 1.0, seed=seed, cached=True)
        counts[tuple(res.tokens)] += 1
        iters += len(res.iterations)
    law = np.zeros((V,) * n_new)
    for seq in itertools.product(range(V), repeat=n_new):
        pr, prefix = 1.0, list(prompt)
        for t in seq:
            pr *= target.prob(prefix)[t]
            prefix.append(t)
        law[seq] = pr
    assert law.sum() == pytest.approx(1.0)
    assert stats.chisquare(counts.ravel(), law.ravel() * runs).pvalue > 1e-3
    assert iters < runs * n_new  # some guesses were accepted


def test_tokens_per_iteration_follow_eq_1_through_the_loop():
    V, gamma = 16, 3
    target, draft = TableModel(V, 0, seed=3, scale=1.5), TableModel(V, 0, seed=4, scale=1.5)
    draft.table = target.table + np.random.default_rng(5).normal(0, 0.7, V)
    alpha = analysis.beta(target.prob([]), draft.prob([]))
    per_iter = []
    tests_eval = tests_pass = 0
    for seed in range(150):
        res = generate.speculative_generate(target, draft, [0], 64, gamma, 1.0, seed=seed)
        assert len(res.tokens) == 64
        for it in res.iterations[:-1]:  # the last iteration may be cut short by n_new
            per_iter.append(it.n_accepted + 1)
        tests_eval += res.tests_evaluated
        tests_pass += res.tests_passed
    per_iter = np.array(per_iter)
    assert per_iter.min() >= 1 and per_iter.max() <= gamma + 1
    assert abs(per_iter.mean() - analysis.expected_tokens(alpha, gamma)) < 4 * per_iter.std() / np.sqrt(per_iter.size)
    assert abs(tests_pass / tests_eval - alpha) < 4 * np.sqrt(alpha * (1 - alpha) / tests_eval)


def test_target_only_sampling_follows_p():
    V = 5
    target = TableModel(V, 0, seed=8)
    counts = np.zeros(V)
    for seed in range(4000):
        toks, _, _ = generate.target_only_generate(target, [0], 2, 1.0, seed=seed)
        for t in toks:
            counts[t] += 1
    assert stats.chisquare(counts, target.prob([]) * counts.sum()).pvalue > 1e-3


def test_generation_is_position_keyed():
    """Restarting from a committed prefix reproduces the rest of the run when the
    prefix ends at an iteration boundary (randomness is keyed by position)."""
    V = 12
    target, draft = TableModel(V, 2, seed=1), TableModel(V, 1, seed=2)
    full = generate.speculative_generate(target, draft, [3, 4], 30, 3, 1.0, seed=9)
    cut = full.iterations[4].start_len  # committed length at the start of iteration 4
    done = cut - 2
    rest = generate.speculative_generate(target, draft, [3, 4] + full.tokens[:done], 30 - done, 3, 1.0, seed=9)
    assert rest.tokens == full.tokens[done:]


def test_bigram_table_draft():
    """A table look-up as M_q (the paper's negligible-cost drafts): logits depend on the
    last token only; a target that is itself that table accepts everything; T = 0
    output equals the target's greedy output whatever the table."""
    from oracle.ngram import BigramTable
    rng = np.random.default_rng(5)
    table = rng.standard_normal((32, 32)) * 2.0
    draft = BigramTable(table)
    a = draft.forward_rows([3, 7, 7])
    assert np.array_equal(a[1], a[2]) and np.array_equal(a[0], table[3]) and draft.cached_len == 3
    draft.truncate(1)
    assert draft.cached_len == 1
    same = generate.speculative_generate(BigramTable(table), BigramTable(table), [1, 2], 30, 4, 1.0, seed=3)
    assert same.tests_passed == same.tests_evaluated and all(it.n_accepted == 4 for it in same.iterations)
    other = BigramTable(rng.standard_normal((32, 32)))
    want, _, _ = generate.target_only_generate(BigramTable(table), [1, 2], 25, 0.0, seed=0)
    got = generate.speculative_generate(BigramTable(table), other, [1, 2], 25, 3, 0.0, seed=0)
    assert got.tokens == want


def test_copy_from_context_draft():
    """Section 3.6's parameter-less draft.  The rule on hand-written sequences; a periodic target
    accepts every guess once one period is in the context; a one-hot draft is accepted with
    probability p(guess); T = 0 output equals the target's greedy output."""
    from oracle.ngram import BigramTable, CopyFromContext
    draft = CopyFromContext(10, 2)
    #            0  1  2  3  4  5  6  7
    assert draft.guess([1, 2, 3, 4, 1, 2]) == 3            # "1 2" was followed by 3
    assert draft.guess([1, 2, 3, 1, 2, 5, 1, 2]) == 5      # the most recent occurrence wins
    assert draft.guess([1, 2, 3, 4]) == 4                  # no earlier "3 4": repeat the last token
    assert draft.guess([7]) == 7 and draft.guess([7, 7]) == 7
    assert draft.guess([7, 7, 7]) == 7                     # overlapping occurrence: "7 7" ends at index 1
    assert CopyFromContext(10, 1).guess([4, 9, 5, 4]) == 9
    assert CopyFromContext(10, 3).guess([1, 2, 3, 9, 2, 3, 8, 1, 2, 3]) == 9
    rows = draft.forward_rows([1, 2, 3, 1, 2])
    assert rows.shape == (5, 10) and draft.cached_len == 5
    assert np.argmax(rows[4]) == 3 and np.isneginf(np.delete(rows[4], 3)).all() and rows[4][3] == 0.0
    assert np.array_equal(rows, draft.forward_full([1, 2, 3, 1, 2]))
    draft.truncate(3)
    assert np.argmax(draft.forward_rows([9])[0]) == 9

    # a target that walks a fixed cycle: next = perm[last]; sharp table, so sampling follows the cycle
    vocab, period = 12, 5
    cycle = [3, 8, 1, 10, 6]
    table = np.full((vocab, vocab), -40.0)
    for a, b in zip(cycle, cycle[1:] + cycle[:1]):
        table[a, b] = 0.0
    for a in set(range(vocab)) - set(cycle):
        table[a, cycle[0]] = 0.0
    prompt = cycle + cycle[:2]  # one full period and a bit: every 2-gram has occurred
    res = generate.speculative_generate(BigramTable(table), CopyFromContext(vocab, 2), prompt, 40, 4, 1.0, seed=2)
    assert res.tests_passed == res.tests_evaluated and all(it.n_accepted == 4 for it in res.iterations)
    assert res.tokens[:6] == [1, 10, 6, 3, 8, 1]

    # one-hot q at x: accepted with probability p(x) (Section 2.3 with q(x) = 1), else drawn from p without x
    target = TableModel(8, 0, seed=3)
    p = target.prob([])
    x = 5
    q_row = np.full(8, -np.inf)
    q_row[x] = 0.0
    trials = 200_000
    us = np.random.default_rng(1).random((trials, 2))
    n, t = sampling.verify_trials(np.stack([target.table, target.table]), q_row[None], np.full((trials, 1), x), us, 1.0)
    assert abs((n == 1).mean() - p[x]) < 4 * np.sqrt(p[x] * (1 - p[x]) / trials)
    rest = p.copy()
    rest[x] = 0.0
    assert not np.any(t[n == 0] == x)
    counts = np.bincount(t[n == 0], minlength=8)
    assert stats.chisquare(np.delete(counts, x), np.delete(rest / rest.sum(), x) * counts.sum()).pvalue > 1e-3

    tcfg = workloads.model_config("tiny_target")
    model = Decoder(tcfg, workloads.make_weights(tcfg, 1))
    rep = workloads.make_repetitive_prompt(5, 24, tcfg["vocab"], 6)
    want, _, _ = generate.target_only_generate(model, rep, 12, 0.0, seed=0)
    got = generate.speculative_generate(model, CopyFromContext(tcfg["vocab"], 2), rep, 12, 3, 0.0, seed=0)
    assert got.tokens == want
