"""Pins for oracle.analysis: the values the paper prints for its closed forms."""
import os

import numpy as np
import pytest

from conftest import read_golden
from oracle import analysis


def test_table1_operations_and_speed(golden_dir):
    rows = read_golden(os.path.join(golden_dir, "table1_ops_speed.txt"))
    assert len(rows) == 6
    for alpha, gamma, ops, speed in rows:
        alpha, gamma = float(alpha), int(gamma)
        assert round(analysis.ops_increase(alpha, gamma, 0.0), 2) == pytest.approx(float(ops), abs=1e-9)
        assert round(analysis.walltime_improvement(alpha, gamma, 0.0), 2) == pytest.approx(float(speed), abs=1e-9)


def test_table4_expected_improvement(golden_dir):
    rows = read_golden(os.path.join(golden_dir, "table4_expected_improvement.txt"))
    assert len(rows) == 12
    for gamma, alpha, c, exp in rows:
        got = analysis.walltime_improvement(float(alpha), int(gamma), float(c))
        assert abs(got - float(exp)) < 0.08, (gamma, alpha, c, exp, got)


def test_bigram_example_of_section_3_6():
    # alpha = 0.2, gamma = 3, c = 0 is quoted as a 1.25X improvement.
    assert round(analysis.walltime_improvement(0.2, 3, 0.0), 2) == 1.25


def test_corollary_3_9_is_theorem_3_8_at_gamma_1():
    for alpha in (0.1, 0.5, 0.9):
        for c in (0.0, 0.05, 0.3):
            assert analysis.walltime_improvement(alpha, 1, c) == pytest.approx(
                analysis.walltime_improvement_lower_bound(alpha, c), rel=1e-14)


def test_expected_tokens_is_the_capped_geometric_mean():
    # Eq. 1 against the direct expectation: k tokens w.p. alpha^(k-1)(1-alpha), cap gamma+1.
    for alpha in (0.0, 0.3, 0.77, 1.0):
        for gamma in (1, 4, 9):
            direct = sum(k * alpha ** (k - 1) * (1 - alpha) for k in range(1, gamma + 1))
            direct += (gamma + 1) * alpha**gamma
            assert analysis.expected_tokens(alpha, gamma) == pytest.approx(direct, rel=1e-12)


def test_lemma_3_3_and_corollary_3_4():
    rng = np.random.default_rng(3)
    for _ in range(20):
        p = rng.dirichlet(np.ones(11))
        q = rng.dirichlet(np.ones(11))
        assert analysis.d_lk(p, q) == pytest.approx(1.0 - analysis.beta(p, q), abs=1e-14)
        assert analysis.d_lk(p, q) == pytest.approx(analysis.d_lk(q, p), abs=1e-14)
        assert 0.0 <= analysis.d_lk(p, q) <= 1.0
    assert analysis.d_lk(p, p) == 0.0
    a = np.array([0.5, 0.5, 0.0, 0.0])
    b = np.array([0.0, 0.0, 0.25, 0.75])
    assert analysis.d_lk(a, b) == 1.0 and analysis.beta(a, b) == 0.0


def test_lenient_acceptance_form():
    rng = np.random.default_rng(4)
    p, q = rng.dirichlet(np.ones(9)), rng.dirichlet(np.ones(9))
    for l in (1.0, 0.5, 0.1):
        direct = float(np.sum(p * q / np.maximum(p, l * q)))  # E_{x~q} p / max(p, l q)
        assert analysis.beta_lenient(p, q, l) == pytest.approx(direct, rel=1e-12)
    assert analysis.beta_lenient(p, q, 1.0) == pytest.approx(analysis.beta(p, q), rel=1e-14)


def test_best_gamma_is_the_integer_argmax():
    for alpha, c in [(0.8, 0.02), (0.6, 0.1), (0.9, 0.0)]:
        g = analysis.best_gamma(alpha, c, gamma_max=40)
        best = analysis.walltime_improvement(alpha, g, c)
        assert all(best >= analysis.walltime_improvement(alpha, k, c) for k in range(1, 41))


def test_generalised_speedup_reduces_to_theorem_3_8():
    alpha, gamma, c = 0.7, 4, 0.05
    tokens = analysis.expected_tokens(alpha, gamma)
    assert analysis.generalised_speedup(tokens, 1.0, 1.0, c, gamma) == pytest.approx(
        analysis.walltime_improvement(alpha, gamma, c), rel=1e-14)
