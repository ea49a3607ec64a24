"""The library's host-side choice of gamma (Section 3.5) against the oracle's closed forms, and
the oracle's loop under a gamma schedule (no GPU needed)."""
import numpy as np
import pytest

from oracle import analysis, generate
from oracle.decoder import Decoder
from paper_2211_17192_b200 import binding, workloads


def test_choice_maximises_theorem_3_8():
    for alpha in np.linspace(0.05, 0.98, 32):
        for c in (0.0, 0.01, 0.05, 0.1, 0.3, 0.8):
            got = binding.spec_choose_gamma(alpha, 1.0, c, 40)
            best = analysis.best_gamma(float(alpha), c, gamma_max=40)
            if got != best:  # a flat maximum (alpha^gamma below rounding): the values must agree to the last digits
                assert analysis.walltime_improvement(alpha, got, c) >= analysis.walltime_improvement(alpha, best, c) * (1 - 1e-14)
                assert c == 0.0
            # scaling both costs changes nothing
            assert binding.spec_choose_gamma(alpha, 2.5, 2.5 * c, 40) == got


def test_choice_with_a_measured_cost_line():
    """The general form: tokens of Eq. 1 over base + per_guess * gamma, by brute force."""
    for alpha in (0.0, 0.3, 0.6, 0.9, 1.0):
        for base, per in ((2.84, 0.55), (0.3, 0.11), (1.0, 0.0)):
            rates = [analysis.expected_tokens(alpha, g) / (base + per * g) for g in range(1, 9)]
            assert binding.spec_choose_gamma(alpha, base, per, 8) == int(np.argmax(rates)) + 1
    assert binding.spec_choose_gamma(0.0, 1.0, 0.1, 8) == 1    # nothing is ever accepted
    assert binding.spec_choose_gamma(1.0, 1.0, 0.01, 8) == 8   # everything is, and guesses are cheap
    for bad in ((-0.1, 1.0, 0.1, 4), (1.1, 1.0, 0.1, 4), (0.5, 0.0, 0.1, 4), (0.5, 1.0, -1.0, 4), (0.5, 1.0, 0.1, 0)):
        with pytest.raises(ValueError):
            binding.spec_choose_gamma(*bad)


def test_oracle_loop_under_a_gamma_schedule():
    tcfg, dcfg = workloads.model_config("tiny_target"), workloads.model_config("tiny_draft")
    target = Decoder(tcfg, workloads.make_weights(tcfg, 1))
    draft = Decoder(dcfg, workloads.make_weights(dcfg, 2))
    prompt = workloads.make_prompt(3, 9, tcfg["vocab"])
    # a constant schedule is the fixed-gamma loop
    fixed = generate.speculative_generate(target, draft, prompt, 20, 3, 1.0, seed=4)
    same = generate.speculative_generate(target, draft, prompt, 20, [3, 3], 1.0, seed=4)
    assert fixed.tokens == same.tokens
    # at T = 0 no schedule changes the output (it is the target's greedy decoding)
    greedy, _, _ = generate.target_only_generate(target, prompt, 20, 0.0, seed=4)
    varied = generate.speculative_generate(target, draft, prompt, 20, [1, 4, 2, 5, 1, 3], 0.0, seed=4)
    assert varied.tokens == greedy
    assert [len(it.draft_tokens) for it in varied.iterations][:3] == [1, 4, 2]
    # cached and cache-free agree under a varying schedule (the draft's cache catches up whatever gamma was)
    a = generate.speculative_generate(target, draft, prompt, 16, [2, 5, 1, 4], 1.0, seed=6, cached=True)
    b = generate.speculative_generate(target, draft, prompt, 16, [2, 5, 1, 4], 1.0, seed=6, cached=False)
    assert a.tokens == b.tokens
