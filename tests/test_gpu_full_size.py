"""Properties that hold at any size, checked at the benchmark's own size and launch configuration: the
Llama-7B-shaped target (32 blocks, full width) with the 160M-shaped draft, a 1024-token prompt, gamma = 2, the
cache capacity the benchmark uses.  The oracle cannot run this size; what Algorithm 1 guarantees can still be
checked: at T = 0 speculative decoding emits the target's own greedy stream (Section 2.3: the output
distribution is the target's; at T = 0 that distribution is a point), the counters add up (Eq. 1's n per
iteration), and with every guess accepted an iteration emits gamma + 1 tokens."""
import numpy as np
import pytest
import torch

import bench
from oracle.encdec import START_TOKEN
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu

PROMPT, NEW, GAMMA = 1024, 24, 2
BF16_ABS = 2e-2


@pytest.fixture(scope="module")
def pair():
    device = torch.device("cuda", 0)
    tcfg, dcfg = workloads.model_config("llama7b_target"), workloads.model_config("llama160m_draft")
    eng = binding.Engine(tcfg, bench.gpu_weights(tcfg, 1, device), dcfg, bench.gpu_weights(dcfg, 2, device), max_batch=1,
                         max_len=PROMPT + 256 + GAMMA + 2, page_size=64, max_gamma=GAMMA)
    yield eng, tcfg
    eng.close()


def test_greedy_speculative_stream_is_the_targets_greedy_stream(pair):
    eng, cfg = pair
    prompt = workloads.make_prompt(31, PROMPT, cfg["vocab"])
    greedy, _ = eng.generate([prompt], NEW, 0, 0.0, 0)
    spec, stats = eng.generate([prompt], NEW, GAMMA, 0.0, 0)
    assert binding.spec_device_error() == 0
    differ = np.nonzero(greedy[0] != spec[0])[0]
    if differ.size:
        # the verification pass (3 rows) and the one-row pass round differently: a tie of the two largest logits
        # within the bf16 tolerance may fall either way; anything else is an error
        k = int(differ[0])
        assert k >= 8, f"streams differ at token {k}"
        eng.reset()
        seq = np.concatenate([prompt, greedy[0, :k]]).astype(np.int32)
        last = None
        for at in range(0, len(seq), 64):
            last = eng.forward_logits(0, seq[None, at:at + 64])
        row = np.sort(last[0, -1].cpu().numpy())
        assert row[-1] - row[-2] <= 2 * BF16_ABS, f"streams differ at token {k} with a top-2 gap of {row[-1] - row[-2]:.3g}"
    assert stats["tokens"] >= NEW and stats["iterations"] <= NEW
    assert sum(stats["accepted_histogram"][:GAMMA + 1]) == stats["iterations"]
    assert stats["tests_passed"] == sum(n * c for n, c in enumerate(stats["accepted_histogram"][:GAMMA + 1]))


def test_sampled_run_counters_add_up(pair):
    eng, cfg = pair
    prompt = workloads.make_prompt(32, PROMPT, cfg["vocab"])
    out, stats = eng.generate([prompt], NEW, GAMMA, 1.0, 5)
    assert binding.spec_device_error() == 0
    assert out.shape == (1, NEW) and int(out.min()) >= 0 and int(out.max()) < cfg["vocab"]
    hist = stats["accepted_histogram"][:GAMMA + 1]
    assert sum(hist) == stats["iterations"]
    assert stats["tokens"] == sum((n + 1) * c for n, c in enumerate(hist))      # n accepted guesses and one more token
    assert stats["tests_passed"] == sum(n * c for n, c in enumerate(hist))
    assert stats["tests_evaluated"] == stats["tests_passed"] + sum(hist[:GAMMA])  # every iteration with n < gamma met one rejection
    again, _ = eng.generate([prompt], NEW, GAMMA, 1.0, 5)
    assert np.array_equal(out, again)                                          # same seed, same stream


def test_every_guess_accepted_gives_gamma_plus_one_tokens_per_iteration(pair):
    eng, cfg = pair
    prompt = workloads.make_prompt(33, PROMPT, cfg["vocab"])
    eng.set_imposed_acceptance(1.0)
    try:
        _, stats = eng.generate([prompt], 3 * (GAMMA + 1), GAMMA, 1.0, 9)
    finally:
        eng.set_imposed_acceptance(None)
    assert stats["iterations"] == 3 and stats["tokens"] == 3 * (GAMMA + 1)
    assert stats["accepted_histogram"][GAMMA] == 3


@pytest.mark.parametrize("target,draft,prompt_len,gamma", [("gpt97m_target", "gpt6m_draft", 128, 5),
                                                          ("t5xxl_target", "t5small_draft", 512, 5)])
def test_greedy_equivalence_on_the_other_benchmark_pairs(target, draft, prompt_len, gamma):
    """The GPT 97M / 6M shapes (128-token prompt) and the T5-XXL / T5-small shapes (512-token source), gamma = 5,
    as the benchmark runs them: the greedy speculative stream is the target's greedy stream."""
    device = torch.device("cuda", 0)
    tcfg, dcfg = workloads.model_config(target), workloads.model_config(draft)
    t5 = tcfg["arch"] == "t5"
    new = 36
    eng = binding.Engine(tcfg, bench.gpu_weights(tcfg, 3, device), dcfg, bench.gpu_weights(dcfg, 4, device), max_batch=1,
                         max_len=(1 if t5 else prompt_len) + new + gamma + 2, page_size=64, max_gamma=gamma,
                         max_src_len=prompt_len if t5 else 0)
    try:
        prompt = workloads.make_prompt(41, prompt_len, tcfg["vocab"])
        greedy, _ = eng.generate([prompt], new, 0, 0.0, 0)
        spec, stats = eng.generate([prompt], new, gamma, 0.0, 0)
        assert binding.spec_device_error() == 0
        differ = np.nonzero(greedy[0] != spec[0])[0]
        if differ.size:  # (see the first test: only a tie within the tolerance may fall either way)
            k = int(differ[0])
            assert k >= 8, f"streams differ at token {k}"
            if t5:
                eng.encode([prompt])
                seq = np.concatenate([[START_TOKEN], greedy[0, :k]]).astype(np.int32)
            else:
                seq = np.concatenate([prompt, greedy[0, :k]]).astype(np.int32)
            eng.reset()
            last = None
            for at in range(0, len(seq), 32):
                last = eng.forward_logits(0, seq[None, at:at + 32])
            row = np.sort(last[0, -1].cpu().numpy())
            assert row[-1] - row[-2] <= 2 * BF16_ABS, f"streams differ at token {k} with a top-2 gap of {row[-1] - row[-2]:.3g}"
        hist = stats["accepted_histogram"][:gamma + 1]
        assert sum(hist) == stats["iterations"] and stats["tokens"] == sum((n + 1) * c for n, c in enumerate(hist))
    finally:
        eng.close()


def test_greedy_equivalence_in_a_ragged_batch_of_sixteen():
    """Config 5's batched corner at full size: 16 sequences with prompts of 1000 .. 1015 tokens, gamma = 4 (80-row
    verification passes, the f16 attention kernel, ragged roll-back every iteration): every sequence's greedy
    speculative stream is its greedy target-only stream."""
    device = torch.device("cuda", 0)
    tcfg, dcfg = workloads.model_config("llama7b_target"), workloads.model_config("llama160m_draft")
    batch, gamma, new = 16, 4, 12
    eng = binding.Engine(tcfg, bench.gpu_weights(tcfg, 1, device), dcfg, bench.gpu_weights(dcfg, 2, device), max_batch=batch,
                         max_len=1016 + new + gamma + 2, page_size=64, max_gamma=gamma)
    try:
        assert eng.attention_plan(0, batch, gamma + 1)["f16"]
        prompts = [workloads.make_prompt(60 + b, 1000 + b, tcfg["vocab"]) for b in range(batch)]
        greedy, _ = eng.generate(prompts, new, 0, 0.0, 0)
        spec, stats = eng.generate(prompts, new, gamma, 0.0, 0)
        assert binding.spec_device_error() == 0
        for b in range(batch):
            differ = np.nonzero(greedy[b] != spec[b])[0]
            if not differ.size:
                continue
            k = int(differ[0])  # only a tie within the tolerance may fall either way
            seq = np.concatenate([prompts[b], greedy[b, :k]]).astype(np.int32)
            eng.reset()
            last = None
            for at in range(0, len(seq), 64):
                last = eng.forward_logits(0, seq[None, at:at + 64])
            row = np.sort(last[0, -1].cpu().numpy())
            assert row[-1] - row[-2] <= 2 * BF16_ABS, f"sequence {b} differs at token {k} with a top-2 gap of {row[-1] - row[-2]:.3g}"
        hist = stats["accepted_histogram"][:gamma + 1]
        assert stats["tokens"] == sum((n + 1) * c for n, c in enumerate(hist))  # over all sequences and iterations
        assert stats["tests_passed"] == sum(n * c for n, c in enumerate(hist))
    finally:
        eng.close()
