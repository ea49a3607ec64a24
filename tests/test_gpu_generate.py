"""End-to-end generation through the C ABI against the CPU oracle: Algorithm 1
with both decoders, free-running, plus the properties the paper fixes."""
import numpy as np
import pytest

from gpu_util import compare_generation
from oracle import generate as oracle_generate
from oracle.decoder import Decoder
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu

# A free-running comparison ends at the first decision that sits within tolerance of a boundary;
# it must have compared at least this many tokens by then (a flagged decision at the very start
# would otherwise pass with nothing verified).
MIN_COMPARED = 10


def _models(target_name, draft_name, **overrides):
    tcfg = workloads.scaled_config(workloads.model_config(target_name), **overrides)
    dcfg = workloads.scaled_config(workloads.model_config(draft_name), **overrides)
    return tcfg, workloads.make_weights(tcfg, 1), dcfg, workloads.make_weights(dcfg, 2)


@pytest.fixture(scope="module")
def tiny():
    tcfg, tw, dcfg, dw = _models("tiny_target", "tiny_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=4, max_len=128, page_size=32, max_gamma=8)
    yield eng, Decoder(tcfg, tw), Decoder(dcfg, dw), tcfg
    eng.close()


@pytest.mark.parametrize("temperature", [1.0, 0.0])
def test_tiny_pair_matches_the_oracle(tiny, temperature):
    """Tiny fp32 pair, gamma = 3, 16-token prompt, 64 new tokens."""
    eng, target, draft, cfg = tiny
    prompt = workloads.make_prompt(7, 16, cfg["vocab"])
    flagged, iters = compare_generation(eng, target, draft, prompt, 64, 3, temperature, seed=11, margin=1e-3,
                                        logit_tol=1e-3)
    assert flagged <= 2, f"{flagged} decisions within tolerance of a boundary in {iters} iterations"


@pytest.mark.parametrize("gamma", [1, 2, 5, 8])
def test_temperature_zero_equals_target_only_greedy(tiny, gamma):
    eng, target, _, cfg = tiny
    prompt = workloads.make_prompt(8, 9, cfg["vocab"])
    greedy, _ = eng.generate([prompt], 40, 0, 0.0, 0)
    spec, stats = eng.generate([prompt], 40, gamma, 0.0, 0)
    assert np.array_equal(greedy, spec)
    ref, rows, _ = oracle_generate.target_only_generate(target, prompt, 40, 0.0, 0, keep_logits=True)
    gaps = [np.sort(r)[-1] - np.sort(r)[-2] for r in rows]
    for k in range(40):
        if greedy[0, k] != ref[k]:
            assert gaps[k] < 2e-3  # an argmax tie within the logit tolerance; the runs diverge from here
            assert k >= MIN_COMPARED, f"only {k} tokens were compared before a tolerance-flagged tie"
            break
    assert stats["iterations"] >= 40 / (gamma + 1)


def test_shortest_prompts_fewest_tokens_and_surplus_guesses(tiny):
    """Prompts of 1, 2 and 3 tokens (the first draft step feeds positions L-2 and L-1: with one token there is
    no L-2), 1, 2 and 5 new tokens with gamma = 1 and gamma = 8 (more guesses than tokens wanted: the surplus of
    the last iteration is dropped), sampled and greedy: token for token the oracle's stream."""
    eng, target, draft, cfg = tiny
    for plen in (1, 2, 3):
        prompt = workloads.make_prompt(40 + plen, plen, cfg["vocab"])
        for n_new in (1, 2, 5):
            for gamma in (1, 8):
                for temperature in (1.0, 0.0):
                    got, _ = eng.generate([prompt], n_new, gamma, temperature, 3)
                    ref = oracle_generate.speculative_generate(target, draft, prompt, n_new, gamma, temperature, 3)
                    if list(got[0]) != list(ref.tokens[:n_new]):  # (a handful of decisions: none may sit on a boundary)
                        raise AssertionError(f"prompt {plen}, {n_new} new, gamma {gamma}, T {temperature}: "
                                             f"{list(got[0])} against {ref.tokens[:n_new]}")


def test_target_only_sampling_matches_the_oracle(tiny):
    eng, target, _, cfg = tiny
    prompt = workloads.make_prompt(9, 5, cfg["vocab"])
    got, stats = eng.generate([prompt], 48, 0, 1.0, 5)
    ref, _, margins = oracle_generate.target_only_generate(target, prompt, 48, 1.0, 5)
    for k in range(48):
        if got[0, k] != ref[k]:
            assert margins[k] < 1e-3
            assert k >= MIN_COMPARED, f"only {k} tokens were compared before a tolerance-flagged draw"
            break
    assert stats["iterations"] == 48 and stats["tests_evaluated"] == 0 and stats["draft_passes"] == 0


def test_draft_equal_to_target_accepts_everything():
    tcfg, tw, _, _ = _models("tiny_target", "tiny_draft", n_layers=2)
    eng = binding.Engine(tcfg, tw, tcfg, tw, max_batch=1, max_len=128, page_size=32, max_gamma=4)
    prompt = workloads.make_prompt(3, 10, tcfg["vocab"])
    out, stats = eng.generate([prompt], 50, 4, 1.0, 3)
    assert stats["tests_passed"] == stats["tests_evaluated"] == 4 * stats["iterations"]
    assert stats["iterations"] == 10 and stats["tokens"] == 50
    eng.close()


def test_ragged_batch_equals_per_sequence_oracle(tiny):
    eng, target, draft, cfg = tiny
    prompts = [workloads.make_prompt(20 + b, n, cfg["vocab"]) for b, n in enumerate([3, 16, 9, 1])]
    out, stats = eng.generate(prompts, 24, 3, 1.0, 17)
    assert stats["tokens"] >= 4 * 24
    for b, prompt in enumerate(prompts):
        ref = oracle_generate.speculative_generate(target, draft, prompt, 24, 3, 1.0, 17, sequence=b)
        got = out[b].tolist()
        diff = next((k for k in range(24) if got[k] != ref.tokens[k]), None)
        if diff is not None:
            index = len(prompt) + diff
            it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
            assert min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins)) < 1e-3
            assert diff >= MIN_COMPARED, f"sequence {b}: only {diff} tokens were compared before a tolerance-flagged decision"


def test_bf16_llama_pair_matches_the_oracle():
    tcfg, tw, dcfg, dw = _models("llama_test_target", "llama_test_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=1, max_len=256, page_size=32, max_gamma=4)
    prompt = workloads.make_prompt(2, 24, tcfg["vocab"])
    for temperature in (1.0, 0.0):
        flagged, iters = compare_generation(eng, Decoder(tcfg, tw), Decoder(dcfg, dw), prompt, 48, 4, temperature,
                                            seed=5, margin=5e-3, logit_tol=5e-3)
        assert flagged <= 3, f"{flagged} flagged of {iters}"
    eng.close()


@pytest.mark.parametrize("prompt_len", [200, 257, 300, 470])
def test_long_prompts_through_the_prompt_pass(prompt_len):
    """Prompts longer than one chunk of the prompt pass (256 rows per chunk: 200 rows in one chunk of three
    80-row token tiles, 256 + 1, 256 + 44, 256 + 214), several pages and key tiles, then free-running
    generation against the oracle, sampled and greedy: a wrong row anywhere in the cached prompt changes the
    stream."""
    tcfg, tw, dcfg, dw = _models("llama_test_target", "llama_test_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=1, max_len=512, page_size=32, max_gamma=3)
    prompt = workloads.make_prompt(50 + prompt_len, prompt_len, tcfg["vocab"])
    try:
        for temperature in (1.0, 0.0):
            flagged, iters = compare_generation(eng, Decoder(tcfg, tw), Decoder(dcfg, dw), prompt, 24, 3, temperature,
                                                seed=6, margin=5e-3, logit_tol=5e-3)
            assert flagged <= 3, f"{flagged} flagged of {iters}"
    finally:
        eng.close()


def test_ragged_long_prompts_in_one_batch():
    """Three sequences with prompts of 300, 130 and 77 tokens decoded together: the prompt pass cuts each into its
    own chunks; every sequence's greedy stream equals the one it gives alone, and the first equals the oracle's."""
    tcfg, tw, dcfg, dw = _models("llama_test_target", "llama_test_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=3, max_len=512, page_size=32, max_gamma=3)
    try:
        prompts = [workloads.make_prompt(70 + b, n, tcfg["vocab"]) for b, n in enumerate([300, 130, 77])]
        together, _ = eng.generate(prompts, 20, 3, 0.0, 0)
        for b in range(3):
            alone, _ = eng.generate([prompts[b]], 20, 3, 0.0, 0)
            assert np.array_equal(alone[0], together[b]), f"sequence {b}"
        ref, rows, _ = oracle_generate.target_only_generate(Decoder(tcfg, tw), prompts[0], 20, 0.0, 0, keep_logits=True)
        for k in range(20):
            if together[0, k] != ref[k]:
                gap = np.sort(rows[k])[-1] - np.sort(rows[k])[-2]
                assert gap < 2e-2 and k >= MIN_COMPARED, f"token {k}: top-2 gap {gap:.3g}"
                break
    finally:
        eng.close()


def test_batch_of_sixteen_on_the_f16_attention_path_matches_the_oracle():
    """16 ragged sequences of the bf16 Llama-shaped test pair decoded together (32 (sequence, KV head) pairs: the
    verification passes take the f16 tensor-core attention, with a ragged roll-back every iteration): at T = 0 every
    sequence's stream is the oracle's greedy stream of the target, up to a tie within the logit tolerance."""
    tcfg, tw, dcfg, dw = _models("llama_test_target", "llama_test_draft")
    batch, gamma, new = 16, 3, 16
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=batch, max_len=512, page_size=32, max_gamma=gamma)
    try:
        assert eng.attention_plan(0, batch, gamma + 1)["f16"]
        prompts = [workloads.make_prompt(90 + b, 20 + 2 * b, tcfg["vocab"]) for b in range(batch)]
        got, stats = eng.generate(prompts, new, gamma, 0.0, 0)
        target = Decoder(tcfg, tw)
        compared = 0
        for b in range(batch):
            ref, rows, _ = oracle_generate.target_only_generate(target, prompts[b], new, 0.0, 0, keep_logits=True)
            for k in range(new):
                if got[b, k] != ref[k]:
                    gap = np.sort(rows[k])[-1] - np.sort(rows[k])[-2]
                    assert gap < 2e-2, f"sequence {b}, token {k}: top-2 gap {gap:.3g}"
                    break
                compared += 1
        assert compared >= batch * new * 3 // 4, f"only {compared} of {batch * new} tokens were compared before ties"
        # sampled: accepted guesses and rejections mix, so the roll-back is ragged; each sequence against its own oracle run
        out, stats = eng.generate(prompts, new, gamma, 1.0, 23)
        draft = Decoder(dcfg, dw)
        compared = 0
        for b in range(batch):
            ref = oracle_generate.speculative_generate(target, draft, prompts[b], new, gamma, 1.0, 23, sequence=b)
            diff = next((k for k in range(new) if out[b, k] != ref.tokens[k]), None)
            if diff is not None:
                index = len(prompts[b]) + diff
                it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
                assert min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins)) < 5e-3, f"sequence {b}, token {diff}"
            compared += new if diff is None else diff
        assert compared >= batch * new // 2, f"only {compared} of {batch * new} tokens were compared before flagged decisions"
        assert 0 < stats["tests_passed"] < stats["tests_evaluated"]
    finally:
        eng.close()


def test_gpt_97m_and_6m_pair_at_full_size_matches_the_oracle():
    """The GPT-like pair of the paper's Section 4.2 shapes at full size (97M-parameter target, 6M-parameter draft with
    tied embeddings, bf16), as the benchmark runs it: 128-token prompt, gamma = 5.  The oracle is fast enough here to
    follow the free-running stream."""
    tcfg, tw, dcfg, dw = _models("gpt97m_target", "gpt6m_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=1, max_len=128 + 64, page_size=64, max_gamma=5)
    prompt = workloads.make_prompt(77, 128, tcfg["vocab"])
    try:
        for temperature in (1.0, 0.0):
            flagged, iters = compare_generation(eng, Decoder(tcfg, tw), Decoder(dcfg, dw), prompt, 32, 5, temperature,
                                                seed=8, margin=5e-3, logit_tol=5e-3)
            assert flagged <= 3, f"{flagged} flagged of {iters}"
    finally:
        eng.close()


def test_statistics_are_consistent(tiny):
    eng, _, _, cfg = tiny
    prompt = workloads.make_prompt(4, 12, cfg["vocab"])
    out, st = eng.generate([prompt], 60, 3, 1.0, 1)
    assert out.shape == (1, 60) and out.min() >= 0 and out.max() < cfg["vocab"]
    assert st["tokens"] == st["iterations"] + st["tests_passed"]          # n + 1 tokens per iteration
    assert st["tests_passed"] <= st["tests_evaluated"] <= 3 * st["iterations"]
    assert 60 <= st["tokens"] <= 60 + 3 and st["target_passes"] >= st["iterations"]
    assert st["decode_ms"] > 0 and st["prefill_ms"] >= 0
    hist = st["accepted_histogram"]
    assert sum(hist) == st["iterations"] and sum(n * c for n, c in enumerate(hist)) == st["tests_passed"]
    assert not any(hist[4:])  # gamma = 3: n <= 3
    again, _ = eng.generate([prompt], 60, 3, 1.0, 1)
    assert np.array_equal(out, again)  # same seed, same tokens
    other, _ = eng.generate([prompt], 60, 3, 1.0, 2)
    assert not np.array_equal(out, other)


def test_phased_generation_equals_the_single_call(tiny):
    eng, _, _, cfg = tiny
    prompts = [workloads.make_prompt(31, 7, cfg["vocab"]), workloads.make_prompt(32, 12, cfg["vocab"])]
    whole, st = eng.generate(prompts, 30, 3, 1.0, 9)
    eng.begin(prompts, 30, 3, 1.0, 9)
    remaining, steps = 30, 0
    while remaining > 0:
        remaining, part = eng.step(2)
        steps += 2
        assert part["target_passes"] == steps and part["decode_ms"] > 0
    assert np.array_equal(eng.read_tokens(), whole)
    assert part["tokens"] == st["tokens"] and part["tests_passed"] == st["tests_passed"]
    # a diagnostic call ends the generation in progress
    eng.reset()
    with pytest.raises(binding.SpecError):
        eng.step(1)


def test_imposed_acceptance_is_iid_with_the_chosen_rate(tiny):
    """The timing instrument: n follows the capped geometric law of Section 3.1
    (Eq. 1) for the imposed alpha, independent of the models."""
    from oracle import analysis
    eng, _, _, cfg = tiny
    prompt = workloads.make_prompt(10, 6, cfg["vocab"])
    gamma = 4
    try:
        for alpha in (0.0, 0.7, 1.0):
            eng.set_imposed_acceptance(alpha)
            total = {"iterations": 0, "tokens": 0, "tests_evaluated": 0, "tests_passed": 0}
            for seed in range(8):
                _, stats = eng.generate([prompt], 100, gamma, 1.0, seed)
                for k in total:
                    total[k] += stats[k]
            per_iteration = total["tokens"] / total["iterations"]
            if alpha in (0.0, 1.0):
                assert per_iteration == (1 if alpha == 0.0 else gamma + 1)
                continue
            rate = total["tests_passed"] / total["tests_evaluated"]
            sigma = (alpha * (1 - alpha) / total["tests_evaluated"]) ** 0.5
            assert abs(rate - alpha) < 4 * sigma
            assert abs(per_iteration - analysis.expected_tokens(alpha, gamma)) < 0.25
    finally:
        eng.set_imposed_acceptance(None)
    a, _ = eng.generate([prompt], 20, gamma, 1.0, 3)
    b, _ = eng.generate([prompt], 20, gamma, 1.0, 3)
    assert np.array_equal(a, b)


def test_lenient_generation_matches_the_oracle_and_accepts_more(tiny):
    """Appendix A.5 through the whole loop: token stream equal to the oracle's with the
    same lenience, and a higher acceptance rate than the strict run."""
    eng, target, draft, cfg = tiny
    prompt = workloads.make_prompt(12, 10, cfg["vocab"])
    try:
        eng.set_lenience(0.2)
        ref = oracle_generate.speculative_generate(target, draft, prompt, 48, 3, 1.0, seed=21, lenience=0.2)
        got, lenient = eng.generate([prompt], 48, 3, 1.0, 21)
        got = got[0].tolist()
        diff = next((k for k in range(48) if got[k] != ref.tokens[k]), None)
        if diff is not None:  # a decision within tolerance of a boundary ends the comparison
            index = len(prompt) + diff
            it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
            assert min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins)) < 1e-3
            assert diff >= MIN_COMPARED, f"only {diff} tokens were compared before a tolerance-flagged decision"
        with pytest.raises(binding.SpecError):
            eng.set_lenience(1.5)
    finally:
        eng.set_lenience(1.0)
    _, strict = eng.generate([prompt], 48, 3, 1.0, 21)
    assert lenient["tests_passed"] / lenient["tests_evaluated"] > strict["tests_passed"] / strict["tests_evaluated"]


@pytest.mark.parametrize("gamma,top_p", [(3, 1.0), (0, 1.0), (3, 0.8), (0, 0.8)])
def test_truncated_generation_matches_the_oracle(tiny, gamma, top_p):
    """Section 2.2's top-k through the whole loop (gamma = 0: target-only decoding from the
    target's top-k distribution): token stream equal to the oracle's with the same k, every
    emitted token inside the target's top-k set, and a stream that differs from the uncut one."""
    eng, target, draft, cfg = tiny
    prompt = workloads.make_prompt(14, 10, cfg["vocab"])
    k = 6
    try:
        eng.set_truncation(k, top_p)
        if gamma:
            ref = oracle_generate.speculative_generate(target, draft, prompt, 48, gamma, 1.0, seed=23, top_k=k, top_p=top_p, keep_logits=True)
            want, records = ref.tokens, ref.iterations
        else:
            want, rows, margins = oracle_generate.target_only_generate(target, prompt, 48, 1.0, seed=23, top_k=k, top_p=top_p, keep_logits=True)
        got, _ = eng.generate([prompt], 48, gamma, 1.0, 23)
        got = got[0].tolist()
        diff = next((i for i in range(48) if got[i] != want[i]), None)
        if diff is not None:  # a decision, or the k-th largest logit, within tolerance of a boundary
            if gamma:
                index = len(prompt) + diff
                it = next(i for i in records if i.start_len <= index <= i.start_len + i.n_accepted)
                logits = np.concatenate([it.target_logits, it.draft_logits])
                margin = min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins))
            else:
                logits, margin = rows[diff][None], margins[diff]
            ordered = np.sort(logits, axis=1)
            cut_gap = float((ordered[:, -k] - ordered[:, -k - 1]).min())
            from oracle.sampling import nucleus_floor
            mass_gap = min(nucleus_floor(r, 1.0, k, top_p)[1] for r in logits)
            assert margin < 1e-3 or cut_gap < 1e-3 or mass_gap < 1e-3
        checked = diff if diff is not None else 48
        assert checked >= 8
        # every token up to the first difference lies in the top-k set of the oracle's target row
        if gamma == 0 and top_p == 1.0:
            for i in range(checked):
                assert rows[i][got[i]] >= np.sort(rows[i])[-k]
        with pytest.raises(binding.SpecError):
            eng.set_truncation(-1, 1.0)
    finally:
        eng.set_truncation(0, 1.0)
    uncut, _ = eng.generate([prompt], 48, gamma, 1.0, 23)
    assert uncut[0].tolist() != got


@pytest.mark.parametrize("temperature", [1.0, 0.0])
def test_bigram_table_draft_matches_the_oracle(temperature):
    """The tiny fp32 target with a bigram table as its draft (no draft passes at all)."""
    from oracle.ngram import BigramTable
    tcfg = workloads.model_config("tiny_target")
    tw = workloads.make_weights(tcfg, 1)
    dcfg = workloads.model_config("bigram_8k")
    dw = workloads.make_weights(dcfg, 2)
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=2, max_len=96, page_size=32, max_gamma=4)
    try:
        prompt = workloads.make_prompt(13, 12, tcfg["vocab"])
        flagged, iters = compare_generation(eng, Decoder(tcfg, tw), BigramTable(dw["table"]), prompt, 48, 3, temperature,
                                            seed=17, margin=1e-3, logit_tol=1e-3)
        assert flagged <= 2
        # a ragged batch of two runs, and greedy equals target-only greedy
        prompts = [prompt, workloads.make_prompt(14, 5, tcfg["vocab"])]
        greedy, _ = eng.generate(prompts, 24, 0, 0.0, 0)
        spec, stats = eng.generate(prompts, 24, 4, 0.0, 0)
        assert np.array_equal(greedy, spec) and stats["draft_passes"] > 0
    finally:
        eng.close()


@pytest.mark.parametrize("ngram", [2, 1, 3])
def test_copy_from_context_draft_matches_the_oracle(ngram):
    """The tiny fp32 target with the parameter-less copy draft.  With a random-init target a
    guess is almost never accepted, so the guesses themselves would go unseen: argmax decoding
    with a vanishing lenience factor accepts every guess (Appendix A.5 at T = 0), and the
    emitted stream is then the draft's guesses interleaved with the target's tokens."""
    from oracle.ngram import CopyFromContext
    tcfg = workloads.model_config("tiny_target")
    tw = workloads.make_weights(tcfg, 1)
    dcfg = workloads.scaled_config(workloads.model_config("copy_8k"), ngram=ngram)
    eng = binding.Engine(tcfg, tw, dcfg, {}, max_batch=2, max_len=160, page_size=32, max_gamma=4)
    target, draft = Decoder(tcfg, tw), CopyFromContext(tcfg["vocab"], ngram)
    try:
        prompt = workloads.make_repetitive_prompt(15, 26, tcfg["vocab"], 7)
        eng.set_lenience(1e-30)
        ref = oracle_generate.speculative_generate(target, draft, prompt, 60, 3, 0.0, seed=0, lenience=1e-30)
        assert ref.tests_passed == ref.tests_evaluated  # every guess shows in the stream
        got, st = eng.generate([prompt], 60, 3, 0.0, 0)
        assert st["tests_passed"] == st["tests_evaluated"]
        got = got[0].tolist()
        diff = next((k for k in range(60) if got[k] != ref.tokens[k]), None)
        if diff is not None:  # only a near-tie of the target's two best logits may end the comparison
            index = len(prompt) + diff
            it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
            assert index == it.start_len + it.n_accepted and it.top2_gap <= 2e-3 and diff >= 12
        # the first iteration copies the next three tokens of the period
        assert got[:3] == [int(t) for t in np.tile(prompt[:7], 8)[26:29]]
        eng.set_lenience(1.0)
        # T = 1 decisions as the oracle's, T = 0 strict equals target-only greedy, in a ragged batch
        flagged, _ = compare_generation(eng, target, draft, prompt, 40, 3, 1.0, seed=19, margin=1e-3, logit_tol=1e-3)
        assert flagged <= 2
        prompts = [prompt, workloads.make_repetitive_prompt(16, 9, tcfg["vocab"], 3)]
        greedy, _ = eng.generate(prompts, 24, 0, 0.0, 0)
        spec, stats = eng.generate(prompts, 24, 4, 0.0, 0)
        assert np.array_equal(greedy, spec) and stats["draft_passes"] > 0
        with pytest.raises(binding.SpecError):
            eng.forward_logits(1, np.zeros((1, 1), dtype=np.int32))
    finally:
        eng.set_lenience(1.0)
        eng.close()


def test_adaptive_gamma_generation(tiny):
    """Section 3.5's varying gamma: the library picks gamma burst by burst.  The trace it reports,
    replayed by the oracle (and by the phased entry points), gives the same tokens; at T = 0 the
    output is the target's greedy decoding whatever the trace."""
    eng, target, draft, cfg = tiny
    prompt = workloads.make_prompt(41, 10, cfg["vocab"])
    n_new, gamma_max = 72, 6
    got, st, trace = eng.generate_adaptive([prompt], n_new, gamma_max, 1.0, 29, burst=3)
    got = got[0].tolist()
    assert trace[0][0] == 1 and trace[1][0] == gamma_max and all(1 <= g <= gamma_max for g, _ in trace)
    assert sum(n for _, n in trace) == st["iterations"] == st["target_passes"]
    assert sum(g * n for g, n in trace) == st["draft_passes"]
    schedule = [g for g, n in trace for _ in range(n)]
    ref = oracle_generate.speculative_generate(target, draft, prompt, n_new, schedule, 1.0, seed=29)
    diff = next((k for k in range(n_new) if got[k] != ref.tokens[k]), None)
    if diff is not None:  # a decision within tolerance of a boundary ends the comparison
        index = len(prompt) + diff
        it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
        assert min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins)) < 1e-3
        assert diff >= 8
    # the same trace through spec_begin / spec_set_gamma / spec_step
    eng.begin([prompt], n_new, gamma_max, 1.0, 29)
    for g, n in trace:
        eng.set_gamma(g)
        eng.step(n)
    assert eng.read_tokens()[0].tolist() == got
    with pytest.raises(binding.SpecError):
        eng.set_gamma(0)
    with pytest.raises(binding.SpecError):
        eng.set_gamma(gamma_max + 1)
    # T = 0: the target's greedy output, in a ragged batch
    prompts = [prompt, workloads.make_prompt(42, 5, cfg["vocab"])]
    greedy, _ = eng.generate(prompts, 40, 0, 0.0, 1)
    adaptive, _, trace0 = eng.generate_adaptive(prompts, 40, gamma_max, 0.0, 1, burst=2)
    assert np.array_equal(adaptive, greedy) and len({g for g, _ in trace0}) >= 2
