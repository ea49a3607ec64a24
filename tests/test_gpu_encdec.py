"""The encoder-decoder (T5-shaped) path through the C ABI against the CPU oracle:
teacher-forced logits of both models after an encoder pass over ragged sources,
roll-back, free-running generation, and the T = 0 guarantee (abstract; Section 2.2)."""
import numpy as np
import pytest

from oracle import generate as oracle_generate
from oracle.encdec import START_TOKEN, EncoderDecoder
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _pair(target_name, draft_name):
    tcfg, dcfg = workloads.model_config(target_name), workloads.model_config(draft_name)
    return tcfg, workloads.make_weights(tcfg, 1), dcfg, workloads.make_weights(dcfg, 2)


@pytest.fixture(scope="module")
def tiny():
    tcfg, tw, dcfg, dw = _pair("t5_tiny_target", "t5_tiny_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=3, max_len=96, page_size=32, max_gamma=5, max_src_len=80)
    yield eng, (tcfg, tw), (dcfg, dw)
    eng.close()


def _sources(vocab, lengths, seed=21):
    return [workloads.make_prompt(seed + i, n, vocab) for i, n in enumerate(lengths)]


def _check_rows(got, want, tol, relative):
    got = got.cpu().numpy().astype(np.float64)
    for r in range(want.shape[0]):
        err = np.abs(got[r] - want[r]).max()
        bound = tol * np.abs(want[r]).max() if relative else tol
        assert err <= bound, f"row {r}: max error {err:.3g} > {bound:.3g}"


def _teacher_forced(eng, models, lengths, tol, relative):
    vocab = models[0][0]["vocab"]
    sources = _sources(vocab, lengths)
    eng.encode(sources)
    for which, (cfg, w) in enumerate(models):
        oracles = []
        for s in sources:
            o = EncoderDecoder(cfg, w)
            o.encode(s)
            oracles.append(o)
        tokens = np.stack([np.concatenate([[START_TOKEN], workloads.make_prompt(40 + b, 10, vocab)]) for b in range(len(sources))])
        # four rows, three more, roll two back and feed four others (what a rejection does)
        first = eng.forward_logits(which, tokens[:, :4])
        second = eng.forward_logits(which, tokens[:, 4:7])
        eng.truncate(which, [5] * len(sources))
        third = eng.forward_logits(which, tokens[:, 7:11])
        for b, o in enumerate(oracles):
            _check_rows(first[b], o.forward_rows(tokens[b, :4]), tol, relative)
            _check_rows(second[b], o.forward_rows(tokens[b, 4:7]), tol, relative)
            o.truncate(5)
            _check_rows(third[b], o.forward_rows(tokens[b, 7:11]), tol, relative)


def test_teacher_forced_logits_fp32(tiny):
    """Ragged sources that span several KV pages and 32-key tiles; both models."""
    eng, target, draft = tiny
    _teacher_forced(eng, (target, draft), [37, 80, 5], 1e-4, True)


def test_teacher_forced_logits_bf16():
    tcfg, tw, dcfg, dw = _pair("t5_test_target", "t5_test_draft")
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=2, max_len=64, page_size=32, max_gamma=3, max_src_len=150)
    try:
        _teacher_forced(eng, ((tcfg, tw), (dcfg, dw)), [150, 33], 2e-2, False)
    finally:
        eng.close()


def test_teacher_forced_logits_of_the_t5_small_shape_at_full_size():
    """The benchmark's draft for the encoder-decoder pair at full size (6 + 6 blocks, d 512, 8 heads, vocabulary
    32128), here as the only model of a context: sources of 96 and 40 tokens."""
    cfg = workloads.model_config("t5small_draft")
    w = workloads.make_weights(cfg, 6)
    eng = binding.Engine(cfg, w, max_batch=2, max_len=64, page_size=32, max_gamma=3, max_src_len=96)
    try:
        _teacher_forced(eng, ((cfg, w),), [96, 40], 2e-2, False)
    finally:
        eng.close()


def _first_difference(got, want):
    return next((k for k in range(len(want)) if got[k] != want[k]), None)


@pytest.mark.parametrize("temperature", [1.0, 0.0])
def test_generation_matches_the_oracle(tiny, temperature):
    """Free-running, gamma = 3.  The decoder cannot be restarted from a given prefix
    through the ABI (its prompt is the start token), so the streams are compared up
    to the first decision that sat within tolerance of a boundary."""
    eng, (tcfg, tw), (dcfg, dw) = tiny
    target, draft = EncoderDecoder(tcfg, tw), EncoderDecoder(dcfg, dw)
    compared = 0
    for trial in range(3):
        source = workloads.make_prompt(60 + trial, 41, tcfg["vocab"])
        target.encode(source)
        draft.encode(source)
        ref = oracle_generate.speculative_generate(target, draft, [START_TOKEN], 40, 3, temperature, seed=13 + trial)
        got, stats = eng.generate([source], 40, 3, temperature, 13 + trial)
        got = got[0].tolist()
        diff = _first_difference(got, ref.tokens)
        if diff is None:
            compared += 40
            continue
        index = 1 + diff
        it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
        if temperature > 0:
            close = min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins)) < 1e-3
        else:
            close = it.top2_gap <= 2e-3
        assert close, f"trial {trial} token {index}: gpu {got[diff]} oracle {ref.tokens[diff]}"
        compared += diff
    assert compared >= 60, f"only {compared} tokens compared before boundary decisions"


@pytest.mark.parametrize("gamma", [1, 2, 5])
def test_temperature_zero_equals_target_only_greedy(tiny, gamma):
    eng, (tcfg, _), _ = tiny
    sources = _sources(tcfg["vocab"], [30, 64, 11], seed=77)
    greedy, _ = eng.generate(sources, 32, 0, 0.0, 0)
    spec, stats = eng.generate(sources, 32, gamma, 0.0, 0)
    assert np.array_equal(greedy, spec)
    # a sequence decodes the same alone as in the ragged batch
    alone, _ = eng.generate([sources[1]], 32, gamma, 0.0, 0)
    assert np.array_equal(alone[0], spec[1])
    assert stats["iterations"] >= 3 * 32 / (gamma + 1)


def test_adaptive_gamma_and_truncation_on_the_encoder_decoder(tiny):
    """The options of the generation loop on this model family too: gamma chosen by the library
    (T = 0: still the target's greedy output), and top-k / nucleus against the oracle at T = 1."""
    eng, (tcfg, tw), (dcfg, dw) = tiny
    sources = _sources(tcfg["vocab"], [30, 64, 11], seed=78)
    greedy, _ = eng.generate(sources, 32, 0, 0.0, 0)
    adaptive, stats, trace = eng.generate_adaptive(sources, 32, 5, 0.0, 0, burst=2)
    assert np.array_equal(greedy, adaptive) and len({g for g, _ in trace}) >= 2
    assert sum(n for _, n in trace) == stats["target_passes"]
    target, draft = EncoderDecoder(tcfg, tw), EncoderDecoder(dcfg, dw)
    target.encode(sources[0])
    draft.encode(sources[0])
    try:
        eng.set_truncation(8, 0.9)
        ref = oracle_generate.speculative_generate(target, draft, [START_TOKEN], 40, 3, 1.0, seed=5, top_k=8, top_p=0.9)
        got, _ = eng.generate([sources[0]], 40, 3, 1.0, 5)
        got = got[0].tolist()
        diff = next((i for i in range(40) if got[i] != ref.tokens[i]), 40)
        assert diff >= 10, f"streams differ at token {diff}"  # (a boundary decision may end the comparison later on)
    finally:
        eng.set_truncation(0, 1.0)


def test_errors(tiny):
    eng, (tcfg, tw), _ = tiny
    with pytest.raises(binding.SpecError) as e:
        eng.encode([workloads.make_prompt(1, 81, tcfg["vocab"])])
    assert e.value.status == -4  # SPEC_ERR_CAPACITY
    eng.reset()
    eng.encode([workloads.make_prompt(1, 8, tcfg["vocab"])])
    with pytest.raises(binding.SpecError):  # only one sequence is encoded
        eng.forward_logits(0, np.zeros((2, 1), dtype=np.int32))
    gcfg = workloads.model_config("tiny_draft")
    plain = binding.Engine(gcfg, workloads.make_weights(gcfg, 3), max_batch=1, max_len=32, page_size=32, max_gamma=0)
    try:
        with pytest.raises(binding.SpecError) as e:
            plain.encode([np.array([1, 2, 3], dtype=np.int32)])
        assert e.value.status == -2  # SPEC_ERR_BAD_CONFIG
    finally:
        plain.close()
    with pytest.raises(binding.SpecError) as e:  # an encoder-decoder context needs max_src_len
        binding.Engine(tcfg, tw, max_batch=1, max_len=32, page_size=32, max_gamma=0)
    assert e.value.status == -2  # SPEC_ERR_BAD_CONFIG
