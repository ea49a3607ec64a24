"""The persistent pass kernel (spec_runtime_cfg::pass_kernel = 1: a pass of at most 16 rows of a
bf16 GPT- or Llama-shaped model as one cooperative kernel) against the CPU oracle, through the
C ABI: teacher-forced logits with roll-back, a ragged batch, free-running generation by
Algorithm 1, bit-identical repeats, and the barrier trace."""
import numpy as np
import pytest

from gpu_util import compare_generation
from oracle.decoder import Decoder
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu

BF16_ABS = 2e-2  # max |delta| per logit against the oracle on the same bf16-rounded weights


def _pair(name, seed=1, **overrides):
    cfg = workloads.scaled_config(workloads.model_config(name), **overrides)
    return cfg, workloads.make_weights(cfg, seed)


@pytest.mark.parametrize("name,overrides", [
    ("llama_test_target", {}),                                          # grouped KV heads, rotary, SwiGLU; matrices with fewer units than CTAs
    ("llama_test_draft", {}),
    ("gpt97m_target", {"n_layers": 3}),                                 # learned positions, GELU
    ("gpt6m_draft", {}),                                                # tied embeddings
    ("llama160m_draft", {"n_layers": 2, "vocab": 4096}),
    ("llama7b_target", {"n_layers": 1, "vocab": 4096, "d_ff": 2752}),   # d_head 128; tiles shared by several CTAs
])
def test_teacher_forced_logits_with_rollback(name, overrides):
    cfg, w = _pair(name, **overrides)
    oracle = Decoder(cfg, w)
    eng = binding.Engine(cfg, w, max_batch=1, max_len=128, page_size=32, max_gamma=10, pass_kernel=True)
    try:
        tokens = workloads.make_prompt(3, 60, cfg["vocab"])
        ref = oracle.forward_full(tokens)
        eng.reset()
        got = [eng.forward_logits(0, tokens[None, :9]).cpu().numpy()[0]]
        eng.forward_logits(0, workloads.make_prompt(4, 6, cfg["vocab"])[None, :])   # speculative rows ...
        eng.truncate(0, [9])                                                          # ... rolled back
        got.append(eng.forward_logits(0, tokens[None, 9:25]).cpu().numpy()[0])        # 16 rows: the most the kernel takes
        got.append(eng.forward_logits(0, tokens[None, 25:26]).cpu().numpy()[0])       # one row
        for at in range(26, 60, 3):                                                  # verification-sized passes across pages
            got.append(eng.forward_logits(0, tokens[None, at:at + 3]).cpu().numpy()[0])
        assert binding.spec_device_error() == 0
        err = np.abs(np.concatenate(got).astype(np.float64) - ref[:np.concatenate(got).shape[0]]).max()
        assert err <= BF16_ABS, f"max absolute logit error {err:.3g}"
    finally:
        eng.close()


def test_ragged_batch_and_identical_repeats():
    cfg, w = _pair("llama_test_target")
    seqs = [workloads.make_prompt(10 + b, 40, cfg["vocab"]) for b in range(4)]
    ref = [Decoder(cfg, w).forward_full(s) for s in seqs]
    runs = []
    for _ in range(2):
        eng = binding.Engine(cfg, w, max_batch=4, max_len=64, page_size=32, max_gamma=3, pass_kernel=True)
        try:
            eng.reset()
            a = eng.forward_logits(0, np.stack([s[:4] for s in seqs])).cpu().numpy()
            b = eng.forward_logits(0, np.stack([s[4:8] for s in seqs])).cpu().numpy()
            eng.truncate(0, [8, 5, 2, 7])                      # ragged roll-back, then three rows each from there
            tails = [seqs[0][8:11], seqs[1][5:8], seqs[2][2:5], seqs[3][7:10]]
            c = eng.forward_logits(0, np.stack(tails)).cpu().numpy()
            runs.append((a, b, c))
        finally:
            eng.close()
    a, b, c = runs[0]
    for i, start in enumerate([8, 5, 2, 7]):
        assert np.abs(a[i] - ref[i][:4]).max() <= BF16_ABS and np.abs(b[i] - ref[i][4:8]).max() <= BF16_ABS
        assert np.abs(c[i] - ref[i][start:start + 3]).max() <= BF16_ABS
    for x, y in zip(runs[0], runs[1]):   # the parts of a tile are added in a fixed order: no run-to-run difference
        assert np.array_equal(x, y)


@pytest.mark.parametrize("temperature,gamma", [(1.0, 3), (0.0, 2)])
def test_generation_matches_the_oracle(temperature, gamma):
    tcfg, tw = _pair("llama_test_target")
    dcfg, dw = _pair("llama_test_draft", seed=2)
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=1, max_len=128, page_size=32, max_gamma=4, pass_kernel=True)
    try:
        prompt = workloads.make_prompt(7, 12, tcfg["vocab"])
        flagged, iterations = compare_generation(eng, Decoder(tcfg, tw), Decoder(dcfg, dw), prompt, 40, gamma, temperature, 11,
                                                 margin=5e-3, logit_tol=BF16_ABS)
        assert iterations >= 10 and flagged <= 3
    finally:
        eng.close()


def test_barrier_trace_and_refusals():
    cfg, w = _pair("llama_test_target")
    eng = binding.Engine(cfg, w, max_batch=1, max_len=64, page_size=32, max_gamma=3, pass_kernel=True)
    try:
        eng.forward_logits(0, workloads.make_prompt(5, 20, cfg["vocab"])[None, :16])
        start, arrivals = eng.pass_trace(0, 1, 3)
        assert arrivals.shape[0] == 1 + 7 * cfg["n_layers"] and arrivals.shape[1] >= 1   # embed, then seven steps per block
        assert (arrivals >= start).all()
        assert (arrivals[1:].min(axis=1) >= arrivals[:-1].max(axis=1)).all()              # nobody passes a barrier early
        with pytest.raises(binding.SpecError):
            eng.pass_trace(0, 1, 70)  # more rows than the workspace holds
    finally:
        eng.close()
    plain = binding.Engine(cfg, w, max_batch=1, max_len=64, page_size=32, max_gamma=3)
    try:
        with pytest.raises(binding.SpecError) as e:
            plain.pass_trace(0, 1, 3)   # the context runs the kernel chain
        assert e.value.status == -2
    finally:
        plain.close()
