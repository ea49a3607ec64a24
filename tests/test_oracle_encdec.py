"""Pins of the encoder-decoder oracle (oracle/encdec.py); CPU only.

The architecture is this build's own definition, so nothing printed in the
paper can be matched.  Pinned instead: the bucket function against an
all-integer restatement and its defining properties; closed forms with zeroed
weights; cached versus cache-free decoding; mask and set-function invariances
of the three attention kinds; and, through the generation loop, the paper's
guarantee that speculative decoding at T = 0 returns the target's greedy
output (abstract; Section 2.2) for this model family too.
"""

import numpy as np
import pytest

from oracle import generate
from oracle.decoder import rmsnorm
from oracle.encdec import START_TOKEN, EncoderDecoder, relative_bucket
from paper_2211_17192_b200 import workloads


def bucket_by_integers(delta, bidirectional, n_buckets, max_distance):
    """The same bucket from comparisons of integers only (no logarithm)."""
    if bidirectional:
        n = n_buckets // 2
        base = n if delta > 0 else 0
        dist = abs(delta)
    else:
        n = n_buckets
        base = 0
        dist = max(-delta, 0)
    exact = n // 2
    if dist < exact:
        return base + dist
    # largest k with (dist / exact)^(n - exact) >= (max_distance / exact)^k
    k = 0
    while dist ** (n - exact) * exact ** (k + 1) >= max_distance ** (k + 1) * exact ** (n - exact):
        k += 1
    return base + min(exact + k, n - 1)


@pytest.mark.parametrize("bidirectional", [True, False])
@pytest.mark.parametrize("n_buckets,max_distance", [(32, 128), (16, 64), (32, 100)])
def test_bucket_matches_the_integer_restatement(bidirectional, n_buckets, max_distance):
    deltas = np.arange(-400, 401)
    got = relative_bucket(deltas, bidirectional, n_buckets, max_distance)
    want = [bucket_by_integers(int(d), bidirectional, n_buckets, max_distance) for d in deltas]
    assert got.tolist() == want


def test_bucket_properties():
    back = relative_bucket(-np.arange(0, 1000), False, 32, 128)
    assert back[0] == 0 and back.max() == 31 and np.all(np.diff(back) >= 0)
    assert back[:16].tolist() == list(range(16))  # one bucket per distance below n/2
    assert np.all(back[128:] == 31)  # everything at or beyond max_distance shares the last bucket
    assert np.all(relative_bucket(np.arange(1, 50), False, 32, 128) == 0)  # the decoder never looks ahead
    both = relative_bucket(np.arange(-300, 301), True, 32, 128)
    assert both.min() == 0 and both.max() == 31
    before, after = both[:300][::-1], both[301:]
    assert np.array_equal(after, before + 16)  # mirrored halves
    assert after[:8].tolist() == list(range(17, 25))


def tiny(seed=1):
    cfg = workloads.model_config("t5_tiny_target")
    return cfg, workloads.make_weights(cfg, seed)


def test_cached_decoding_equals_cache_free():
    cfg, w = tiny()
    m = EncoderDecoder(cfg, w)
    m.encode(workloads.make_prompt(3, 17, cfg["vocab"]))
    tokens = [START_TOKEN] + workloads.make_prompt(4, 9, cfg["vocab"]).tolist()
    full = m.forward_full(tokens)
    m.reset()
    pieces = [m.forward_rows(tokens[:1]), m.forward_rows(tokens[1:4]), m.forward_rows(tokens[4:])]
    assert np.allclose(np.concatenate(pieces), full, atol=1e-12)
    # roll back three rows, feed other tokens, roll back again and re-feed the originals
    m.truncate(7)
    m.forward_rows([1, 2, 3])
    m.truncate(7)
    again = m.forward_rows(tokens[7:])
    assert np.allclose(again, full[7:], atol=1e-12)


def test_causal_mask_and_encoder_visibility():
    cfg, w = tiny()
    m = EncoderDecoder(cfg, w)
    src = workloads.make_prompt(5, 12, cfg["vocab"])
    m.encode(src)
    a = m.forward_full([0, 5, 6, 7, 8])
    b = m.forward_full([0, 5, 6, 99, 100])
    assert np.allclose(a[:3], b[:3], atol=1e-12) and not np.allclose(a[3:], b[3:], atol=1e-6)
    # every decoder row sees every source position: changing the last source token changes row 0
    src2 = src.copy()
    src2[-1] = (src2[-1] + 1) % cfg["vocab"]
    m.encode(src2)
    assert not np.allclose(m.forward_full([0, 5, 6, 7, 8])[0], a[0], atol=1e-6)


def test_zero_blocks_reduce_to_the_closed_form():
    cfg, w = tiny()
    for name in w:
        if name.endswith(("wo", "w_out", "wo_x")):
            w[name] = np.zeros_like(w[name])
    m = EncoderDecoder(cfg, w)
    m.encode([1, 2, 3])
    tokens = np.array([0, 9, 4])
    want = rmsnorm(w["tok_emb"][tokens].astype(np.float64), 1.0, cfg["rms_eps"]) @ w["head"].astype(np.float64).T
    assert np.allclose(m.forward_full(tokens), want, atol=1e-12)


def test_cross_attention_over_one_source_token_returns_its_value_row():
    cfg = workloads.scaled_config(workloads.model_config("t5_tiny_target"), n_layers=1)
    w = workloads.make_weights(cfg, 7)
    m = EncoderDecoder(cfg, w)
    memory = m.encode([11])
    logits = m.forward_full([0, 3])
    # softmax over a single key is 1: the cross term is Wo_x . V_x whatever the query projection is
    w2 = dict(w)
    w2["l0.wq_x"] = w["l0.wq_x"] * 0.0 + 0.3
    m2 = EncoderDecoder(cfg, w2)
    m2.encode([11])
    assert np.allclose(m2.forward_full([0, 3]), logits, atol=1e-12)
    # and the value row is the lower half of Wkv_x applied to the encoder output
    H, dh = cfg["n_heads"], cfg["d_head"]
    v = memory[0] @ w["l0.wkv_x"].astype(np.float64).T[:, H * dh :]
    assert np.allclose(m.cross_v[0].reshape(-1), v, atol=1e-12)


def test_decoder_is_a_set_function_of_the_source_when_the_encoder_bias_is_flat():
    cfg, w = tiny()
    w["enc.rel_bias"] = np.full_like(w["enc.rel_bias"], 0.25)
    src = workloads.make_prompt(8, 10, cfg["vocab"])
    m = EncoderDecoder(cfg, w)
    m.encode(src)
    a = m.forward_full([0, 1, 2])
    m.encode(src[::-1].copy())
    assert np.allclose(m.forward_full([0, 1, 2]), a, atol=1e-10)
    # with the drawn table the order of the source matters
    cfg, w = tiny()
    m = EncoderDecoder(cfg, w)
    m.encode(src)
    a = m.forward_full([0, 1, 2])
    m.encode(src[::-1].copy())
    assert not np.allclose(m.forward_full([0, 1, 2]), a, atol=1e-6)


def test_decoder_bias_enters_the_self_attention_scores():
    cfg, w = tiny()
    m = EncoderDecoder(cfg, w)
    m.encode([4, 5, 6])
    a = m.forward_full([0, 1, 2, 3])
    w2 = dict(w)
    w2["rel_bias"] = w["rel_bias"].astype(np.float64) + 1.0  # a constant shift cancels in the softmax
    m2 = EncoderDecoder(cfg, w2)
    m2.encode([4, 5, 6])
    assert np.allclose(m2.forward_full([0, 1, 2, 3]), a, atol=1e-10)
    w2["rel_bias"] = w["rel_bias"].copy()
    w2["rel_bias"][1] += 1.0  # distance 1 only
    m3 = EncoderDecoder(cfg, w2)
    m3.encode([4, 5, 6])
    b = m3.forward_full([0, 1, 2, 3])
    assert np.allclose(b[0], a[0], atol=1e-12)  # row 0 has no key at distance 1
    assert not np.allclose(b[1:], a[1:], atol=1e-6)


def test_fp32_agrees_with_fp64():
    cfg, w = tiny()
    src = workloads.make_prompt(9, 16, cfg["vocab"])
    m64, m32 = EncoderDecoder(cfg, w), EncoderDecoder(cfg, w, dtype=np.float32)
    m64.encode(src)
    m32.encode(src)
    tokens = [0] + workloads.make_prompt(10, 7, cfg["vocab"]).tolist()
    assert np.abs(m64.forward_full(tokens) - m32.forward_full(tokens)).max() < 2e-4


@pytest.mark.parametrize("gamma", [1, 3])
def test_greedy_speculative_output_equals_target_greedy(gamma):
    tcfg, dcfg = workloads.model_config("t5_tiny_target"), workloads.model_config("t5_tiny_draft")
    target = EncoderDecoder(tcfg, workloads.make_weights(tcfg, 1))
    draft = EncoderDecoder(dcfg, workloads.make_weights(dcfg, 2))
    src = workloads.make_prompt(11, 14, tcfg["vocab"])
    target.encode(src)
    draft.encode(src)
    want, _, _ = generate.target_only_generate(target, [START_TOKEN], 12, 0.0, seed=5)
    got = generate.speculative_generate(target, draft, [START_TOKEN], 12, gamma, 0.0, seed=5)
    assert got.tokens == want
    uncached = generate.speculative_generate(target, draft, [START_TOKEN], 12, gamma, 1.0, seed=5, cached=False)
    cached = generate.speculative_generate(target, draft, [START_TOKEN], 12, gamma, 1.0, seed=5, cached=True)
    assert uncached.tokens == cached.tokens
