"""Pins for oracle.decoder.  The architecture is this build's own definition, so
these are structural: cached equals cache-free, causality, closed-form special
cases, rotary relativity, grouped-KV equivalence."""
import numpy as np
import pytest

from oracle.decoder import Decoder, gelu_tanh, rmsnorm, rope, silu
from paper_2211_17192_b200 import workloads


def _small(arch, **kw):
    cfg = workloads.model_config("tiny_draft" if arch == "gpt" else "llama_test_target")
    cfg = workloads.scaled_config(cfg, vocab=97, max_positions=64, **kw)
    return cfg, workloads.make_weights(cfg, 5)


@pytest.mark.parametrize("arch", ["gpt", "llama"])
def test_cached_equals_cache_free_with_rollback(arch):
    cfg, w = _small(arch)
    model = Decoder(cfg, w)
    tokens = workloads.make_prompt(1, 20, cfg["vocab"])
    full = model.forward_full(tokens)
    model.reset()
    a = model.forward_rows(tokens[:7])
    junk = model.forward_rows([3, 1, 4, 1])  # speculative rows, then rolled back
    model.truncate(7)
    b = model.forward_rows(tokens[7:12])
    c = model.forward_rows(tokens[12:])
    assert np.allclose(np.concatenate([a, b, c]), full, atol=1e-11)
    assert junk.shape == (4, cfg["vocab"]) and model.cached_len == 20


@pytest.mark.parametrize("arch", ["gpt", "llama"])
def test_causality(arch):
    cfg, w = _small(arch)
    model = Decoder(cfg, w)
    tokens = workloads.make_prompt(2, 12, cfg["vocab"])
    other = tokens.copy()
    other[8:] = (other[8:] + 1) % cfg["vocab"]
    a, b = model.forward_full(tokens), model.forward_full(other)
    assert np.array_equal(a[:8], b[:8])
    assert not np.allclose(a[8:], b[8:])


def test_zero_blocks_reduce_to_the_embedding_readout():
    cfg, w = _small("gpt")
    for name in w:
        if ".wo" in name or ".w_out" in name:
            w[name] = np.zeros_like(w[name])
    model = Decoder(cfg, w)
    tokens = np.array([5, 9, 5])
    h = w["tok_emb"][tokens].astype(np.float64) + w["pos_emb"][:3].astype(np.float64)
    h = h / np.sqrt((h * h).mean(-1, keepdims=True) + cfg["rms_eps"])
    assert np.allclose(model.forward_full(tokens), h @ w["head"].astype(np.float64).T, atol=1e-12)


def test_single_layer_by_hand():
    """One layer, one head, d = 2: every intermediate written out explicitly."""
    cfg = dict(arch="gpt", ffn="gelu", n_layers=1, d_model=2, n_heads=1, n_kv_heads=1, d_head=2, d_ff=2,
               vocab=3, max_positions=4, tied=True, rms_eps=0.0, rope_base=1e4, dtype="fp32")
    eye = np.eye(2)
    w = {"tok_emb": np.array([[1.0, 0.0], [0.0, 2.0], [1.0, 1.0]]), "pos_emb": np.zeros((4, 2)),
         "l0.ln1": np.ones(2), "l0.wqkv": np.concatenate([eye, eye, eye]), "l0.wo": eye,
         "l0.ln2": np.ones(2), "l0.w_in": eye, "l0.w_out": 2 * eye, "ln_f": np.ones(2)}
    out = Decoder(cfg, w).forward_full([0, 1])
    s2 = np.sqrt(2.0)
    a0, a1 = np.array([s2, 0.0]), np.array([0.0, s2])  # rmsnorm of the two embeddings
    # row 0 attends to itself only; row 1 to both with scores (0, 2)/sqrt(2)
    e = np.exp(np.array([0.0, 2.0 / s2]) - 2.0 / s2)
    att1 = (e[0] * a0 + e[1] * a1) / e.sum()
    h0 = np.array([1.0, 0.0]) + a0
    h1 = np.array([0.0, 2.0]) + att1
    def block2(h):
        b = h / np.sqrt((h * h).mean())
        return h + 2 * gelu_tanh(b)
    h0, h1 = block2(h0), block2(h1)
    ref = np.stack([h / np.sqrt((h * h).mean()) for h in (h0, h1)]) @ w["tok_emb"].T
    assert np.allclose(out, ref, atol=1e-13)


def test_elementwise_functions():
    x = np.array([-3.0, -0.5, 0.0, 0.7, 4.0])
    # tanh-GELU is within 1e-3 of the exact erf GELU, odd part is x/2
    from scipy.special import erf
    assert np.allclose(gelu_tanh(x), 0.5 * x * (1 + erf(x / np.sqrt(2))), atol=1e-3)
    assert np.allclose(gelu_tanh(x) - gelu_tanh(-x), x, atol=1e-14)
    assert np.allclose(silu(x), x * (1 / (1 + np.exp(-x))))
    assert np.allclose(silu(x) - silu(-x), x, atol=1e-14)
    v = np.array([[3.0, 4.0]])
    assert np.allclose(rmsnorm(v, np.array([1.0, 2.0]), 0.0), [[3 / np.sqrt(12.5), 8 / np.sqrt(12.5)]])


def test_rotary_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(0)
    q, k = rng.normal(size=(1, 1, 8)), rng.normal(size=(1, 1, 8))
    def score(pq, pk):
        return float((rope(q, [pq], 1e4) * rope(k, [pk], 1e4)).sum())
    assert score(5, 2) == pytest.approx(score(105, 102), abs=1e-11)
    assert score(0, 0) == pytest.approx(float((q * k).sum()), abs=1e-13)
    assert abs(score(5, 2) - score(5, 3)) > 1e-3
    # norm preserving; position 0 is the identity
    assert np.allclose(np.linalg.norm(rope(q, [17], 1e4)), np.linalg.norm(q))
    assert np.allclose(rope(q, [0], 1e4), q)
    # first pair (j = 0) rotates by exactly `position` radians
    x = np.zeros((1, 1, 8)); x[0, 0, 0] = 1.0
    y = rope(x, [2], 1e4)[0, 0]
    assert y[0] == pytest.approx(np.cos(2.0)) and y[4] == pytest.approx(np.sin(2.0))


def test_grouped_kv_equals_repeated_kv_heads():
    cfg, w = _small("llama")  # 4 query heads over 2 KV heads
    H, Hkv, dh = cfg["n_heads"], cfg["n_kv_heads"], cfg["d_head"]
    wide_cfg = workloads.scaled_config(cfg, n_kv_heads=H)
    wide = dict(w)
    for l in range(cfg["n_layers"]):
        m = w[f"l{l}.wqkv"]
        qw, kw, vw = m[: H * dh], m[H * dh : (H + Hkv) * dh], m[(H + Hkv) * dh :]
        rep = lambda a: np.repeat(a.reshape(Hkv, dh, -1), H // Hkv, axis=0).reshape(H * dh, -1)
        wide[f"l{l}.wqkv"] = np.concatenate([qw, rep(kw), rep(vw)])
    tokens = workloads.make_prompt(3, 9, cfg["vocab"])
    assert np.allclose(Decoder(cfg, w).forward_full(tokens), Decoder(wide_cfg, wide).forward_full(tokens), atol=1e-11)


def test_fp32_mode_tracks_fp64():
    cfg, w = _small("llama")
    tokens = workloads.make_prompt(4, 16, cfg["vocab"])
    a = Decoder(cfg, w, dtype=np.float64).forward_full(tokens)
    b = Decoder(cfg, w, dtype=np.float32).forward_full(tokens)
    assert np.abs(a - b).max() < 1e-4 * np.abs(a).max()
