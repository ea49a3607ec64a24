"""Seeded synthetic inputs: model shapes, random-init weights, prompts, logits.

This module holds none of the method's arithmetic.  It only draws numbers
from numpy's seeded generators, so the CUDA library and the CPU oracle can be
given the very same inputs without sharing any code of their own.  It imports
nothing else from this package.

The inputs stand in for the paper's trained checkpoints and datasets, none of
which are available offline: only the shapes follow the paper (Section 4.2: a
GPT-like 97M target with a 6M draft at an 8k vocabulary) and the benchmark
configs of this repository.
"""

import numpy as np

INIT_STD = 0.02


def model_config(name):
    """Shapes of the synthetic models, by config name."""
    base = dict(rms_eps=1e-6, rope_base=10000.0, tied=False, arch="gpt", ffn="gelu", n_enc_layers=0,
                rel_buckets=32, rel_max_distance=128, bias_std=0.5)
    table = {
        # tiny fp32 pair (correctness config)
        "tiny_target": dict(n_layers=4, d_model=256, n_heads=4, n_kv_heads=4, d_head=64, d_ff=1024,
                            vocab=8192, max_positions=128, dtype="fp32", head_std=3.0 / 16.0),
        "tiny_draft": dict(n_layers=2, d_model=128, n_heads=2, n_kv_heads=2, d_head=64, d_ff=512,
                           vocab=8192, max_positions=128, dtype="fp32", head_std=3.0 / np.sqrt(128.0)),
        # paper-shaped GPT-like pair, bf16
        "gpt97m_target": dict(n_layers=12, d_model=768, n_heads=12, n_kv_heads=12, d_head=64, d_ff=3072,
                              vocab=8192, max_positions=1024, dtype="bf16", head_std=INIT_STD),
        "gpt6m_draft": dict(n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, d_head=64, d_ff=1024,
                            vocab=8192, max_positions=1024, dtype="bf16", head_std=INIT_STD, tied=True),
        # Llama-shaped serving pair, bf16
        "llama7b_target": dict(arch="llama", ffn="swiglu", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=8,
                               d_head=128, d_ff=11008, vocab=32000, max_positions=2048, dtype="bf16",
                               head_std=INIT_STD),
        "llama160m_draft": dict(arch="llama", ffn="swiglu", n_layers=12, d_model=768, n_heads=12, n_kv_heads=12,
                                d_head=64, d_ff=3072, vocab=32000, max_positions=2048, dtype="bf16",
                                head_std=INIT_STD),
        # small Llama-shaped pair with grouped KV heads, for tests
        "llama_test_target": dict(arch="llama", ffn="swiglu", n_layers=3, d_model=256, n_heads=4, n_kv_heads=2,
                                  d_head=64, d_ff=704, vocab=2048, max_positions=512, dtype="bf16",
                                  head_std=INIT_STD),
        "llama_test_draft": dict(arch="llama", ffn="swiglu", n_layers=1, d_model=128, n_heads=2, n_kv_heads=1,
                                 d_head=64, d_ff=384, vocab=2048, max_positions=512, dtype="bf16",
                                 head_std=INIT_STD),
        # bigram tables: negligible-cost drafts (next-token logits from the last token alone)
        "bigram_8k": dict(arch="bigram", vocab=8192, dtype="fp32", head_std=1.0),
        "bigram_32k": dict(arch="bigram", vocab=32000, dtype="bf16", head_std=0.3),
        # copy-from-context drafts: parameter-less, guess = what followed the last `ngram` tokens before
        "copy_8k": dict(arch="copy", vocab=8192, ngram=2, dtype="fp32"),
        "copy_32k": dict(arch="copy", vocab=32000, ngram=2, dtype="fp32"),
        # T5-shaped encoder-decoder pair (XXL-shaped target, small-shaped draft), bf16
        "t5xxl_target": dict(arch="t5", ffn="gated_gelu", n_layers=24, n_enc_layers=24, d_model=4096, n_heads=64,
                             n_kv_heads=64, d_head=64, d_ff=10240, vocab=32128, max_positions=1024, dtype="bf16",
                             head_std=INIT_STD),
        "t5small_draft": dict(arch="t5", ffn="gated_gelu", n_layers=6, n_enc_layers=6, d_model=512, n_heads=8,
                              n_kv_heads=8, d_head=64, d_ff=2048, vocab=32128, max_positions=1024, dtype="bf16",
                              head_std=INIT_STD),
        # small encoder-decoder pairs for tests
        "t5_test_target": dict(arch="t5", ffn="gated_gelu", n_layers=2, n_enc_layers=2, d_model=256, n_heads=4,
                               n_kv_heads=4, d_head=64, d_ff=512, vocab=2048, max_positions=512, dtype="bf16",
                               head_std=INIT_STD),
        "t5_test_draft": dict(arch="t5", ffn="gated_gelu", n_layers=1, n_enc_layers=1, d_model=128, n_heads=2,
                              n_kv_heads=2, d_head=64, d_ff=256, vocab=2048, max_positions=512, dtype="bf16",
                              head_std=INIT_STD),
        "t5_tiny_target": dict(arch="t5", ffn="gated_gelu", n_layers=2, n_enc_layers=2, d_model=128, n_heads=2,
                               n_kv_heads=2, d_head=64, d_ff=256, vocab=512, max_positions=256, dtype="fp32",
                               head_std=3.0 / np.sqrt(128.0)),
        "t5_tiny_draft": dict(arch="t5", ffn="gated_gelu", n_layers=1, n_enc_layers=1, d_model=64, n_heads=1,
                              n_kv_heads=1, d_head=64, d_ff=128, vocab=512, max_positions=256, dtype="fp32",
                              head_std=3.0 / 8.0),
    }
    cfg = dict(base)
    cfg.update(table[name])
    cfg["name"] = name
    return cfg


def scaled_config(cfg, **overrides):
    """A copy of `cfg` with some fields replaced (reduced depth for big shapes)."""
    out = dict(cfg)
    out.update(overrides)
    return out


def tensor_shapes(cfg):
    """Ordered (name, shape, kind) of a model's tensors; kind is 'gain', 'matrix', 'bias' or 'head'."""
    if cfg["arch"] == "bigram":
        return [("table", (cfg["vocab"], cfg["vocab"]), "head")]
    if cfg["arch"] == "copy":
        return []
    d, H, Hkv, dh, F = cfg["d_model"], cfg["n_heads"], cfg["n_kv_heads"], cfg["d_head"], cfg["d_ff"]
    f_in = F if cfg["ffn"] == "gelu" else 2 * F
    t5 = cfg["arch"] == "t5"
    out = [("tok_emb", (cfg["vocab"], d), "matrix")]
    if cfg["arch"] == "gpt":
        out.append(("pos_emb", (cfg["max_positions"], d), "matrix"))

    def block(prefix):
        return [
            (prefix + "ln1", (d,), "gain"),
            (prefix + "wqkv", ((H + 2 * Hkv) * dh, d), "matrix"),
            (prefix + "wo", (d, H * dh), "matrix"),
            (prefix + "ln2", (d,), "gain"),
            (prefix + "w_in", (f_in, d), "matrix"),
            (prefix + "w_out", (d, F), "matrix"),
        ]

    if t5:  # encoder stack, then the decoder's bias table
        out.append(("enc.rel_bias", (cfg["rel_buckets"], H), "bias"))
        for l in range(cfg["n_enc_layers"]):
            out += block(f"enc.l{l}.")
        out.append(("enc.ln_f", (d,), "gain"))
        out.append(("rel_bias", (cfg["rel_buckets"], H), "bias"))
    for l in range(cfg["n_layers"]):
        out += block(f"l{l}.")
        if t5:  # cross-attention
            out += [
                (f"l{l}.lnx", (d,), "gain"),
                (f"l{l}.wq_x", (H * dh, d), "matrix"),
                (f"l{l}.wkv_x", (2 * H * dh, d), "matrix"),
                (f"l{l}.wo_x", (d, H * dh), "matrix"),
            ]
    out.append(("ln_f", (d,), "gain"))
    if not cfg["tied"]:
        out.append(("head", (cfg["vocab"], d), "head"))
    return out


def round_to_bf16(a):
    """Round fp32 values to the nearest bf16 (ties to even); returns fp32."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def bf16_bits(a):
    """The 16-bit patterns of values that are already bf16-representable."""
    return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def make_weights(cfg, seed):
    """Random-init weights: matrices N(0, 0.02^2), head N(0, head_std^2), relative-position
    bias tables N(0, bias_std^2) (always fp32), gains 1.

    Every tensor has its own generator keyed by (seed, index in tensor_shapes),
    so a tensor's values do not depend on the others.  For dtype "bf16" the
    matrices are rounded to bf16 and returned as fp32 arrays holding those
    values; gains stay fp32.
    """
    weights = {}
    for index, (name, shape, kind) in enumerate(tensor_shapes(cfg)):
        if kind == "gain":
            weights[name] = np.ones(shape, dtype=np.float32)
            continue
        rng = np.random.default_rng([int(seed), index])
        std = cfg["head_std"] if kind == "head" else cfg["bias_std"] if kind == "bias" else INIT_STD
        a = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
        if cfg["dtype"] == "bf16" and kind != "bias":
            a = round_to_bf16(a)
        weights[name] = a
    return weights


def make_prompt(seed, length, vocab):
    """`length` token ids, uniform on [0, vocab)."""
    rng = np.random.default_rng([int(seed), 0x70726F6D])
    return rng.integers(0, vocab, size=length, dtype=np.int64).astype(np.int32)


def make_repetitive_prompt(seed, length, vocab, period):
    """`length` token ids that repeat a uniform segment of `period` tokens (contexts in which long
    stretches recur, the case a copy-from-context draft is meant for)."""
    segment = make_prompt(seed, period, vocab)
    return np.tile(segment, length // period + 1)[:length].copy()


def make_sampler_logits(seed, batch, gamma, vocab, draft_noise, logit_std=3.0):
    """Standalone-sampler inputs: target logits i.i.d. N(0, logit_std^2) of shape
    [batch, gamma+1, vocab]; draft logits = target[:, :gamma] + N(0, draft_noise^2)."""
    rng = np.random.default_rng([int(seed), 0x6C6F67])
    target = rng.standard_normal((batch, gamma + 1, vocab), dtype=np.float32) * np.float32(logit_std)
    noise = rng.standard_normal((batch, gamma, vocab), dtype=np.float32) * np.float32(draft_noise)
    draft = target[:, :gamma, :] + noise
    return target, np.ascontiguousarray(draft)


def make_uniform_grid(seed, shape):
    """Uniforms on the open grid (2k+1)/2^24, k uniform on [0, 2^23): exact in fp32."""
    rng = np.random.default_rng([int(seed), 0x756E69])
    k = rng.integers(0, 1 << 23, size=shape, dtype=np.int64)
    return ((2 * k + 1).astype(np.float64) / float(1 << 24)).astype(np.float32)
