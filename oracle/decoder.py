"""The decoder-only model families of the synthetic configs, on the CPU.

Test infrastructure (see the package docstring).

The paper fixes only sizes (a GPT-like Transformer decoder with GELU, given
dims; T5 names) and treats M_p and M_q as black boxes that map a prefix to a
next-token distribution (Section 2.1).  The architecture below is therefore
this build's own definition, stated here once:

* pre-RMSNorm blocks: h += Wo . attn(rmsnorm(h)); h += W_out . act(W_in . rmsnorm(h));
  logits = W_head . rmsnorm(h).  rmsnorm(x) = x / sqrt(mean(x^2) + eps) * gain.
  No biases anywhere.
* attention: causal, softmax(q.k / sqrt(d_head)) in full precision, n_heads
  query heads over n_kv_heads key/value heads (query head h reads KV head
  h // (n_heads // n_kv_heads)).
* arch "gpt": h_0 = tok_emb[token] + pos_emb[position]; FFN "gelu" with the
  tanh approximation.
* arch "llama": h_0 = tok_emb[token]; rotary positions on q and k in the
  rotate-half convention (pairs j, j + d_head/2; angle position * base^(-2j/d_head));
  FFN "swiglu": silu(gate) * up with W_in = [gate rows; up rows].
  FFN "gated_gelu" is the same with gelu on the gate.
* tied = True reuses tok_emb as W_head.

Weights arrive as a dict of arrays (see `paper_2211_17192_b200.workloads` for
the seeded generator and the tensor names); this module never draws them.

Pins (tests/test_oracle_decoder.py): the architecture is ours, so there is no
printed value to match.  What is pinned: the cached path equals the
cache-free path (which recomputes the whole prefix, so it cannot carry a
stale row); logits at row j do not change when later rows change (causal
mask); with all block weights zero the logits reduce to the closed form
W_head . rmsnorm(embedding); one layer with hand-checkable weights;
rotary attention scores depend only on relative position; grouped KV heads
equal the same model with the KV heads physically repeated.  Beyond that:
parity unpinned (oracle-versus-CUDA agreement only).
"""

import numpy as np


def rmsnorm(x, gain, eps):
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def gelu_tanh(x):
    return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x * x * x)))


def silu(x):
    return x / (1.0 + np.exp(-x))


def rope(x, positions, base):
    """x [rows, heads, d_head]; rotate-half convention."""
    half = x.shape[-1] // 2
    j = np.arange(half, dtype=np.float64)
    inv_freq = base ** (-2.0 * j / x.shape[-1])
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]
    cos = np.cos(ang)[:, None, :].astype(x.dtype)
    sin = np.sin(ang)[:, None, :].astype(x.dtype)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


class Decoder:
    """One model (target or draft) with an optional KV cache for one sequence."""

    def __init__(self, cfg, weights, dtype=np.float64):
        self.cfg = dict(cfg)
        self.dtype = dtype
        self.w = {k: np.asarray(v, dtype=dtype) for k, v in weights.items()}
        c = self.cfg
        self.group = c["n_heads"] // c["n_kv_heads"]
        self.reset()

    # -- cache ---------------------------------------------------------------
    def reset(self):
        c = self.cfg
        self.k_cache = [np.zeros((0, c["n_kv_heads"], c["d_head"]), dtype=self.dtype) for _ in range(c["n_layers"])]
        self.v_cache = [np.zeros((0, c["n_kv_heads"], c["d_head"]), dtype=self.dtype) for _ in range(c["n_layers"])]

    @property
    def cached_len(self):
        return self.k_cache[0].shape[0]

    def truncate(self, length):
        """Roll the cache back to `length` rows (drops the speculative rows)."""
        for l in range(self.cfg["n_layers"]):
            self.k_cache[l] = self.k_cache[l][:length]
            self.v_cache[l] = self.v_cache[l][:length]

    # -- forward -------------------------------------------------------------
    def forward_rows(self, tokens):
        """Feed `tokens` at positions cached_len.. and append their K,V rows.

        Returns logits [len(tokens), vocab]: row j is the next-token logits
        after the prefix that ends with tokens[j].
        """
        start = self.cached_len
        positions = np.arange(start, start + len(tokens))
        return self._forward(np.asarray(tokens), positions, use_cache=True)

    def forward_full(self, tokens, last=None):
        """Cache-free: the whole sequence from position 0, nothing kept.  With `last`
        given, only the logits of the last `last` rows are formed and returned (the
        LM head of the earlier rows is skipped; nothing else changes)."""
        saved = (self.k_cache, self.v_cache)
        self.reset()
        out = self._forward(np.asarray(tokens), np.arange(len(tokens)), use_cache=True, last=last)
        self.k_cache, self.v_cache = saved
        return out

    def _forward(self, tokens, positions, use_cache, last=None):
        c, w = self.cfg, self.w
        H, Hkv, dh = c["n_heads"], c["n_kv_heads"], c["d_head"]
        m = len(tokens)
        h = w["tok_emb"][tokens].copy()
        if c["arch"] == "gpt":
            h = h + w["pos_emb"][positions]
        scale = 1.0 / np.sqrt(dh)
        for l in range(c["n_layers"]):
            a = rmsnorm(h, w[f"l{l}.ln1"], c["rms_eps"])
            qkv = a @ w[f"l{l}.wqkv"].T
            q = qkv[:, : H * dh].reshape(m, H, dh)
            k = qkv[:, H * dh : (H + Hkv) * dh].reshape(m, Hkv, dh)
            v = qkv[:, (H + Hkv) * dh :].reshape(m, Hkv, dh)
            if c["arch"] == "llama":
                q = rope(q, positions, c["rope_base"])
                k = rope(k, positions, c["rope_base"])
            self.k_cache[l] = np.concatenate([self.k_cache[l], k], axis=0)
            self.v_cache[l] = np.concatenate([self.v_cache[l], v], axis=0)
            K, Vv = self.k_cache[l], self.v_cache[l]
            o = np.zeros((m, H, dh), dtype=self.dtype)
            for head in range(H):
                kv = head // self.group
                s = (q[:, head, :] @ K[:, kv, :].T) * scale  # [m, cached]
                key_pos = np.arange(K.shape[0])
                s = np.where(key_pos[None, :] <= positions[:, None], s, -np.inf)
                s = s - s.max(axis=-1, keepdims=True)
                e = np.exp(s)
                o[:, head, :] = (e / e.sum(axis=-1, keepdims=True)) @ Vv[:, kv, :]
            h = h + o.reshape(m, H * dh) @ w[f"l{l}.wo"].T
            b = rmsnorm(h, w[f"l{l}.ln2"], c["rms_eps"])
            u = b @ w[f"l{l}.w_in"].T
            F = c["d_ff"]
            if c["ffn"] == "gelu":
                f = gelu_tanh(u)
            elif c["ffn"] == "gated_gelu":
                f = gelu_tanh(u[:, :F]) * u[:, F:]
            elif c["ffn"] == "swiglu":
                f = silu(u[:, :F]) * u[:, F:]
            else:
                raise ValueError(c["ffn"])
            h = h + f @ w[f"l{l}.w_out"].T
        if last is not None:
            h = h[len(tokens) - last:]
        hf = rmsnorm(h, w["ln_f"], c["rms_eps"])
        head = w["tok_emb"] if c["tied"] else w["head"]
        return hf @ head.T
