"""The encoder-decoder (T5-shaped) model family of the synthetic configs, on the CPU.

Test infrastructure (see the package docstring).

The paper names T5 v1.1 checkpoints (Section 4.1) and draws them as an encoder
that runs once and a decoder that is called repeatedly (Appendix A.4 figure of
the encoder-decoder case); it gives no architecture details.  The definition
below is this build's own, stated here once.  It follows the decoder family of
`oracle.decoder` wherever the two overlap:

* pre-RMSNorm blocks, no biases, tanh-approximate GELU, gated FFN
  gelu(gate) * up with W_in = [gate rows; up rows], attention scale
  1 / sqrt(d_head) (kept although the original T5 omits it, so that
  random-init scores stay benign), untied LM head, one token embedding shared
  by encoder and decoder, no absolute positions.
* encoder block: h += Wo . attn_full(rmsnorm(h)) ; h += FFN(rmsnorm(h)); the
  output is rmsnorm(h) with gain "enc.ln_f".  attn_full lets every source
  position see every source position.
* decoder block: h += Wo . attn_causal(rmsnorm(h)); h += Wo_x . attn_cross(
  Wq_x . rmsnorm(h), K_x, V_x); h += FFN(rmsnorm(h)), where [K_x; V_x] =
  Wkv_x . (encoder output) is computed once per source and every decoder row
  sees all source positions.
* self-attention scores (encoder and decoder) get an additive bias
  table[bucket(key position - query position), head] after scaling, with one
  table per stack shared by its blocks.  The buckets are the usual
  log-spaced ones: half of them (all of them in the causal decoder, which only
  looks back) hold one distance each, the rest split the distances up to
  `rel_max_distance` evenly in log space, and everything farther shares the
  last bucket.  The encoder uses separate halves for keys after and keys
  before the query.  Cross-attention has no bias.
* decoding starts from token id 0.

Pins (tests/test_oracle_encdec.py): the bucket function against an
all-integer restatement and its defining properties; with zero block weights
the logits are the closed form W_head . rmsnorm(embedding); cached versus
cache-free decoding; causal-mask invariance; the decoder's logits do not
depend on source positions when the cross-attention output projection is zero
and do when it is not; permuting source positions together with a flat bias
table leaves the decoder unchanged (attention is a set function of the
source).  Beyond that: parity unpinned (oracle-versus-CUDA agreement only).
"""

import numpy as np

from .decoder import gelu_tanh, rmsnorm

START_TOKEN = 0


def relative_bucket(delta, bidirectional, n_buckets, max_distance):
    """Bucket of delta = key position - query position (integer array)."""
    delta = np.asarray(delta, dtype=np.int64)
    if bidirectional:
        n = n_buckets // 2
        base = np.where(delta > 0, n, 0)  # keys after the query use the upper half
        dist = np.abs(delta)
    else:
        n = n_buckets
        base = np.zeros_like(delta)
        dist = np.maximum(-delta, 0)  # only keys at or before the query matter
    exact = n // 2  # distances below this have a bucket each
    safe = np.maximum(dist, 1).astype(np.float64)
    spread = np.floor(np.log(safe / exact) / np.log(max_distance / exact) * (n - exact)).astype(np.int64)
    far = np.minimum(exact + spread, n - 1)
    return base + np.where(dist < exact, dist, far)


def _attention(q, K, V, scale, bias, allowed):
    """q [m, H, dh]; K, V [n, H, dh]; bias [H, m, n] or None; allowed [m, n] bool."""
    m, H, dh = q.shape
    out = np.zeros((m, H, dh), dtype=q.dtype)
    for head in range(H):
        s = (q[:, head, :] @ K[:, head, :].T) * scale
        if bias is not None:
            s = s + bias[head]
        s = np.where(allowed, s, -np.inf)
        s = s - s.max(axis=-1, keepdims=True)
        e = np.exp(s)
        out[:, head, :] = (e / e.sum(axis=-1, keepdims=True)) @ V[:, head, :]
    return out


class EncoderDecoder:
    """One model (target or draft): encode a source once, then decode with a KV cache."""

    def __init__(self, cfg, weights, dtype=np.float64):
        self.cfg = dict(cfg)
        self.dtype = dtype
        self.w = {k: np.asarray(v, dtype=dtype) for k, v in weights.items()}
        self.cross_k = self.cross_v = None
        self.reset()

    # -- shared pieces -------------------------------------------------------
    def _ffn(self, x, prefix):
        F = self.cfg["d_ff"]
        u = x @ self.w[prefix + "w_in"].T
        return (gelu_tanh(u[:, :F]) * u[:, F:]) @ self.w[prefix + "w_out"].T

    def _bias(self, table, query_pos, key_pos, bidirectional):
        c = self.cfg
        delta = np.asarray(key_pos)[None, :] - np.asarray(query_pos)[:, None]
        bucket = relative_bucket(delta, bidirectional, c["rel_buckets"], c["rel_max_distance"])
        return np.transpose(table[bucket], (2, 0, 1))  # [H, m, n]

    # -- encoder -------------------------------------------------------------
    def encode(self, source):
        """Run the encoder over `source` token ids and keep the cross-attention K, V."""
        c, w = self.cfg, self.w
        H, dh = c["n_heads"], c["d_head"]
        source = np.asarray(source)
        n = len(source)
        pos = np.arange(n)
        h = w["tok_emb"][source].copy()
        bias = self._bias(w["enc.rel_bias"], pos, pos, True)
        everything = np.ones((n, n), dtype=bool)
        scale = 1.0 / np.sqrt(dh)
        for l in range(c["n_enc_layers"]):
            p = f"enc.l{l}."
            qkv = rmsnorm(h, w[p + "ln1"], c["rms_eps"]) @ w[p + "wqkv"].T
            q, k, v = (qkv[:, i * H * dh : (i + 1) * H * dh].reshape(n, H, dh) for i in range(3))
            h = h + _attention(q, k, v, scale, bias, everything).reshape(n, H * dh) @ w[p + "wo"].T
            h = h + self._ffn(rmsnorm(h, w[p + "ln2"], c["rms_eps"]), p)
        memory = rmsnorm(h, w["enc.ln_f"], c["rms_eps"])
        self.cross_k, self.cross_v = [], []
        for l in range(c["n_layers"]):
            kv = memory @ w[f"l{l}.wkv_x"].T
            self.cross_k.append(kv[:, : H * dh].reshape(n, H, dh))
            self.cross_v.append(kv[:, H * dh :].reshape(n, H, dh))
        self.reset()
        return memory

    # -- decoder cache -------------------------------------------------------
    def reset(self):
        c = self.cfg
        self.k_cache = [np.zeros((0, c["n_heads"], c["d_head"]), dtype=self.dtype) for _ in range(c["n_layers"])]
        self.v_cache = [np.zeros((0, c["n_heads"], c["d_head"]), dtype=self.dtype) for _ in range(c["n_layers"])]

    @property
    def cached_len(self):
        return self.k_cache[0].shape[0]

    def truncate(self, length):
        for l in range(self.cfg["n_layers"]):
            self.k_cache[l] = self.k_cache[l][:length]
            self.v_cache[l] = self.v_cache[l][:length]

    # -- decoder -------------------------------------------------------------
    def forward_rows(self, tokens):
        """Feed decoder `tokens` at positions cached_len.. ; returns their next-token logits."""
        start = self.cached_len
        return self._decode(np.asarray(tokens), np.arange(start, start + len(tokens)))

    def forward_full(self, tokens):
        """Cache-free: the whole decoder sequence from position 0, nothing kept."""
        saved = (self.k_cache, self.v_cache)
        self.reset()
        out = self._decode(np.asarray(tokens), np.arange(len(tokens)))
        self.k_cache, self.v_cache = saved
        return out

    def _decode(self, tokens, positions):
        c, w = self.cfg, self.w
        if self.cross_k is None:
            raise RuntimeError("encode() a source first")
        H, dh = c["n_heads"], c["d_head"]
        m = len(tokens)
        h = w["tok_emb"][tokens].copy()
        scale = 1.0 / np.sqrt(dh)
        n_src = self.cross_k[0].shape[0]
        see_all = np.ones((m, n_src), dtype=bool)
        for l in range(c["n_layers"]):
            p = f"l{l}."
            qkv = rmsnorm(h, w[p + "ln1"], c["rms_eps"]) @ w[p + "wqkv"].T
            q, k, v = (qkv[:, i * H * dh : (i + 1) * H * dh].reshape(m, H, dh) for i in range(3))
            self.k_cache[l] = np.concatenate([self.k_cache[l], k], axis=0)
            self.v_cache[l] = np.concatenate([self.v_cache[l], v], axis=0)
            key_pos = np.arange(self.k_cache[l].shape[0])
            bias = self._bias(w["rel_bias"], positions, key_pos, False)
            causal = key_pos[None, :] <= positions[:, None]
            o = _attention(q, self.k_cache[l], self.v_cache[l], scale, bias, causal)
            h = h + o.reshape(m, H * dh) @ w[p + "wo"].T
            qx = (rmsnorm(h, w[p + "lnx"], c["rms_eps"]) @ w[p + "wq_x"].T).reshape(m, H, dh)
            ox = _attention(qx, self.cross_k[l], self.cross_v[l], scale, None, see_all)
            h = h + ox.reshape(m, H * dh) @ w[p + "wo_x"].T
            h = h + self._ffn(rmsnorm(h, w[p + "ln2"], c["rms_eps"]), p)
        return rmsnorm(h, w["ln_f"], c["rms_eps"]) @ w["head"].T
