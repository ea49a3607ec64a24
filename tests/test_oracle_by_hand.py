"""Hand-written scalar walk-throughs of one block of each gated FFN kind and of a one-block
encoder-decoder (d = 2, one head, two source tokens): every intermediate is formed with plain
Python floats and loops over explicit indices, no matrix routine and none of the oracle's
helpers, so that a transposed operand, a swapped gate/up half, a misplaced gain, a bias read
at the wrong offset or rotary positions applied to the wrong tensor in `oracle.decoder` /
`oracle.encdec` changes the comparison."""
import math

import numpy as np
import pytest

from oracle.decoder import Decoder
from oracle.encdec import EncoderDecoder


def matvec(W, x):
    return [sum(W[i][j] * x[j] for j in range(len(x))) for i in range(len(W))]


def rms_norm(x, gain):
    r = math.sqrt(sum(v * v for v in x) / len(x))
    return [v / r * g for v, g in zip(x, gain)]


def gelu(x):
    return 0.5 * x * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))


def silu(x):
    return x / (1.0 + math.exp(-x))


def attend(q, keys, values, biases):
    """softmax(q.k / sqrt(d) + bias) over the given keys, times the values."""
    d = len(q)
    scores = [sum(a * b for a, b in zip(q, k)) / math.sqrt(d) + bias for k, bias in zip(keys, biases)]
    top = max(scores)
    e = [math.exp(s - top) for s in scores]
    return [sum(e[j] * values[j][i] for j in range(len(keys))) / sum(e) for i in range(d)]


def add(a, b):
    return [x + y for x, y in zip(a, b)]


EMB = [[1.0, 0.0], [0.0, 2.0], [1.0, 1.0]]
WQ, WK, WV = [[1.0, 0.0], [0.0, 1.0]], [[0.0, 1.0], [1.0, 0.0]], [[2.0, 0.0], [0.0, 2.0]]
WO = [[1.0, 1.0], [0.0, 1.0]]
W_IN = [[1.0, 0.0], [0.0, 1.0], [2.0, 0.0], [0.0, 3.0]]   # rows 0-1 the gate, rows 2-3 the up projection
W_OUT = [[1.0, 0.0], [1.0, 1.0]]
LN1, LN2, LNF = [1.0, 0.5], [2.0, 1.0], [1.0, 3.0]


def gated_ffn(x, act):
    u = matvec(W_IN, x)
    return matvec(W_OUT, [act(u[0]) * u[2], act(u[1]) * u[3]])


@pytest.mark.parametrize("ffn,act", [("swiglu", silu), ("gated_gelu", gelu)])
def test_gated_block_with_rotary_positions_by_hand(ffn, act):
    """Two tokens through one rotary block: q and k of row 1 are turned by one radian, v is not."""
    cfg = dict(arch="llama", ffn=ffn, n_layers=1, d_model=2, n_heads=1, n_kv_heads=1, d_head=2, d_ff=2,
               vocab=3, max_positions=4, tied=True, rms_eps=0.0, rope_base=1e4, dtype="fp32")
    w = {"tok_emb": np.array(EMB), "l0.ln1": np.array(LN1), "l0.wqkv": np.array(WQ + WK + WV), "l0.wo": np.array(WO),
         "l0.ln2": np.array(LN2), "l0.w_in": np.array(W_IN), "l0.w_out": np.array(W_OUT), "ln_f": np.array(LNF)}
    out = Decoder(cfg, w).forward_full([1, 2])

    def turn(x, angle):  # the pair (0, 1) of a 2-wide head rotates by `angle`
        return [x[0] * math.cos(angle) - x[1] * math.sin(angle), x[1] * math.cos(angle) + x[0] * math.sin(angle)]

    h = [EMB[1], EMB[2]]
    a = [rms_norm(x, LN1) for x in h]
    q = [turn(matvec(WQ, a[p]), float(p)) for p in range(2)]
    k = [turn(matvec(WK, a[p]), float(p)) for p in range(2)]
    v = [matvec(WV, a[p]) for p in range(2)]
    att = [attend(q[0], k[:1], v[:1], [0.0]), attend(q[1], k, v, [0.0, 0.0])]
    h = [add(h[p], matvec(WO, att[p])) for p in range(2)]
    h = [add(h[p], gated_ffn(rms_norm(h[p], LN2), act)) for p in range(2)]
    ref = [matvec(EMB, rms_norm(h[p], LNF)) for p in range(2)]
    assert np.allclose(out, np.array(ref), atol=1e-13)


def test_one_block_encoder_decoder_by_hand():
    """Source of two tokens, decoder rows [start, 2]: encoder self-attention with the mirrored
    bias buckets, cross K,V from the normalised encoder output, causal decoder self-attention
    with the backward buckets, cross-attention without bias, gated-GELU FFNs."""
    enc_bias = [0.0, 0.5, -0.5, 1.0]   # bucket -> bias (one head); 4 buckets, far distance 8
    dec_bias = [0.25, -0.75, 0.1, 0.2]
    WQX, WKVX, WOX = [[0.0, 1.0], [1.0, 0.0]], [[1.0, 0.0], [0.0, 1.0], [0.0, 3.0], [1.0, 0.0]], [[1.0, 0.0], [2.0, 1.0]]
    HEAD = [[1.0, 2.0], [0.5, -1.0], [0.0, 1.0]]
    LNX, ENC_LNF = [1.0, 2.0], [0.5, 1.0]
    cfg = dict(arch="t5", ffn="gated_gelu", n_layers=1, n_enc_layers=1, d_model=2, n_heads=1, n_kv_heads=1, d_head=2,
               d_ff=2, vocab=3, max_positions=8, tied=False, rms_eps=0.0, rope_base=1e4, dtype="fp32",
               rel_buckets=4, rel_max_distance=8)
    block = {"ln1": np.array(LN1), "wqkv": np.array(WQ + WK + WV), "wo": np.array(WO), "ln2": np.array(LN2),
             "w_in": np.array(W_IN), "w_out": np.array(W_OUT)}
    w = {"tok_emb": np.array(EMB), "enc.rel_bias": np.array(enc_bias)[:, None], "rel_bias": np.array(dec_bias)[:, None],
         "enc.ln_f": np.array(ENC_LNF), "ln_f": np.array(LNF), "head": np.array(HEAD),
         "l0.lnx": np.array(LNX), "l0.wq_x": np.array(WQX), "l0.wkv_x": np.array(WKVX), "l0.wo_x": np.array(WOX)}
    for name, value in block.items():
        w["enc.l0." + name] = value
        w["l0." + name] = value
    model = EncoderDecoder(cfg, w)
    memory = model.encode([1, 2])
    out = model.forward_full([0, 2])

    # encoder: with 4 buckets in two mirrored halves, distance 0 is bucket 0, the key one step
    # before the query bucket 1, the key one step after it bucket 3
    h = [EMB[1], EMB[2]]
    a = [rms_norm(x, LN1) for x in h]
    q, k, v = ([matvec(W, x) for x in a] for W in (WQ, WK, WV))
    att = [attend(q[0], k, v, [enc_bias[0], enc_bias[3]]), attend(q[1], k, v, [enc_bias[1], enc_bias[0]])]
    h = [add(h[p], matvec(WO, att[p])) for p in range(2)]
    h = [add(h[p], gated_ffn(rms_norm(h[p], LN2), gelu)) for p in range(2)]
    mem = [rms_norm(x, ENC_LNF) for x in h]
    assert np.allclose(memory, np.array(mem), atol=1e-13)
    cross = [matvec(WKVX, x) for x in mem]
    ck, cv = [c[:2] for c in cross], [c[2:] for c in cross]

    # decoder: backward buckets only: distance 0 is bucket 0, one step back bucket 1
    h = [EMB[0], EMB[2]]
    a = [rms_norm(x, LN1) for x in h]
    q, k, v = ([matvec(W, x) for x in a] for W in (WQ, WK, WV))
    att = [attend(q[0], k[:1], v[:1], [dec_bias[0]]), attend(q[1], k, v, [dec_bias[1], dec_bias[0]])]
    h = [add(h[p], matvec(WO, att[p])) for p in range(2)]
    qx = [matvec(WQX, rms_norm(x, LNX)) for x in h]
    h = [add(h[p], matvec(WOX, attend(qx[p], ck, cv, [0.0, 0.0]))) for p in range(2)]
    h = [add(h[p], gated_ffn(rms_norm(h[p], LN2), gelu)) for p in range(2)]
    ref = [matvec(HEAD, rms_norm(x, LNF)) for x in h]
    assert np.allclose(out, np.array(ref), atol=1e-13)
