"""Parity at the shapes and launch configurations the benchmark runs (Algorithm 1's
parallel pass of M_p; the premise of Section 3.4 that gamma + 1 rows share one stream
of the weights): a one-block model of the full 7B width with more than 1024 cached
tokens, at batch 1 (3 and 7 rows) and at batch 16 with ragged lengths and a ragged
roll-back; the benchmark's GEMM shapes against the plain definition in fp64; and
the encoder-decoder's cross-attention over a 512-token source.  Every case also
checks, through `spec_attention_plan`, that the kernel variant it means to cover
is the one the library chose."""
import numpy as np
import pytest
import torch

from oracle.decoder import Decoder
from oracle.encdec import START_TOKEN, EncoderDecoder
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu

BF16_ABS = 2e-2   # max |delta| per logit against the oracle on the same bf16-rounded weights
MAX_LEN = 1284    # the benchmark's cache capacity at gamma = 2: 1024-token prompt + 256 new + gamma + 2


@pytest.fixture(scope="module")
def wide_block():
    """One block of the 7B shape at full width: d 4096, 32 query / 8 KV heads of 128, FFN 11008, vocab 32000."""
    cfg = workloads.scaled_config(workloads.model_config("llama7b_target"), n_layers=1)
    w = workloads.make_weights(cfg, 11)
    return cfg, w, Decoder(cfg, w, dtype=np.float32)


def _feed(eng, which, tokens, step):
    """Teacher-forces tokens [B, n] in passes of `step` rows; returns the logits of every pass."""
    outs = []
    for at in range(0, tokens.shape[1], step):
        outs.append(eng.forward_logits(which, tokens[:, at:at + step]).cpu().numpy())
    return outs


def test_long_context_verify_rows_at_batch_one(wide_block):
    """1030 cached tokens, then 3 rows (gamma = 2) and 7 rows (gamma = 6): the tensor-core attention
    with more key slices than a cluster merges (separate combine kernel, K and V staged side by
    side), the 22016 x 4096, 4096 x 11008 and 32000 x 4096 GEMMs with their real split-K."""
    cfg, w, oracle = wide_block
    eng = binding.Engine(cfg, w, max_batch=1, max_len=MAX_LEN, page_size=64, max_gamma=6)
    try:
        for rows in (3, 7):
            plan = eng.attention_plan(0, 1, rows)
            assert plan["tensor_cores"] and not plan["cluster_merge"] and not plan["in_turn"] and plan["slices"] > 8, plan
        tokens = workloads.make_prompt(5, 1040, cfg["vocab"])[None, :]
        eng.reset()
        chunks = _feed(eng, 0, tokens[:, :1030], 64)         # 16 passes of 64 rows and one of 6
        three = eng.forward_logits(0, tokens[:, 1030:1033]).cpu().numpy()
        seven = eng.forward_logits(0, tokens[:, 1033:1040]).cpu().numpy()
        assert binding.spec_device_error() == 0
        ref = oracle.forward_full(tokens[0], last=80)        # rows 960 .. 1039
        got = np.concatenate([chunks[15][0], chunks[16][0], three[0], seven[0]])
        err = np.abs(got.astype(np.float64) - ref).max(axis=-1)
        assert err.max() <= BF16_ABS, f"max absolute logit error {err.max():.3g} at row {960 + int(err.argmax())}"
    finally:
        eng.close()


_RAGGED_ORACLE = {}


@pytest.mark.parametrize("kv_dtype", ["fp16", "fp32"])
def test_ragged_batch_of_sixteen_with_rollback(wide_block, kv_dtype):
    """16 sequences x 5 rows over ragged cached lengths (453 .. 1008 tokens), then a ragged roll-back
    (0 .. 4 of the 5 rows kept) and 5 more rows, 80-row GEMM tiles.  fp16 rows (the default): the f16
    tensor-core attention, the 20 queries of a KV head in one CTA, two key slices merged in a cluster.
    fp32 rows: the tf32 tensor-core attention with K and V staged in turn, two 16-query blocks per KV head."""
    cfg, w, oracle = wide_block
    B, rows = 16, 5
    eng = binding.Engine(cfg, w, max_batch=B, max_len=MAX_LEN, page_size=64, max_gamma=15, kv_dtype=kv_dtype)
    try:
        plan = eng.attention_plan(0, B, rows)
        if kv_dtype == "fp16":
            assert plan["f16"] and plan["cluster_merge"] and plan["slices"] == 2, plan
        else:
            assert plan["tensor_cores"] and not plan["f16"] and plan["in_turn"], plan
        seqs = np.stack([workloads.make_prompt(100 + b, 1008 + 2 * rows, cfg["vocab"]) for b in range(B)])
        eng.reset()
        _feed(eng, 0, seqs[:, :1008], 16)
        lengths = [1008 - 37 * b for b in range(B)]
        eng.truncate(0, lengths)
        first = np.stack([seqs[b, 1008:1008 + rows] for b in range(B)])
        got1 = eng.forward_logits(0, first).cpu().numpy()
        keep = [(3 * b + 1) % rows for b in range(B)]          # rows of the first pass that stay cached
        eng.truncate(0, [lengths[b] + keep[b] for b in range(B)])
        second = np.stack([seqs[b, 1008 + rows:1008 + 2 * rows] for b in range(B)])
        got2 = eng.forward_logits(0, second).cpu().numpy()
        assert binding.spec_device_error() == 0
        worst = 0.0
        for b in (0, 3, 6, 9, 12, 15):                         # the oracle is slow at this width: six of the sixteen
            if b not in _RAGGED_ORACLE:                        # (the same for both cache types)
                _RAGGED_ORACLE[b] = (
                    oracle.forward_full(np.concatenate([seqs[b, :lengths[b]], first[b]]), last=rows),
                    oracle.forward_full(np.concatenate([seqs[b, :lengths[b]], first[b, :keep[b]], second[b]]), last=rows))
            a, c = _RAGGED_ORACLE[b]
            worst = max(worst, np.abs(got1[b] - a).max(), np.abs(got2[b] - c).max())
        assert worst <= BF16_ABS, f"max absolute logit error {worst:.3g}"
    finally:
        eng.close()


@pytest.mark.parametrize("rows,n_out,k", [(3, 22016, 4096), (3, 4096, 11008), (3, 32000, 4096), (7, 6144, 4096),
                                          (224, 4096, 11008), (224, 22016, 4096), (6, 32128, 4096),
                                          (6, 20480, 4096), (6, 4096, 10240)])
def test_benchmark_gemm_shapes_against_the_plain_definition(rows, n_out, k):
    """y = x W^T at the target models' own matrix shapes (tile-major weights, the engine's
    split-K) against numpy in fp64."""
    rng = np.random.default_rng(rows * 100003 + n_out + k)
    x = rng.standard_normal((rows, k)).astype(np.float32)
    w = workloads.round_to_bf16(rng.standard_normal((n_out, k)).astype(np.float32) * 0.02)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    xd = torch.from_numpy(x).cuda()
    packed = binding.spec_pack_weight(torch.from_numpy(w).cuda().to(torch.bfloat16))
    got = binding.spec_linear(xd, packed, "tensor_packed", n_out=n_out).cpu().numpy()
    assert binding.spec_device_error() == 0
    assert np.abs(got - ref).max() <= 1e-4 * np.abs(ref).max()


def test_cross_attention_over_a_long_source_on_the_tensor_cores():
    """Six decoder rows of eight sequences over sources of up to 512 tokens: the cross-attention
    (and here the self-attention too, with its relative-position bias) takes the f16 tensor-core kernel."""
    cfg = workloads.model_config("t5_test_target")
    w = workloads.make_weights(cfg, 1)
    B, rows = 8, 6
    eng = binding.Engine(cfg, w, max_batch=B, max_len=512, page_size=64, max_gamma=rows - 1, max_src_len=512)
    try:
        assert eng.attention_plan(0, B, rows, cross=True)["f16"]
        assert eng.attention_plan(0, B, rows)["f16"]
        sources = [workloads.make_prompt(300 + b, n, cfg["vocab"]) for b, n in enumerate([512, 509, 480, 333, 257, 129, 64, 7])]
        eng.encode(sources)
        tokens = np.stack([np.concatenate([[START_TOKEN], workloads.make_prompt(400 + b, 2 * rows - 1, cfg["vocab"])])
                           for b in range(B)])
        got = [eng.forward_logits(0, tokens[:, :rows]).cpu().numpy(), eng.forward_logits(0, tokens[:, rows:]).cpu().numpy()]
        assert binding.spec_device_error() == 0
        worst = 0.0
        for b in range(B):
            o = EncoderDecoder(cfg, w)
            o.encode(sources[b])
            worst = max(worst, np.abs(got[0][b] - o.forward_rows(tokens[b, :rows])).max(),
                        np.abs(got[1][b] - o.forward_rows(tokens[b, rows:])).max())
        assert worst <= BF16_ABS, f"max absolute logit error {worst:.3g}"
    finally:
        eng.close()


def test_one_row_steps_of_a_batch_over_a_long_source_on_the_tensor_cores():
    """A draft step of an encoder-decoder in a batch: one decoder row for each of 32 sequences (one query per head,
    128 (sequence, head) pairs), sources of up to 512 tokens; both the cross-attention and the biased self-attention
    take the f16 tensor-core kernel.  Five steps, four of the sequences against the oracle."""
    cfg = workloads.model_config("t5_test_target")
    w = workloads.make_weights(cfg, 1)
    B, steps = 32, 5
    eng = binding.Engine(cfg, w, max_batch=B, max_len=512, page_size=64, max_gamma=1, max_src_len=512)
    try:
        assert eng.attention_plan(0, B, 1, cross=True)["f16"]
        assert eng.attention_plan(0, B, 1)["f16"]
        lengths = [512 - 16 * b for b in range(B)]
        sources = [workloads.make_prompt(500 + b, n, cfg["vocab"]) for b, n in enumerate(lengths)]
        eng.encode(sources)
        tokens = np.stack([np.concatenate([[START_TOKEN], workloads.make_prompt(600 + b, steps - 1, cfg["vocab"])])
                           for b in range(B)])
        got = np.stack([eng.forward_logits(0, tokens[:, t:t + 1]).cpu().numpy()[:, 0] for t in range(steps)], axis=1)
        assert binding.spec_device_error() == 0
        worst = 0.0
        for b in (0, 11, 22, 31):
            o = EncoderDecoder(cfg, w)
            o.encode(sources[b])
            worst = max(worst, np.abs(got[b] - o.forward_rows(tokens[b])).max())
        assert worst <= BF16_ABS, f"max absolute logit error {worst:.3g}"
    finally:
        eng.close()
