"""The f16 tensor-core attention over fp16 K,V rows (the parallel pass of Algorithm 1 for a batch of
sequences: every row of a sequence attends to the cached prefix and to the rows before it), variant by
variant: 16, 32 and 64 queries per CTA, more than 64 queries per KV head (two query blocks), heads of 64
and of 128, key slices merged in a cluster, by the combine kernel, or a single slice written directly.
Each case checks through `spec_attention_plan` that it runs the variant it means to cover, then compares
the logits of a ragged batch with the oracle on the same bf16-rounded weights."""
import numpy as np
import pytest

from oracle.decoder import Decoder
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu

BF16_ABS = 2e-2


def _model(d_head, n_kv_heads=2):
    base = workloads.model_config("llama_test_target")
    return workloads.scaled_config(base, n_layers=1, d_head=d_head, d_model=4 * d_head,  # 4 query heads, 2 KV heads
                                   n_kv_heads=n_kv_heads, max_positions=1024)


def _run(cfg, w, batch, rows, max_len, context, expect, check=(0, 1, -1), page_size=32):
    """`batch` sequences with ragged cached lengths (context - 5 b, wrapped into [context // 2, context]),
    then one pass of `rows` new rows each."""
    eng = binding.Engine(cfg, w, max_batch=batch, max_len=max_len, page_size=page_size, max_gamma=max(rows - 1, 1))
    try:
        plan = eng.attention_plan(0, batch, rows)
        assert plan["f16"], plan
        for key, value in expect.items():
            assert plan[key] == value, plan
        lengths = [context - (5 * b) % (context // 2) for b in range(batch)]
        seqs = np.stack([workloads.make_prompt(700 + b, context + rows, cfg["vocab"]) for b in range(batch)])
        eng.reset()
        step = max(1, 64 // batch)
        for at in range(0, context, step):
            eng.forward_logits(0, seqs[:, at:min(at + step, context)])
        eng.truncate(0, lengths)
        new = np.stack([seqs[b, context:context + rows] for b in range(batch)])
        got = eng.forward_logits(0, new).cpu().numpy()
        assert binding.spec_device_error() == 0
        oracle = Decoder(cfg, w)
        worst = 0.0
        for b in check:
            ref = oracle.forward_full(np.concatenate([seqs[b, :lengths[b]], new[b]]), last=rows)
            worst = max(worst, np.abs(got[b] - ref).max())
        assert worst <= BF16_ABS, f"max absolute logit error {worst:.3g}"
    finally:
        eng.close()


@pytest.mark.parametrize("d_head", [64, 128])
@pytest.mark.parametrize("rows", [3, 12, 20])
def test_query_blocks_of_16_32_and_64_merged_in_a_cluster(d_head, rows):
    """2 query heads per KV head x 3 / 12 / 20 rows = 6 / 24 / 40 queries of a KV head in one CTA; 16
    sequences, 150 .. 300 cached tokens (ragged tails inside a 64-key tile, several tiles per slice)."""
    cfg = _model(d_head)
    w = workloads.make_weights(cfg, 21)
    _run(cfg, w, 16, rows, 352, 300, dict(cluster_merge=True))


def test_more_than_64_queries_per_kv_head():
    """40 rows x 2 query heads = 80 queries: two query blocks per KV head (64 + 16)."""
    cfg = _model(64)
    w = workloads.make_weights(cfg, 22)
    _run(cfg, w, 16, 40, 352, 280, dict(cluster_merge=True))


def test_more_key_slices_than_a_cluster_merges():
    """A capacity of 640 tokens gives 10 key slices: partial states in global memory, combine kernel."""
    cfg = _model(64)
    w = workloads.make_weights(cfg, 23)
    _run(cfg, w, 16, 5, 640, 600, dict(cluster_merge=False, slices=10))


def test_a_single_key_slice_is_written_directly():
    """160 sequences x 2 KV heads fill the GPU with one CTA each: no merge step at all."""
    cfg = _model(128)
    w = workloads.make_weights(cfg, 24)
    _run(cfg, w, 160, 4, 128, 100, dict(slices=1), check=(0, 77, 159))


@pytest.mark.parametrize("n_kv_heads,d_head", [(4, 64), (2, 64), (4, 128)])
def test_one_row_passes_of_a_batch(n_kv_heads, d_head):
    """A draft model's step in a batch: one row per sequence, so one query per KV head (4 KV heads for 4 query
    heads) or two (2 KV heads); 40 sequences give 160 or 80 (sequence, KV head) pairs, enough for the f16 kernel
    to take them; 700 .. 1000 cached tokens so that the pass has work for it."""
    cfg = _model(d_head, n_kv_heads)
    w = workloads.make_weights(cfg, 25)
    _run(cfg, w, 40, 1, 1024, 1000, {}, check=(0, 19, 39))


@pytest.mark.parametrize("page_size", [64, 128, 256])
def test_larger_pages(page_size):
    """The tiles are fetched as 32-key boxes inside a page: pages of 64, 128 and 256 tokens (a tile then lies in one
    page, or two tiles, or four), 16 sequences x 5 rows on 128-wide heads, ragged lengths."""
    cfg = _model(128)
    w = workloads.make_weights(cfg, 26)
    _run(cfg, w, 16, 5, 512, 420, {}, page_size=page_size)

