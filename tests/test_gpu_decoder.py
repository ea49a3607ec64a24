"""Parity of the decoder forward pass (teacher-forced logits, KV roll-back,
paging) with the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle.decoder import Decoder
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu

FP32_REL = 1e-4   # max |delta| / max |ref| per logit row, fp32 models
BF16_ABS = 2e-2   # max |delta| per logit, bf16 models (oracle on the same bf16-rounded weights)


def _check_logits(got, ref, dtype):
    got = got.astype(np.float64)
    if dtype == "fp32":
        rel = np.abs(got - ref).max(axis=-1) / np.abs(ref).max(axis=-1)
        assert rel.max() <= FP32_REL, f"max relative logit error {rel.max():.3g}"
        return rel.max()
    err = np.abs(got - ref).max()
    assert err <= BF16_ABS, f"max absolute logit error {err:.3g}"
    return err


def _pair(name, seed=1, **overrides):
    cfg = workloads.scaled_config(workloads.model_config(name), **overrides)
    return cfg, workloads.make_weights(cfg, seed)


@pytest.mark.parametrize("name,overrides", [
    ("tiny_target", {}),
    ("tiny_draft", {}),
    ("llama_test_target", {}),
    ("llama_test_draft", {}),
    ("gpt97m_target", {}),
    ("gpt6m_draft", {}),                                   # tied embeddings
    ("llama160m_draft", {"n_layers": 2, "vocab": 4096}),   # d_head 64 rotary, wide FFN
    ("llama160m_draft", {}),                               # the benchmark's draft at full size (12 blocks, vocabulary 32000)
    ("llama7b_target", {"n_layers": 1, "vocab": 4096, "d_ff": 1024}),  # d_head 128, 32 query / 8 KV heads
])
def test_teacher_forced_logits_with_rollback(name, overrides):
    cfg, w = _pair(name, **overrides)
    oracle = Decoder(cfg, w)
    eng = binding.Engine(cfg, w, max_batch=1, max_len=128, page_size=32, max_gamma=10)
    tokens = workloads.make_prompt(3, 40, cfg["vocab"])
    ref = oracle.forward_full(tokens)  # cache-free: cannot carry a stale row
    eng.reset()
    got = [eng.forward_logits(0, tokens[None, :9]).cpu().numpy()[0]]
    junk = workloads.make_prompt(4, 6, cfg["vocab"])
    eng.forward_logits(0, junk[None, :])             # speculative rows ...
    eng.truncate(0, [9])                             # ... rolled back
    got.append(eng.forward_logits(0, tokens[None, 9:20]).cpu().numpy()[0])
    eng.forward_logits(0, junk[None, :3])
    eng.truncate(0, [18])                            # roll back into rows that were kept before
    got.append(eng.forward_logits(0, tokens[None, 18:19]).cpu().numpy()[0])   # single row
    got.append(eng.forward_logits(0, tokens[None, 19:40]).cpu().numpy()[0])   # crosses page boundaries
    _check_logits(got[0], ref[:9], cfg["dtype"])
    _check_logits(got[1], ref[9:20], cfg["dtype"])
    _check_logits(got[2], ref[18:19], cfg["dtype"])
    _check_logits(got[3], ref[19:40], cfg["dtype"])
    eng.close()


def test_bf16_kv_cache_option_stays_close():
    """K,V rows rounded to bf16: allowed as an option, with a looser bound that is
    reported, not the parity bar."""
    cfg, w = _pair("llama_test_target")
    tokens = workloads.make_prompt(3, 40, cfg["vocab"])
    ref = Decoder(cfg, w).forward_full(tokens)
    eng = binding.Engine(cfg, w, max_batch=1, max_len=64, page_size=32, max_gamma=3, kv_dtype="bf16")
    eng.reset()
    got = eng.forward_logits(0, tokens[None, :]).cpu().numpy()[0]
    err = np.abs(got - ref).max()
    assert 0 < err < 5e-2
    eng.close()


def test_sixteen_bit_kv_rows_on_a_wide_block():
    """One block of the 7B width (32 query / 8 KV heads of 128): fp16 K,V rows, the default for bf16
    models, stay inside the parity bar like fp32 rows; bf16 rows keep 8 bits and are looser."""
    cfg, w = _pair("llama7b_target", n_layers=1, vocab=4096, d_ff=1024)
    tokens = workloads.make_prompt(3, 96, cfg["vocab"])
    ref = Decoder(cfg, w).forward_full(tokens)
    errs = {}
    for kv in ("fp32", "fp16", "bf16"):
        eng = binding.Engine(cfg, w, max_batch=1, max_len=128, page_size=32, max_gamma=3, kv_dtype=kv)
        eng.reset()
        got = np.concatenate([eng.forward_logits(0, tokens[None, :64]).cpu().numpy()[0],
                              eng.forward_logits(0, tokens[None, 64:96]).cpu().numpy()[0]])
        errs[kv] = np.abs(got - ref).max()
        eng.close()
    assert errs["fp32"] <= BF16_ABS and errs["fp16"] <= BF16_ABS, errs
    assert errs["fp16"] < errs["bf16"] < 1e-1, errs


def test_batched_sequences_are_independent_and_page_size_is_invisible():
    cfg, w = _pair("llama_test_target")
    seqs = [workloads.make_prompt(10 + b, 30, cfg["vocab"]) for b in range(3)]
    ref = [Decoder(cfg, w).forward_full(s) for s in seqs]
    outs = []
    for page in (32, 128):
        eng = binding.Engine(cfg, w, max_batch=3, max_len=64, page_size=page, max_gamma=7)
        eng.reset()
        a = eng.forward_logits(0, np.stack([s[:8] for s in seqs])).cpu().numpy()
        # ragged roll-back: different lengths per sequence, then continue from there
        eng.truncate(0, [8, 5, 2])
        tails = [seqs[0][8:16], seqs[1][5:13], seqs[2][2:10]]
        b = eng.forward_logits(0, np.stack(tails)).cpu().numpy()
        outs.append((a, b))
        for i in range(3):
            _check_logits(a[i], ref[i][:8], "bf16")
        _check_logits(b[0], ref[0][8:16], "bf16")
        _check_logits(b[1], ref[1][5:13], "bf16")
        _check_logits(b[2], ref[2][2:10], "bf16")
        eng.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


def test_both_models_of_a_pair_share_a_context():
    tcfg, tw = _pair("tiny_target")
    dcfg, dw = _pair("tiny_draft", seed=2)
    eng = binding.Engine(tcfg, tw, dcfg, dw, max_batch=2, max_len=64, page_size=32, max_gamma=3)
    tokens = np.stack([workloads.make_prompt(5, 12, 8192), workloads.make_prompt(6, 12, 8192)])
    eng.reset()
    t = eng.forward_logits(0, tokens).cpu().numpy()
    d = eng.forward_logits(1, tokens).cpu().numpy()
    for b in range(2):
        _check_logits(t[b], Decoder(tcfg, tw).forward_full(tokens[b]), "fp32")
        _check_logits(d[b], Decoder(dcfg, dw).forward_full(tokens[b]), "fp32")
    eng.close()


def test_errors_are_reported():
    cfg, w = _pair("tiny_draft")
    with pytest.raises(binding.SpecError) as e:
        binding.Engine(workloads.scaled_config(cfg, d_head=48), w)
    assert e.value.status == -2
    eng = binding.Engine(cfg, w, max_batch=1, max_len=32, page_size=32, max_gamma=2)
    with pytest.raises(binding.SpecError) as e:
        eng.forward_logits(0, np.zeros((1, 40), dtype=np.int32))
    assert e.value.status == -4
    with pytest.raises(binding.SpecError) as e:
        eng.forward_logits(0, np.full((1, 2), 8192, dtype=np.int32))
    assert e.value.status == -1
    with pytest.raises(binding.SpecError) as e:
        eng.generate([np.array([1, 2, 3])], 8, 1, 1.0, 0)  # gamma > 0 without a draft model
    assert e.value.status == -2
    with pytest.raises(binding.SpecError) as e:
        eng.generate([np.array([1, 2, 3])], 40, 0, 1.0, 0)  # does not fit max_len
    assert e.value.status == -4
    eng.close()


@pytest.mark.parametrize("rows,n_out,k", [(1, 128, 64), (5, 300, 200), (3, 768, 768), (11, 2304, 768), (16, 704, 256),
                                          (17, 256, 512), (70, 384, 256), (130, 256, 192), (7, 8192, 768),
                                          (40, 384, 320), (48, 256, 256), (96, 512, 192), (160, 384, 256), (250, 256, 128)])
def test_linear_layer_paths_agree_with_the_plain_definition(rows, n_out, k):
    """y = x W^T on the FMA pipes, on the tensor cores (row-major and tile-major
    weights) against numpy in fp64; the two tensor-core layouts are bit-identical."""
    rng = np.random.default_rng(rows * 1000 + k)
    x = rng.standard_normal((rows, k)).astype(np.float32)
    w = workloads.round_to_bf16(rng.standard_normal((n_out, k)).astype(np.float32) * 0.05)
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    xd = torch.from_numpy(x).cuda()
    wd = torch.from_numpy(w).cuda().to(torch.bfloat16)
    scale = np.abs(ref).max()
    alu = binding.spec_linear(xd, wd, "alu").cpu().numpy()
    tc = binding.spec_linear(xd, wd, "tensor")
    packed = binding.spec_linear(xd, binding.spec_pack_weight(wd), "tensor_packed", n_out=n_out)
    f32 = binding.spec_linear(xd, torch.from_numpy(w).cuda(), "auto").cpu().numpy()
    torch.cuda.synchronize()
    assert binding.spec_device_error() == 0
    assert np.abs(alu - ref).max() <= 1e-5 * scale
    assert np.abs(f32 - ref).max() <= 1e-5 * scale
    # two bf16 terms keep 16 mantissa bits of x: relative error ~ 2^-16 per product
    assert np.abs(tc.cpu().numpy() - ref).max() <= 1e-4 * scale
    assert torch.equal(tc, packed)
    # the GEMM kernel alone: its split-K partial sums, added in split order, are the same result
    ws = torch.empty(binding.spec_linear_workspace_bytes(rows, n_out, k), dtype=torch.uint8, device="cuda")
    pk = binding.spec_pack_weight(wd)
    parts = binding.spec_linear_partials(xd, pk, n_out, ws)
    total = parts[0].clone()
    for s in range(1, parts.shape[0]):
        total += parts[s]
    assert torch.equal(total, tc)
    again = binding.spec_linear_partials(None, pk, n_out, ws, split_input=False, rows=rows, k=k)  # reuses the split
    assert torch.equal(again.sum(0), parts.sum(0))


def test_timing_a_pass_leaves_the_caches_alone():
    """spec_time_forward replays a pass beyond the cached rows: positive device time,
    and the teacher-forced logits that follow are those of the untouched prefix."""
    cfg, w = _pair("llama_test_target")
    tokens = workloads.make_prompt(5, 30, cfg["vocab"])
    ref = Decoder(cfg, w).forward_full(tokens)
    eng = binding.Engine(cfg, w, max_batch=1, max_len=64, page_size=32, max_gamma=3)
    eng.forward_logits(0, tokens[None, :20])
    one, four = eng.time_forward(0, 1, 1, repeats=5), eng.time_forward(0, 1, 4, repeats=5)
    assert 0.0 < one < 50.0 and 0.0 < four < 50.0
    got = eng.forward_logits(0, tokens[None, 20:30]).cpu().numpy()[0]
    _check_logits(got, ref[20:30], cfg["dtype"])
    with pytest.raises(binding.SpecError):
        eng.time_forward(1, 1, 1)  # no draft model
    eng.close()
