"""Failure paths of the library, exercised without faulting the GPU: non-finite logits are
reported (not sampled from in silence), and a bounded device-side wait that runs out
comes back as a status while the context stays usable."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import sampling as oracle_sampling
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _pair():
    tcfg, dcfg = workloads.model_config("llama_test_target"), workloads.model_config("llama_test_draft")
    return tcfg, workloads.make_weights(tcfg, 1), dcfg, workloads.make_weights(dcfg, 2)


@pytest.mark.parametrize("which,value,temperature,gamma", [
    ("target", np.nan, 1.0, 3), ("target", np.inf, 1.0, 3), ("target", np.nan, 0.0, 2),
    ("draft", np.nan, 1.0, 3), ("draft", np.nan, 0.0, 2), ("target", np.nan, 1.0, 0),
])
def test_non_finite_logits_are_reported(which, value, temperature, gamma):
    """A NaN (or +inf) planted in one row of an LM head makes one logit of every row non-finite:
    the generation call returns SPEC_ERR_NONFINITE; the same pair without it generates."""
    tcfg, tw, dcfg, dw = _pair()
    prompt = workloads.make_prompt(3, 8, tcfg["vocab"])
    good = binding.Engine(tcfg, tw, dcfg, dw, max_batch=1, max_len=64, page_size=32, max_gamma=3)
    out, stats = good.generate([prompt], 12, gamma, temperature, 1)
    assert out.shape == (1, 12)
    good.close()
    bad_t, bad_d = dict(tw), dict(dw)
    victim = bad_t if which == "target" else bad_d
    head = victim["head"].copy()
    head[7, :] = value
    victim["head"] = head
    eng = binding.Engine(tcfg, bad_t, dcfg, bad_d, max_batch=1, max_len=64, page_size=32, max_gamma=3)
    try:
        with pytest.raises(binding.SpecError) as e:
            eng.generate([prompt], 12, gamma, temperature, 1)
        assert e.value.status == -7
    finally:
        eng.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_library_usable():
    h = binding.lib()
    h.spec_timeout_drill.restype = ctypes.c_int
    h.spec_timeout_drill.argtypes = [ctypes.c_void_p]
    torch.cuda.synchronize()
    assert binding.spec_device_error() == 0
    status = h.spec_timeout_drill(torch.cuda.current_stream().cuda_stream)
    assert status == -6, h.spec_last_error().decode()      # SPEC_ERR_DEVICE_TIMEOUT, as the drill intends
    assert b"gave up on a bounded wait" in h.spec_last_error()
    assert binding.spec_device_error() == 0                  # the drill consumed the flag it raised
    # the same kernel does its work right afterwards
    rng = np.random.default_rng(0)
    x = rng.standard_normal((3, 256)).astype(np.float32)
    w = workloads.round_to_bf16(rng.standard_normal((384, 256)).astype(np.float32) * 0.05)
    got = binding.spec_linear(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda().to(torch.bfloat16), "tensor").cpu().numpy()
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(got - ref).max() <= 1e-4 * np.abs(ref).max()
    assert binding.spec_device_error() == 0


def test_greedy_guess_off_the_drafts_argmax():
    """T = 0 with a drafted token that is not the draft's own maximum (x ~ q cannot produce it,
    so Algorithm 1's test decides nothing): library and oracle accept it iff it is the
    target's maximum."""
    vocab, gamma = 64, 2
    tl, ql = workloads.make_sampler_logits(5, 3, gamma, vocab, 1.0)
    xs = np.zeros((3, gamma), dtype=np.int32)
    top = tl.argmax(axis=-1)                     # [3, gamma + 1]
    draft_top = ql.argmax(axis=-1)
    xs[0] = [top[0, 0], top[0, 1]]               # the target's maxima (whatever the draft prefers): both accepted
    xs[1] = [top[1, 0], (top[1, 1] + 1) % vocab]  # second guess is not the target's maximum: rejected there
    xs[2] = [(draft_top[2, 0] + 3) % vocab if (draft_top[2, 0] + 3) % vocab != top[2, 0] else (draft_top[2, 0] + 4) % vocab, top[2, 1]]
    us = workloads.make_uniform_grid(6, (3, gamma + 1))
    n, t = binding.spec_verify_sample(torch.from_numpy(tl).cuda(), torch.from_numpy(ql).cuda(), torch.from_numpy(xs).cuda(),
                                      torch.from_numpy(us).cuda(), 0.0)
    n, t = n.cpu().numpy(), t.cpu().numpy()
    assert n.tolist() == [2, 1, 0]
    for b in range(3):
        ref = oracle_sampling.verify_step(tl[b], ql[b], xs[b], us[b], 0.0)
        assert (int(n[b]), int(t[b])) == (ref.n_accepted, ref.next_token)
        assert t[b] == top[b, n[b]]
