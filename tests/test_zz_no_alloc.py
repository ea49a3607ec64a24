"""The allocation-free variant of speculative sampling.

Some hosts of the library cannot call cudaMalloc at the moment they need to
sample (all device memory already belongs to their own pool, or allocation is
forbidden after warm-up), so they cannot provide the workspace that
spec_verify_sample needs.  spec_verify_sample_static keeps that scratch in a
fixed array inside the library instead.  This test checks, through the C ABI,
that it returns exactly what spec_verify_sample returns, on two calls in a row
(the array keeps the previous call's contents, which must not matter), and that
shapes beyond the array's capacity are refused.

The file name makes pytest collect it last, so a run that stops at the first
failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _inputs(seed, batch, gamma, vocab):
    dev = torch.device("cuda:0")
    tl, ql = workloads.make_sampler_logits(seed, batch, gamma, vocab, 1.0)
    us = workloads.make_uniform_grid(seed + 1, (batch, gamma + 1))
    draw = workloads.make_uniform_grid(seed + 2, (batch * gamma,))
    tl_d, ql_d = torch.from_numpy(tl).to(dev), torch.from_numpy(ql).to(dev)
    xs = binding.spec_sample(ql_d.view(-1, vocab), torch.from_numpy(draw).to(dev), 1.0).view(batch, gamma).contiguous()
    return tl_d, ql_d, xs, torch.from_numpy(us).to(dev)


def test_static_variant_matches_the_workspace_variant_twice_in_a_row():
    dev = torch.device("cuda:0")
    # two different shapes back to back: the second call finds the first one's leftovers in the array
    for seed, (batch, gamma, vocab, temperature) in enumerate([(64, 7, 32000, 1.0), (9, 3, 8193, 0.7), (5, 4, 32000, 0.0)]):
        tl, ql, xs, us = _inputs(40 + seed, batch, gamma, vocab)
        want_n, want_t = binding.spec_verify_sample(tl, ql, xs, us, temperature)
        n = torch.full((batch,), -1, dtype=torch.int32, device=dev)
        t = torch.full((batch,), -1, dtype=torch.int32, device=dev)
        for _ in range(2):
            n.fill_(-1)
            t.fill_(-1)
            binding.spec_verify_sample_static(tl, ql, xs, us, temperature, n, t)
            torch.cuda.synchronize()
            # same kernels on the same inputs: identical decisions and tokens
            assert torch.equal(n, want_n) and torch.equal(t, want_t)


def test_shapes_beyond_the_built_in_array_are_refused():
    lib = binding.lib()
    capacity = lib.spec_verify_sample_static_capacity()
    assert capacity == 1 << 20
    batch, gamma, vocab = 1024, 7, 32000
    assert binding.spec_verify_sample_workspace_bytes(batch, gamma, vocab) > capacity
    # The shape is refused before any pointer is used, so one small buffer can stand in for all of them.
    buf = torch.zeros(16, device="cuda:0")
    p = buf.data_ptr()
    status = lib.spec_verify_sample_static(p, p, p, p, batch, gamma, vocab, 1.0, p, p, None)
    assert status == -4 and b"built-in array" in lib.spec_last_error()
    # a shape that fits is accepted right after the refusal
    tl, ql, xs, us = _inputs(50, 4, 2, 4096)
    n = torch.empty(4, dtype=torch.int32, device="cuda:0")
    t = torch.empty(4, dtype=torch.int32, device="cuda:0")
    binding.spec_verify_sample_static(tl, ql, xs, us, 1.0, n, t)
    want_n, want_t = binding.spec_verify_sample(tl, ql, xs, us, 1.0)
    torch.cuda.synchronize()
    assert torch.equal(n, want_n) and torch.equal(t, want_t)
