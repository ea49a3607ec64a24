"""Parity of the fused speculative-sampling kernel, the plain sampler and the
device uniforms with the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch
from scipy import stats

from gpu_util import MARGIN, compare_verify, dev, to_dev
from oracle import analysis, philox
from oracle import sampling as oracle_sampling
from paper_2211_17192_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _draft_tokens(ql, seed, temperature, top_k=0, top_p=1.0):
    """x_i ~ q_i drawn by the oracle with seeded uniforms."""
    batch, gamma, _ = ql.shape
    draw = workloads.make_uniform_grid(seed, (batch, max(gamma, 1)))
    xs = np.zeros((batch, gamma), dtype=np.int32)
    for b in range(batch):
        for i in range(gamma):
            xs[b, i] = oracle_sampling.sample_token(ql[b, i], draw[b, i], temperature, top_k, top_p)[0]
    return xs, draw


def _run(tl, ql, xs, us, temperature, lenience=1.0, top_k=0, top_p=1.0):
    n, t = binding.spec_verify_sample(to_dev(tl), to_dev(ql) if ql.size else None,
                                      to_dev(xs) if xs.size else None, to_dev(us), temperature, lenience=lenience,
                                      top_k=top_k, top_p=top_p)
    torch.cuda.synchronize()
    return n, t


@pytest.mark.parametrize("noise", [0.5, 1.0, 2.0])
def test_standalone_sampler_workload(noise):
    """Batch 64 x (gamma+1 = 8) x vocab 32000, T = 1: decisions and tokens identical."""
    batch, gamma, vocab = 64, 7, 32000
    tl, ql = workloads.make_sampler_logits(100 + int(noise * 10), batch, gamma, vocab, noise)
    xs, _ = _draft_tokens(ql, 7, 1.0)
    us = workloads.make_uniform_grid(8, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, 1.0)
    flagged, total = compare_verify(n, t, tl, ql, xs, us, 1.0)
    assert flagged <= 2, f"{flagged} of {total} sequences within {MARGIN} of a decision boundary"
    ns = n.cpu().numpy()
    assert ns.min() >= 0 and ns.max() <= gamma
    if noise == 0.5:
        assert ns.mean() > 2.0  # a close draft is accepted often


@pytest.mark.parametrize("batch,gamma,vocab,temperature", [
    (3, 0, 1000, 1.0),       # gamma = 0: plain draw from p
    (5, 1, 1, 1.0),          # single-token vocabulary
    (5, 2, 5, 1.0),
    (7, 3, 1001, 0.7),       # rows not 16-byte aligned: scalar loads
    (4, 10, 8192, 1.0),      # rows split into two chunks
    (4, 5, 8193, 1.3),       # ragged chunk boundary
    (2, 3, 100003, 1.0),     # several chunks, ragged tail
    (1, 2, 262144, 1.0),     # one sequence, long rows: many chunks per row
    (300, 1, 4100, 1.0),     # large batch: whole-row CTAs
    (9, 4, 32000, 0.0),      # greedy
    (6, 6, 1001, 0.0),
    (3, 64, 257, 1.0),       # maximum gamma
    (6, 3, 32000, 0.05),     # cold: nearly one-hot rows, exponents scaled by 29
    (6, 3, 32000, 8.0),      # hot: nearly flat rows
    (5, 2, 50257, 0.1),      # cold, scalar loads
])
def test_shapes_and_edges(batch, gamma, vocab, temperature):
    tl, ql = workloads.make_sampler_logits(batch * 1000 + gamma, batch, gamma, vocab, 1.0)
    xs, _ = _draft_tokens(ql, 3, temperature)
    us = workloads.make_uniform_grid(4, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, temperature)
    flagged, _ = compare_verify(n, t, tl, ql, xs, us, temperature)
    assert flagged <= 1


@pytest.mark.parametrize("temperature", [1.0, 0.0])
@pytest.mark.parametrize("lenience", [0.5, 0.1])
def test_lenience(temperature, lenience):
    """Appendix A.5: decisions and tokens identical to the oracle; more drafted tokens
    survive than under the strict rule."""
    batch, gamma, vocab = 48, 5, 8192
    tl, ql = workloads.make_sampler_logits(77, batch, gamma, vocab, 2.0)
    xs, _ = _draft_tokens(ql, 5, 1.0)  # drafted by sampling, also for the argmax case: a spread of logits at x
    us = workloads.make_uniform_grid(6, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, temperature, lenience)
    flagged, _ = compare_verify(n, t, tl, ql, xs, us, temperature, lenience)
    assert flagged <= 1
    strict, _ = _run(tl, ql, xs, us, temperature)
    assert n.sum().item() >= strict.sum().item()
    if temperature > 0:
        assert n.sum().item() > strict.sum().item()
    with pytest.raises(binding.SpecError):
        _run(tl, ql, xs, us, temperature, 0.0)


def test_identical_and_disjoint_distributions():
    batch, gamma, vocab = 6, 4, 4096
    tl, _ = workloads.make_sampler_logits(5, batch, gamma, vocab, 1.0)
    ql = np.ascontiguousarray(tl[:, :gamma])
    xs, _ = _draft_tokens(ql, 9, 1.0)
    us = workloads.make_uniform_grid(10, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, 1.0)
    assert n.cpu().tolist() == [gamma] * batch  # p = q: everything accepted (Corollary 3.4)
    compare_verify(n, t, tl, ql, xs, us, 1.0)
    # disjoint supports: never accepted, t from p restricted to its support
    tl2, ql2 = tl.copy(), ql.copy()
    tl2[:, :, vocab // 2:] = -1e4
    ql2[:, :, : vocab // 2] = -1e4
    xs2, _ = _draft_tokens(ql2, 9, 1.0)
    n, t = _run(tl2, ql2, xs2, us, 1.0)
    assert n.cpu().tolist() == [0] * batch and int(t.max()) < vocab // 2
    compare_verify(n, t, tl2, ql2, xs2, us, 1.0)


@pytest.mark.parametrize("vocab", [32000, 4096])
def test_vanished_residual_falls_back_to_the_target_row(vocab):
    """p = q and a rejection all the same (a guess outside the vocabulary is rejected by rule): max(0, p - q)
    sums to zero, so t is a plain draw from p_{n+1} (the reading taken for a vanishing normaliser).  At vocabulary
    32000 the draw runs in a 4-CTA cluster and the inverse CDF is entered twice (residual, then plain)."""
    batch, gamma = 3, 2
    tl, _ = workloads.make_sampler_logits(12, batch, gamma, vocab, 1.0)
    ql = np.ascontiguousarray(tl[:, :gamma])
    first = oracle_sampling.sample_token(ql[2, 0], 0.37, 1.0)[0]  # a guess q_1 can give: accepted, since p_1 = q_1
    xs = np.array([[-1, 5], [vocab, 1], [first, -1]], dtype=np.int32)
    us = workloads.make_uniform_grid(13, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, 1.0)
    assert n.cpu().tolist() == [0, 0, 1]
    for b, rows_kept in enumerate([0, 0, 1]):
        ref, margin = oracle_sampling.sample_token(tl[b, rows_kept], us[b, gamma], 1.0)
        assert int(t[b]) == ref or margin < MARGIN


def test_out_of_range_draft_token_is_rejected():
    tl, ql = workloads.make_sampler_logits(6, 2, 3, 500, 0.1)
    xs = np.array([[1, 500, 2], [-1, 3, 4]], dtype=np.int32)
    us = np.full((2, 4), 1.0 / 2**24, dtype=np.float32)
    n, t = _run(tl, ql, xs, us, 1.0)
    assert n.cpu().tolist() == [1, 0] and 0 <= int(t.min()) and int(t.max()) < 500


def test_workspace_is_reusable_and_checked():
    tl, ql = workloads.make_sampler_logits(7, 4, 2, 3000, 1.0)
    xs, _ = _draft_tokens(ql, 1, 1.0)
    us = workloads.make_uniform_grid(2, (4, 3))
    ws = torch.zeros(binding.spec_verify_sample_workspace_bytes(4, 2, 3000), dtype=torch.uint8, device=dev())
    args = (to_dev(tl), to_dev(ql), to_dev(xs), to_dev(us), 1.0)
    a = binding.spec_verify_sample(*args, workspace=ws)
    a = (a[0].clone(), a[1].clone())
    b = binding.spec_verify_sample(*args, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    with pytest.raises(binding.SpecError):
        binding.spec_verify_sample(*args, workspace=ws[:64])


def test_distribution_over_a_million_trials():
    """Appendix A.1 and Theorem 3.5 on the GPU: vocabulary 64, fixed p and q."""
    vocab, per_launch, launches = 64, 62500, 16
    tl, ql = workloads.make_sampler_logits(11, 1, 1, vocab, 1.0)
    p = oracle_sampling.standardise(tl[0, 0], 1.0)
    q = oracle_sampling.standardise(ql[0, 0], 1.0)
    tl_d = to_dev(tl).expand(per_launch, 2, vocab).contiguous()
    ql_d = to_dev(ql).expand(per_launch, 1, vocab).contiguous()
    first = np.zeros(vocab)
    accepted = 0
    seq = torch.zeros(per_launch, dtype=torch.int32, device=dev())
    for k in range(launches):
        pos = torch.arange(k * per_launch, (k + 1) * per_launch, dtype=torch.int32, device=dev())
        u_draft = binding.spec_uniforms(5, pos, seq, 0)
        r = binding.spec_uniforms(5, pos, seq, 1)
        u = binding.spec_uniforms(5, pos, seq, 2)
        x = binding.spec_sample(ql_d.view(per_launch, vocab), u_draft, 1.0)
        n, t = binding.spec_verify_sample(tl_d, ql_d, x.view(-1, 1), torch.stack([r, u], dim=1).contiguous(), 1.0)
        emitted = torch.where(n == 1, x, t)
        first += np.bincount(emitted.cpu().numpy(), minlength=vocab)
        accepted += int((n == 1).sum())
    trials = per_launch * launches
    expected = p * trials
    keep = expected >= 5
    counts = np.append(first[keep], first[~keep].sum())
    exp = np.append(expected[keep], expected[~keep].sum())
    if exp[-1] == 0:
        counts, exp = counts[:-1], exp[:-1]
    assert stats.chisquare(counts, exp).pvalue > 1e-3
    beta = analysis.beta(p, q)
    assert abs(accepted / trials - beta) < 4 * np.sqrt(beta * (1 - beta) / trials)


def test_device_uniforms_are_bit_exact():
    pos = np.array([0, 1, 2, 77, 123456, 2**31 - 1], dtype=np.int32)
    seqs = np.array([0, 0, 5, 31, 2, 9], dtype=np.int32)
    for seed in (0, 42, 0xDEADBEEF_12345678):
        for purpose in (0, 1, 2):
            got = binding.spec_uniforms(seed, to_dev(pos), to_dev(seqs), purpose).cpu().numpy().astype(np.float64)
            ref = philox.uniforms_vec(seed, pos, seqs, purpose)
            assert np.array_equal(got, ref)


@pytest.mark.parametrize("rows,vocab,temperature", [(64, 8192, 1.0), (5, 1001, 0.5), (3, 7, 1.0), (16, 32000, 0.0),
                                                    (2, 100003, 1.0)])
def test_plain_sampler(rows, vocab, temperature):
    logits, _ = workloads.make_sampler_logits(rows + vocab, rows, 0, vocab, 1.0)
    logits = logits[:, 0]
    us = workloads.make_uniform_grid(12, (rows,))
    got = binding.spec_sample(to_dev(logits), to_dev(us), temperature).cpu().numpy()
    flagged = 0
    for r in range(rows):
        ref, margin = oracle_sampling.sample_token(logits[r], us[r], temperature)
        if got[r] != ref:
            assert margin < MARGIN
            flagged += 1
    assert flagged <= 1


@pytest.mark.parametrize("rows,vocab", [(6, 7), (5, 1001), (9, 8192), (16, 32000), (4, 32128), (3, 50257), (2, 100003)])
def test_top_k_floors_are_bit_exact(rows, vocab):
    """The k-th largest logit of every row, for k across the range; also with heavy ties."""
    logits, _ = workloads.make_sampler_logits(rows * 7 + vocab, rows, 0, vocab, 1.0)
    logits = np.ascontiguousarray(logits[:, 0])
    tied = np.round(logits * 2).astype(np.float32) / 2  # a few dozen distinct values, both signs and zero
    tied[0, : min(3, vocab)] = -0.0
    for data in (logits, tied):
        d = to_dev(data)
        for k in sorted({1, 2, min(40, vocab), max(1, vocab // 2), vocab - 1, vocab} - {0}):
            if k == vocab:
                continue  # no cut: the entry point refuses
            got = binding.spec_truncation_floors(d, 1.0, top_k=k).cpu().numpy()
            want = np.sort(data, axis=1)[:, vocab - k]
            assert np.array_equal(got, want), (vocab, k)
            if 0 < k < vocab:
                assert [oracle_sampling.top_k_floor(data[r], k) for r in range(rows)] == want.astype(np.float64).tolist()


@pytest.mark.parametrize("batch,gamma,vocab,temperature,top_k", [
    (64, 7, 32000, 1.0, 40),
    (64, 7, 32000, 1.0, 1),     # both models one-hot: accepted iff the two maxima coincide
    (8, 3, 8192, 0.7, 5),
    (5, 2, 1001, 1.0, 10),      # scalar loads
    (2, 3, 100003, 1.0, 50),    # rows re-read per bit
    (7, 4, 4096, 1.0, 4096),    # k = V: no cut
    (7, 4, 4096, 1.0, 5000),    # k > V: no cut
    (6, 0, 32128, 1.0, 20),     # gamma = 0: plain top-k draw from p
    (9, 4, 32000, 0.0, 3),      # T = 0 ignores k
])
def test_top_k_verify(batch, gamma, vocab, temperature, top_k):
    tl, ql = workloads.make_sampler_logits(batch + gamma + vocab, batch, gamma, vocab, 1.0)
    xs, _ = _draft_tokens(ql, 3, temperature, top_k)
    us = workloads.make_uniform_grid(4, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, temperature, top_k=top_k)
    flagged, _ = compare_verify(n, t, tl, ql, xs, us, temperature, top_k=top_k)
    assert flagged <= 1
    if temperature > 0 and 0 < top_k < vocab:
        # every emitted token lies in the target's top-k set of its row
        ns, ts = n.cpu().numpy(), t.cpu().numpy()
        for b in range(batch):
            row = tl[b, ns[b]]
            assert row[ts[b]] >= np.sort(row)[vocab - top_k]
        plain_n, _ = _run(tl, ql, xs, us, temperature)
        if top_k == 1:
            same = (tl[:, :gamma].argmax(-1) == ql.argmax(-1)) if gamma else np.zeros((batch, 0), bool)
            want = [int(np.argmin(np.append(same[b], False))) for b in range(batch)]
            assert ns.tolist() == want
        del plain_n


@pytest.mark.parametrize("rows,vocab,temperature,top_k", [(64, 8192, 1.0, 50), (5, 1001, 0.5, 3), (3, 7, 1.0, 2),
                                                          (16, 32000, 1.0, 1), (2, 100003, 1.0, 40), (4, 32000, 0.0, 5)])
def test_plain_sampler_top_k(rows, vocab, temperature, top_k):
    logits, _ = workloads.make_sampler_logits(rows + vocab, rows, 0, vocab, 1.0)
    logits = logits[:, 0]
    us = workloads.make_uniform_grid(12, (rows,))
    got = binding.spec_sample(to_dev(logits), to_dev(us), temperature, top_k=top_k).cpu().numpy()
    flagged = 0
    for r in range(rows):
        ref, margin = oracle_sampling.sample_token(logits[r], us[r], temperature, top_k)
        if got[r] != ref:
            assert margin < MARGIN
            flagged += 1
    assert flagged <= 1
    if top_k == 1:
        assert got.tolist() == logits.argmax(-1).tolist()


def _nucleus_slack(row, temperature, top_k, top_p, floor):
    """How far top_p would have to move for `floor` to be the exact nucleus cut of `row`
    (0 when it is): the kept mass must reach top_p, and must not without its lowest logit."""
    z = oracle_sampling.keep_top_k(row, top_k)
    w = np.exp((z - z.max()) / temperature)
    inside = w[z >= floor].sum() / w.sum()
    without_lowest = w[z > floor].sum() / w.sum()
    return max(0.0, top_p - inside, without_lowest - top_p)


NUCLEUS_TOL = 5e-5  # fp32 weights from the hardware exp2 and fp32 sums over up to 10^5 of them


@pytest.mark.parametrize("rows,vocab", [(6, 7), (5, 1001), (9, 8192), (16, 32000), (4, 32128), (3, 50257), (2, 100003)])
@pytest.mark.parametrize("temperature", [1.0, 0.5])
def test_nucleus_floors(rows, vocab, temperature):
    """The nucleus cut of every row, alone and after top-k: the oracle's, or (where the
    kept mass comes within fp32 rounding of top_p) the exact cut for a top_p that differs
    by less than NUCLEUS_TOL; always a logit of the row; identical when repeated."""
    logits, _ = workloads.make_sampler_logits(rows * 11 + vocab, rows, 0, vocab, 1.0)
    logits = np.ascontiguousarray(logits[:, 0])
    d = to_dev(logits)
    differ = 0
    for top_p in (0.02, 0.5, 0.9, 0.999):
        for top_k in (0, min(50, vocab - 1)):
            got = binding.spec_truncation_floors(d, temperature, top_k=top_k, top_p=top_p).cpu().numpy()
            again = binding.spec_truncation_floors(d, temperature, top_k=top_k, top_p=top_p).cpu().numpy()
            assert np.array_equal(got, again)
            for r in range(rows):
                want, margin = oracle_sampling.nucleus_floor(logits[r], temperature, top_k, top_p)
                if got[r] != np.float32(want):
                    assert got[r] in logits[r]
                    slack = _nucleus_slack(logits[r].astype(np.float64), temperature, top_k, top_p, float(got[r]))
                    assert margin < NUCLEUS_TOL and slack < NUCLEUS_TOL, (vocab, top_p, top_k, r, got[r], want, margin, slack)
                    # far in the tail consecutive tokens differ by less than fp32 rounding of the
                    # total mass, so there a different cut is the rule; elsewhere it is rare
                    differ += top_p <= 0.9
    assert differ <= 2


@pytest.mark.parametrize("vocab", [32000, 32003])
@pytest.mark.parametrize("temperature", [1.0, 0.3])
def test_nucleus_floors_with_ties_and_masked_logits(vocab, temperature):
    """Rows the binned selection has to work for: logits rounded to halves (thousands of equal values: the bin
    where the mass is crossed holds more logits than are ranked at once, and its range collapses to one value),
    a third of the row masked with -inf (not every element is in play), all logits equal, one finite logit."""
    base, _ = workloads.make_sampler_logits(77 + vocab, 6, 0, vocab, 1.0)
    base = np.ascontiguousarray(base[:, 0])
    rng = np.random.default_rng(5)
    logits = base.copy()
    logits[0] = np.round(base[0] * 2) / 2
    logits[1] = np.round(base[1] * 8) / 8
    logits[2, rng.random(vocab) < 1 / 3] = -np.inf
    logits[3] = 1.25
    logits[4] = -np.inf
    logits[4, vocab // 2] = 0.5
    logits[5] = np.round(base[5] * 2) / 2
    logits[5, rng.random(vocab) < 0.5] = -np.inf
    d = to_dev(logits)
    for top_p in (0.1, 0.5, 0.9, 0.99):
        for top_k in (0, 50, 300):  # alone; after a top-k found through the threads' maxima; after a binned top-k
            got = binding.spec_truncation_floors(d, temperature, top_k=top_k, top_p=top_p).cpu().numpy()
            again = binding.spec_truncation_floors(d, temperature, top_k=top_k, top_p=top_p).cpu().numpy()
            assert np.array_equal(got, again)
            for r in range(logits.shape[0]):
                want, margin = oracle_sampling.nucleus_floor(logits[r], temperature, top_k, top_p)
                if got[r] != np.float32(want):
                    assert got[r] in logits[r]
                    slack = _nucleus_slack(logits[r].astype(np.float64), temperature, top_k, top_p, float(got[r]))
                    assert margin < NUCLEUS_TOL and slack < NUCLEUS_TOL, (vocab, top_p, top_k, r, got[r], want, margin, slack)
    for top_k in (1, 50, 128, 129, 300):  # top-k alone on the same rows: the k-th largest by a sort, or -inf when
        got = binding.spec_truncation_floors(d, temperature, top_k=top_k, top_p=1.0).cpu().numpy()  # fewer logits are finite
        for r in range(logits.shape[0]):
            finite = np.sort(logits[r][np.isfinite(logits[r])])[::-1]
            want = finite[top_k - 1] if top_k <= finite.size else -np.inf
            assert got[r] == np.float32(want), (vocab, top_k, r, got[r], want)


@pytest.mark.parametrize("batch,gamma,vocab,temperature,top_k,top_p", [
    (64, 7, 32000, 1.0, 0, 0.9),
    (64, 7, 32000, 1.0, 40, 0.8),   # both cuts
    (8, 3, 8192, 0.7, 0, 0.5),
    (5, 2, 1001, 1.0, 10, 0.95),    # scalar loads
    (2, 3, 100003, 1.0, 0, 0.3),    # rows re-read per bit
    (7, 4, 4096, 1.0, 0, 1.0),      # top_p = 1: no cut
    (7, 4, 4096, 1.0, 0, 1e-6),     # only the maximum survives
    (6, 0, 32128, 1.0, 0, 0.7),     # gamma = 0: plain nucleus draw from p
    (9, 4, 32000, 0.0, 0, 0.5),     # T = 0 ignores it
])
def test_nucleus_verify(batch, gamma, vocab, temperature, top_k, top_p):
    tl, ql = workloads.make_sampler_logits(batch + gamma + vocab + 1, batch, gamma, vocab, 1.0)
    xs, _ = _draft_tokens(ql, 3, temperature, top_k, top_p)
    us = workloads.make_uniform_grid(4, (batch, gamma + 1))
    n, t = _run(tl, ql, xs, us, temperature, top_k=top_k, top_p=top_p)
    flagged, _ = compare_verify(n, t, tl, ql, xs, us, temperature, top_k=top_k, top_p=top_p)
    assert flagged <= 1
    if top_p == 1e-6:
        same = (tl[:, :gamma].argmax(-1) == ql.argmax(-1))
        assert n.cpu().numpy().tolist() == [int(np.argmin(np.append(same[b], False))) for b in range(batch)]


@pytest.mark.parametrize("rows,vocab,temperature,top_k,top_p", [(64, 8192, 1.0, 0, 0.9), (5, 1001, 0.5, 20, 0.6),
                                                                (3, 7, 1.0, 0, 0.5), (16, 32000, 1.0, 0, 0.25),
                                                                (2, 100003, 1.0, 0, 0.8), (4, 32000, 0.0, 0, 0.5)])
def test_plain_sampler_nucleus(rows, vocab, temperature, top_k, top_p):
    logits, _ = workloads.make_sampler_logits(rows + vocab, rows, 0, vocab, 1.0)
    logits = logits[:, 0]
    us = workloads.make_uniform_grid(12, (rows,))
    got = binding.spec_sample(to_dev(logits), to_dev(us), temperature, top_k=top_k, top_p=top_p).cpu().numpy()
    flagged = 0
    for r in range(rows):
        ref, margin = oracle_sampling.sample_token(logits[r], us[r], temperature, top_k, top_p)
        if got[r] != ref:
            assert margin < MARGIN or oracle_sampling.nucleus_floor(logits[r], temperature, top_k, top_p)[1] < NUCLEUS_TOL
            flagged += 1
    assert flagged <= 1
