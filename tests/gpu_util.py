"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import sampling as oracle_sampling

MARGIN = 1e-5  # decisions closer than this to a boundary may differ (counted, not failed)


def dev():
    return torch.device("cuda:0")


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev())


def compare_verify(n_gpu, t_gpu, tl, ql, xs, us, temperature, lenience=1.0, top_k=0, top_p=1.0):
    """Element-by-element comparison with the oracle.  Returns (flagged, total):
    sequences whose decision sat within MARGIN of a boundary and differed.  Any
    other difference raises."""
    n_gpu, t_gpu = n_gpu.cpu().numpy(), t_gpu.cpu().numpy()
    flagged = 0
    for b in range(tl.shape[0]):
        q_rows = ql[b] if ql is not None else np.zeros((0, tl.shape[2]))
        ref = oracle_sampling.verify_step(tl[b], q_rows, xs[b], us[b], temperature, lenience, top_k, top_p)
        if (int(n_gpu[b]), int(t_gpu[b])) == (ref.n_accepted, ref.next_token):
            continue
        if temperature > 0:
            close = min(ref.accept_margin, ref.cdf_margin) < MARGIN
            if not close and 0.0 < top_p < 1.0:  # a nucleus whose mass came within fp32 rounding of top_p
                rows = list(tl[b]) + list(q_rows)
                close = min(oracle_sampling.nucleus_floor(r, temperature, top_k, top_p)[1] for r in rows) < 5e-5
        else:  # a zero top-2 gap, or (lenient argmax) a drafted logit within rounding of the threshold
            close = ref.top2_gap == 0.0 or (lenience < 1.0 and ref.accept_margin < 1e-5)
        assert close, (f"sequence {b}: gpu (n={n_gpu[b]}, t={t_gpu[b]}) oracle (n={ref.n_accepted}, "
                       f"t={ref.next_token}) margins {ref.accept_margin:.3g} {ref.cdf_margin:.3g}")
        flagged += 1
    return flagged, tl.shape[0]


def compare_generation(engine, oracle_target, oracle_draft, prompt, n_new, gamma, temperature, seed, margin,
                       logit_tol, sequence=0):
    """Free-running comparison of token streams.  At the first difference the
    oracle's own margins decide whether the decision was within tolerance of a
    boundary (then it is counted, both sides restart from the oracle's prefix at
    the end of that iteration, which the position-keyed randomness allows);
    any other difference raises.  Returns (flagged, iterations)."""
    from oracle import generate as oracle_generate

    assert sequence == 0
    ref = oracle_generate.speculative_generate(oracle_target, oracle_draft, prompt, n_new, gamma, temperature, seed)
    prompt = [int(t) for t in prompt]
    done = 0
    flagged = 0
    while done < n_new:
        got, _ = engine.generate([np.array(prompt + ref.tokens[:done], dtype=np.int32)], n_new - done, gamma,
                                 temperature, seed)
        got = got[0].tolist()
        want = ref.tokens[done:]
        diff = next((k for k in range(len(want)) if got[k] != want[k]), None)
        if diff is None:
            break
        index = len(prompt) + done + diff  # absolute position of the first differing token
        it = next(i for i in ref.iterations if i.start_len <= index <= i.start_len + i.n_accepted)
        if temperature > 0:
            close = min([it.accept_margin, it.cdf_margin] + list(it.draft_cdf_margins)) < margin
        else:
            close = it.top2_gap <= 2 * logit_tol
        assert close, (f"token {index}: gpu {got[diff]} oracle {want[diff]}; iteration margins accept "
                       f"{it.accept_margin:.3g} cdf {it.cdf_margin:.3g} draft {it.draft_cdf_margins} gap {it.top2_gap:.3g}")
        flagged += 1
        done = it.start_len + it.n_accepted + 1 - len(prompt)
    return flagged, len(ref.iterations)
