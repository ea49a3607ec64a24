"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from oracle import sampling as oracle_sampling

MARGIN = 1e-5  # decisions closer than this to a boundary may differ (counted, not failed)


def dev():
    return torch.device("cuda:0")


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dev())


def compare_verify(n_gpu, t_gpu, tl, ql, xs, us, temperature):
    """Element-by-element comparison with the oracle.  Returns (flagged, total):
    sequences whose decision sat within MARGIN of a boundary and differed.  Any
    other difference raises."""
    n_gpu, t_gpu = n_gpu.cpu().numpy(), t_gpu.cpu().numpy()
    flagged = 0
    for b in range(tl.shape[0]):
        q_rows = ql[b] if ql is not None else np.zeros((0, tl.shape[2]))
        ref = oracle_sampling.verify_step(tl[b], q_rows, xs[b], us[b], temperature)
        if (int(n_gpu[b]), int(t_gpu[b])) == (ref.n_accepted, ref.next_token):
            continue
        close = min(ref.accept_margin, ref.cdf_margin) < MARGIN if temperature > 0 else ref.top2_gap == 0.0
        assert close, (f"sequence {b}: gpu (n={n_gpu[b]}, t={t_gpu[b]}) oracle (n={ref.n_accepted}, "
                       f"t={ref.next_token}) margins {ref.accept_margin:.3g} {ref.cdf_margin:.3g}")
        flagged += 1
    return flagged, tl.shape[0]
