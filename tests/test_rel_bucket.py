"""The library's host-side relative-position bucket against the oracle's (no GPU needed)."""
import ctypes

import numpy as np
import pytest

from oracle.encdec import relative_bucket
from paper_2211_17192_b200 import binding


@pytest.mark.parametrize("bidirectional", [0, 1])
@pytest.mark.parametrize("n_buckets,max_distance", [(32, 128), (16, 64), (32, 100), (8, 20)])
def test_library_bucket_equals_the_oracle(bidirectional, n_buckets, max_distance):
    h = binding.lib()
    h.spec_rel_bucket.restype = ctypes.c_int
    h.spec_rel_bucket.argtypes = [ctypes.c_int] * 4
    deltas = np.arange(-1200, 1201)
    want = relative_bucket(deltas, bool(bidirectional), n_buckets, max_distance)
    got = [h.spec_rel_bucket(int(d), bidirectional, n_buckets, max_distance) for d in deltas]
    assert got == want.tolist()


def test_bad_table_shapes_are_rejected():
    h = binding.lib()
    h.spec_rel_bucket.restype = ctypes.c_int
    h.spec_rel_bucket.argtypes = [ctypes.c_int] * 4
    assert h.spec_rel_bucket(1, 0, 6, 128) < 0
    assert h.spec_rel_bucket(1, 0, 32, 16) < 0
