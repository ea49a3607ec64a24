"""Pins for oracle.philox: known-answer vectors and the uniform grid."""
import os

import numpy as np

from conftest import read_golden
from oracle import philox


def test_known_answer_vectors(golden_dir):
    rows = read_golden(os.path.join(golden_dir, "philox4x32_10_kat.txt"))
    assert len(rows) == 3
    for row in rows:
        words = [int(w, 16) for w in row]
        assert list(philox.philox4x32_10(words[0:4], words[4:6])) == words[6:10]


def test_uniform_is_on_the_open_grid():
    for word, expected in [(0, 1 / 2**24), (0xFFFFFFFF, 1 - 1 / 2**24), (1 << 9, 3 / 2**24)]:
        assert philox.word_to_uniform(word) == expected
    u = philox.uniforms_vec(7, np.arange(20000), 0, 1)
    assert u.min() > 0.0 and u.max() < 1.0
    assert np.all(u.astype(np.float32).astype(np.float64) == u)  # exact in fp32
    # mean and variance of U(0,1) within 5 sigma
    assert abs(u.mean() - 0.5) < 5 * np.sqrt(1 / 12 / u.size)
    assert abs(u.var() - 1 / 12) < 5 * np.sqrt(1 / 180 / u.size)


def test_vector_form_equals_scalar_form():
    seed = 0x1234567_89ABCDEF
    pos = np.array([0, 1, 17, 2**31 + 5])
    for seq in (0, 3):
        for purpose in (0, 1, 2):
            vec = philox.uniforms_vec(seed, pos, seq, purpose)
            for i, p in enumerate(pos):
                assert vec[i] == philox.uniform(seed, int(p), seq, purpose)


def test_streams_differ_by_purpose_sequence_and_seed():
    base = philox.uniform(1, 5, 0, 0)
    assert base != philox.uniform(1, 5, 0, 1)
    assert base != philox.uniform(1, 5, 1, 0)
    assert base != philox.uniform(2, 5, 0, 0)
    assert base != philox.uniform(1 + (1 << 32), 5, 0, 0)  # high key word is used
