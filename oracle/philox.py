"""Philox4x32-10 counter-based generator and the open uniform grid.

Test infrastructure (see the package docstring).  The paper does not say how
randomness is consumed (Algorithm 1 only writes r_i ~ U(0,1), x_i ~ q_i,
t ~ p').  This build fixes it as follows so that the CPU oracle and the CUDA
library can draw the same numbers without sharing code:

* generator: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11);
  key = the 64-bit seed (low word, high word); counter = (position,
  sequence index, purpose, 0); the first output word is used.
* purpose 0: the draft model's draw x ~ q for the token at `position`;
  purpose 1: the accept test r for the token at `position`;
  purpose 2: the final draw t ~ p' for the token at `position`.
  `position` is the absolute index of the token slot being decided, so the
  stream does not depend on how many iterations came before.
* uniform: u = (2k + 1) * 2**-24 with k the top 23 bits of the word.  u lies
  strictly inside (0, 1), is exact in fp32 and fp64, and is never 0 (so a
  token of probability zero can never pass r*q <= p with q > 0).

Pin: the three known-answer vectors of the Random123 distribution for
philox4x32-10 (tests/golden/philox4x32_10_kat.txt).
"""

import numpy as np

_M0 = 0xD2511F53
_M1 = 0xCD9E8D57
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = 0xFFFFFFFF

PURPOSE_DRAFT = 0
PURPOSE_ACCEPT = 1
PURPOSE_FINAL = 2


def philox4x32_10(counter, key):
    """One Philox4x32-10 block.  counter: 4 words, key: 2 words -> 4 words."""
    c0, c1, c2, c3 = (int(c) & _MASK for c in counter)
    k0, k1 = (int(k) & _MASK for k in key)
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        c0, c1, c2, c3 = (
            ((p1 >> 32) ^ c1 ^ k0) & _MASK,
            p1 & _MASK,
            ((p0 >> 32) ^ c3 ^ k1) & _MASK,
            p0 & _MASK,
        )
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return (c0, c1, c2, c3)


def word_to_uniform(word):
    """Map a 32-bit word to the open grid (2k+1)/2**24, k = word >> 9."""
    k = (int(word) & _MASK) >> 9
    return (2 * k + 1) / float(1 << 24)


def uniform(seed, position, sequence, purpose):
    """The uniform the method uses for (`position`, `sequence`, `purpose`)."""
    seed = int(seed)
    key = (seed & _MASK, (seed >> 32) & _MASK)
    words = philox4x32_10((position, sequence, purpose, 0), key)
    return word_to_uniform(words[0])


def uniforms_vec(seed, positions, sequences, purposes):
    """Vectorised `uniform` over broadcastable integer arrays (fp64 out)."""
    positions, sequences, purposes = np.broadcast_arrays(
        np.asarray(positions, dtype=np.uint64),
        np.asarray(sequences, dtype=np.uint64),
        np.asarray(purposes, dtype=np.uint64),
    )
    seed = int(seed)
    mask = np.uint64(_MASK)
    c0 = positions & mask
    c1 = sequences & mask
    c2 = purposes & mask
    c3 = np.zeros_like(c0)
    k0 = np.uint64(seed & _MASK)
    k1 = np.uint64((seed >> 32) & _MASK)
    s32 = np.uint64(32)
    for _ in range(10):
        p0 = np.uint64(_M0) * c0
        p1 = np.uint64(_M1) * c2
        c0, c1, c2, c3 = (
            ((p1 >> s32) ^ c1 ^ k0) & mask,
            p1 & mask,
            ((p0 >> s32) ^ c3 ^ k1) & mask,
            p0 & mask,
        )
        k0 = (k0 + np.uint64(_W0)) & mask
        k1 = (k1 + np.uint64(_W1)) & mask
    k = c0 >> np.uint64(9)
    return (2.0 * k.astype(np.float64) + 1.0) / float(1 << 24)
