"""Negligible-cost approximation models: a bigram table, on the CPU.

Test infrastructure (see the package docstring).

The paper's experiments include trivial drafts (unigram and bigram models,
Section 4) whose cost is negligible (c close to 0).  A bigram model maps the
last token to next-token logits by one table look-up.  The class below has the
interface of the decoders (forward_rows / forward_full / truncate / reset) so
that the generation loop takes it as M_q unchanged; it keeps no state besides
the number of tokens it has been fed.

Pins (tests/test_oracle_generate.py): logits depend on the last token only;
with the table built from a target that is itself a bigram model the draft
equals the target and every guess is accepted; T = 0 output equals the
target's greedy output whatever the table.
"""

import numpy as np


class BigramTable:
    def __init__(self, table, dtype=np.float64):
        self.table = np.asarray(table, dtype=dtype)  # [vocab, vocab]: row = last token
        self._fed = 0

    def reset(self):
        self._fed = 0

    @property
    def cached_len(self):
        return self._fed

    def truncate(self, length):
        self._fed = min(self._fed, int(length))

    def forward_rows(self, tokens):
        tokens = np.asarray(tokens, dtype=np.int64)
        self._fed += len(tokens)
        return self.table[tokens]

    def forward_full(self, tokens):
        return self.table[np.asarray(tokens, dtype=np.int64)]
