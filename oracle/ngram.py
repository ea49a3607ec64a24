"""Negligible-cost approximation models: a bigram table and a copy-from-context rule, on the CPU.

Test infrastructure (see the package docstring).

The paper's experiments include trivial drafts (unigram and bigram models,
Section 4) whose cost is negligible (c close to 0).  A bigram model maps the
last token to next-token logits by one table look-up.  The class below has the
interface of the decoders (forward_rows / forward_full / truncate / reset) so
that the generation loop takes it as M_q unchanged; it keeps no state besides
the number of tokens it has been fed.

Section 3.6 also suggests a parameter-less draft that copies tokens from the
context where a matching prefix is found, without giving a procedure.
Reading (`CopyFromContext`): with s the sequence so far and n the match
length, the guess is the token that followed the most recent earlier
occurrence of the last n tokens of s; if there is none, or s is shorter than
n + 1, the last token is repeated.  q is one-hot at the guess (logit 0, -inf
elsewhere), so a guess x is accepted with probability p(x) and a rejection
draws from p with x removed (Algorithm 1 with a deterministic M_q).

Pins (tests/test_oracle_generate.py): the copy rule on hand-written sequences;
on a target that repeats with a fixed period every guess after the first
period is accepted and the tokens per iteration reach gamma + 1; the accept
frequency of a one-hot draft equals p(x); T = 0 output equals the target's
greedy output.  For the table: logits depend on the last token only;
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


class CopyFromContext:
    def __init__(self, vocab, ngram):
        self.vocab, self.ngram = int(vocab), int(ngram)
        self.history = []

    def reset(self):
        self.history = []

    @property
    def cached_len(self):
        return len(self.history)

    def truncate(self, length):
        self.history = self.history[: int(length)]

    def guess(self, seq):
        """The token that followed the most recent earlier occurrence of seq's last n tokens."""
        n, last = self.ngram, len(seq) - 1
        for j in range(last - 1, n - 2, -1):  # j = where an earlier occurrence would end
            if seq[j - n + 1 : j + 1] == seq[last - n + 1 : last + 1]:
                return seq[j + 1]
        return seq[last]

    def _row(self, seq):
        row = np.full(self.vocab, -np.inf)
        row[self.guess(seq)] = 0.0
        return row

    def forward_rows(self, tokens):
        rows = []
        for t in tokens:
            self.history.append(int(t))
            rows.append(self._row(self.history))
        return np.stack(rows)

    def forward_full(self, tokens):
        seq = [int(t) for t in tokens]
        return np.stack([self._row(seq[: i + 1]) for i in range(len(seq))])
