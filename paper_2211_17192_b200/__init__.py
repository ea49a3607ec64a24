"""B200-native speculative decoding hot path (verify pass, speculative sampling,
KV rollback) behind a C-ABI library.

Importing the package is cheap and loads nothing native: the CUDA library is
opened by `paper_2211_17192_b200.binding` on first use and raises if it has not
been built.  `paper_2211_17192_b200.workloads` (seeded synthetic inputs) has no
dependency on the native library.
"""

__all__ = ["binding", "build", "workloads"]
