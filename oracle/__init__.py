"""CPU oracle for the ASER W4A8 + low-rank linear layer (arXiv 2411.07762).

TEST INFRASTRUCTURE ONLY.  A plain, slow restatement of the method written from
the paper: `forward` (C loops, `aser_oracle.c`) is what the CUDA library is
compared against; `construct` (NumPy fp64) builds the smoothing vector, the int4
weights and the whitening-SVD factors that the forward pass consumes.  Nothing
here is shared with, imported by, or falls back from the CUDA path.

Pinned by tests/test_oracle_*.py against closed forms, brute force, special
cases and the paper's printed overhead table.  Not pinned ("parity unpinned"):
the numerical values of the factors L_A, L_B themselves and any accuracy or
perplexity figure -- the paper prints no worked example and its models and
datasets are not available; only invariants of the factors are checked.
"""
from . import build as _build  # noqa: F401
from . import forward, construct  # noqa: F401
