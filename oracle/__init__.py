"""fp64 CPU oracle for budgeted-KV decode attention (BaKlaVa, arXiv 2502.13176).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain definition that the
CUDA library is checked against.  It is imported by the test-suite, by the
smoke check and by the benchmark's CPU-baseline leg, and by nothing else; the
product path never calls it and shares no code with it.

Everything here is numpy in float64, one function per step of the method, in
the paper's order and notation:

  attention.py   Eq. 1 / Eq. 4 / Eq. 7   softmax attention, decode and causal
  profiling.py   Algorithm 1             head similarity and KV-cache importance
  allocation.py  Algorithm 2             threshold / reduction budget reallocation
  eviction.py    Eq. 5-6 + policy        which entries stay, bulk compaction
  cache.py       Eq. 4-7 iterated        one head's slab and one decode step

Parity status: every function is pinned by the CPU tests (closed forms,
library routines, brute force, invariants) except the choice of the search
parameters (t, r) and anything that needs model weights or benchmark data:
those are "parity unpinned" and are not part of this oracle.
"""
