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
  prefill.py     Eq. 1 column sums       accumulated attention a prompt leaves on its tokens
  search.py      Algorithm 3             parameter search loop with an attention-output loss
  fp8.py         quantised slabs         FP8 E4M3 codec and the per-head scale rule

Parity status: every function is pinned by the CPU tests (closed forms,
library routines, brute force, invariants).  The search loop and its loss are
pinned as arithmetic; which (t, r) is best for a real model, and anything else
that needs model weights or benchmark data, is "parity unpinned" and is not
part of this oracle.
"""
