"""CPU oracle for the token-wise RNN-T beam search (Algorithm 1, Eq. 1-7).

TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Plain, slow, fp64, natural-log-space
numpy written from the paper's equations and algorithm.  It shares no code
with the CUDA path and must never be imported by it; only the test-suite,
the smoke check and the benchmark's CPU-baseline leg may call it.

Modules
  rnnt_model        joiner + softmax (Sec. 3.1), stateless / LSTM predictor
  segment_math      Eq. 3-7 in their explicit double-sum form
  token_wise_search Algorithm 1
  standard_search   the frame-wise breadth-first search of Eq. 1 (a separately
                    written routine; Algorithm 1 at S=1 must reproduce it)
  exact_forward     textbook RNN-T forward recursion and brute-force alignment
                    enumeration (what Algorithm 1 sums when nothing is pruned)

Parity pins: every function here is pinned by tests/test_oracle_*.py against
closed forms, invariants, a library LSTM, hand-worked values under
tests/golden/ and brute force; none is "parity unpinned".  The accuracy
columns of the paper's tables (WER) are not reproducible without its data
and are out of scope.
"""
