"""CPU oracle for the RADAR speculative-step hot path.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
what the hot path computes.  It exists so that the CUDA library can be checked
element by element against something that can be read next to the paper.  It
shares no code with the CUDA path and never imports it.  Only the test-suite,
the smoke check and the benchmark's CPU-baseline / reference arm may import it;
the product path never routes through it.

Parity status of each function (what pins it is listed in its docstring):
  expand / frontier / rerank / tree build / attention / greedy / stochastic:
      pinned by brute force, invariants, library routines and a Monte-Carlo
      marginal (see tests/test_oracle_*.py).
  gate: arithmetic pinned against torch.nn.LSTM + Linear; the *reading* of which
      confidence scores feed the gate, of the decision rule and of the call
      schedule is not fixed by the paper's text -> "parity unpinned" against the
      authors' own code for those three readings.
"""
