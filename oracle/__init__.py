"""CPU oracle for the activation-sampling estimator of Randomized Automatic
Differentiation (Sec. 4.2 of the paper).

TEST INFRASTRUCTURE ONLY.  Plain numpy in float64, written from the paper and
from the published definition of Philox-4x32-10; slow on purpose, with no
blocking, fusion or reordering.  It shares no code with the CUDA library and
never imports it.  Only the tests, the smoke check and the benchmark's CPU
baseline may import this package; the product path never does.

Parity status
  * estimator, exact forward/backward, loss, store layout, byte accounting:
    pinned by tests/test_oracle_*.py (p = 1 equals exact backprop, exhaustive
    expectation and variance over all masks, finite differences, torch
    autograd in float64, the memory figures printed in App. A and Table 1).
  * Philox-4x32-10: pinned against the known-answer vectors published with the
    generator's reference code (tests/golden), an independent big-integer
    restatement, invertible rounds and uniformity.
  * the with-replacement law, the fixed-count law and the random projection:
    pinned by tests/test_oracle_replace.py, test_oracle_fixed.py and
    test_oracle_project.py (all draw sequences / subsets / sign matrices of
    tiny layers, closed-form variances, special cases that are exact).
"""
from . import philox, rad, memory_model, irnn, cnn  # noqa: F401
