"""Float64 CPU oracle for the AIS log-probability / correction path.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain statement of what
the GPU library computes.  It shares no code with the CUDA path and must never
be imported by the product package; only the test-suite, the smoke check and
the CPU-baseline / reference legs of the benchmark may call it.

Modules
-------
e4m3      bit-exact FP8-E4M3 codec and per-block quantisation (Section 2.1,
          quantisation equation, instantiated for the E4M3 grid)
ais       log-probabilities, importance ratios, GRPO advantages, the three
          AIS diagnostics, the mixing coefficient, the rectified loss and its
          gradient with respect to the hidden states (Section 3, Algorithm 1,
          AIS-GRPO objective)

Parity status: every function in both modules is pinned by the CPU tests
(closed forms and hand numbers, brute force, finite differences, an independent
float8 library used as a black box), the monitor outputs kl_k1 / mean_abs_dp of
ais.diagnostics included.  Nothing is "parity unpinned".  The oracle returns
plain arrays only; byte layouts of the C ABI are not its business.
"""

from . import e4m3, ais  # noqa: F401
