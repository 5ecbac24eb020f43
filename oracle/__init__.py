"""CPU oracle for the PipeMare training step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, by-eye-checkable statement of what the hot path computes:
the delayed-update recurrence of Section 2.1 with PipeMare's delays (Table 1),
learning-rate rescheduling (T1, Eq. 2 of Section 3.1), discrepancy correction
(T2, Section 3.2) and the momentum update of Appendix B.3, in the paper's own
microbatch-major form with a queue of stale weight versions.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA library and imports nothing
from it; the only module both sides use is the seeded input generator.

Pins (what ties each part to something other than itself) are listed in each
module's docstring.  Parts with no pin from the paper or from mathematics:
  * full MLP training trajectories on the synthetic workloads -- parity
    unpinned (the paper prints no losses for them); they are covered only
    through the layer-level finite-difference checks and the recurrence-level
    special cases.
"""
