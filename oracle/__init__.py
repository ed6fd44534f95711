"""CPU float64 oracle of the per-stage training step.  TEST INFRASTRUCTURE ONLY.

It states, as slowly and plainly as possible, what one HPP-Round computes on one
stage (Section 3.2 of the Asteroid paper): forward over M micro-batches, backward
over the same micro-batches, gradient accumulation, one parameter update.  The
paper fixes the round's structure; layer-level conventions (cross-correlation
with zero padding, training-mode BatchNorm with per-micro-batch statistics,
SGD with momentum, mean-reduced losses) are the usual definitions of these
layers, written out.

Only tests, the smoke check and the benchmark's CPU-baseline leg may use this
package.  It shares no code with the CUDA library and never calls it.

Pins (tests/test_oracle_*.py): brute-force direct convolution, central finite
differences, adjoint identities, BatchNorm closed forms and invariants, loss
special cases, closed-form SGD steps, the micro-batch accumulation invariant (also across the
devices of a data-parallel group),
agreement with torch.autograd in float64 on whole stages, and the K_p values the
paper prints for a three-stage pipeline; the storage-mirroring mode by tests/test_oracle_mirror.py;
the planner (oracle/planner.py) by closed forms and exhaustive search on tiny instances
(tests/test_oracle_planner.py).  No function here is unpinned.
"""
from .layers import *      # noqa: F401,F403
from .stage import *       # noqa: F401,F403
from . import planner       # noqa: F401
