"""CPU checker for Pipelined Backpropagation with Spike Compensation and
Linear Weight Prediction.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow numpy program in float64,
written from the paper's equations so that it can be read against them.  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may use it; the
CUDA library never imports it and shares no code, table or helper with it.

Pins (see tests/test_oracle_*.py): the optimizer against closed forms and the
paper's state-transition recurrences (Appendix "State Transition Equations");
each layer against finite differences, brute-force loops and torch CPU
autograd; the schedule against the one-stage reduction to plain SGD with
momentum, the 2S-1 latency and the per-stage staleness of Eq. (F_i).

Parity unpinned: the paper prints no PB+SC+LWP trajectory for S > 1, so the
whole-pipeline result is pinned only through those pieces plus an independent
per-sample replay of every gradient from logged weight versions.
"""
from .optimizer import StageOptimizer, sc_coefficients
from .pipeline import PBOracle
from . import layers

__all__ = ["StageOptimizer", "sc_coefficients", "PBOracle", "layers"]
