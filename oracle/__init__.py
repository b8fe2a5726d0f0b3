"""TEST INFRASTRUCTURE ONLY.

CPU oracle for join-agg execution over tensor relations, written from the paper's definitions
(Definitions 3.1-3.7, Sections 3.3, 4.3, 5.3).  Only tests, the smoke check and the benchmark's
cpu_baseline / reference legs may import this package; the GPU library never does.
"""
from . import blocked, core, operators, relational  # noqa: F401
