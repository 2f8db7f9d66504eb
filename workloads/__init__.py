"""Seeded synthetic workloads (frames + detector heads) shared by the oracle tests, the
CUDA parity tests and the benchmark.  Holds none of the stage's arithmetic."""
from .synth import WORKLOADS, Workload, Batch, make_batch, make_heads, num_anchors, rows_to_planes  # noqa: F401
