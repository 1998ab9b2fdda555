"""Seeded synthetic clusters, workflow forests and ready-call batches.

This package only draws inputs (shapes, sizes, value distributions and graph
structure).  It holds none of the scheduler's arithmetic: no latency model, no
longest path, no scoring.  Both the CPU oracle's tests and the CUDA library's
tests and benchmark feed on the same arrays produced here.
"""
from .workloads import (CALL_DTYPE, CONFIG_NAMES, Workload, make_decode_queue, make_workload,
                        sub_forest)

__all__ = ["CALL_DTYPE", "CONFIG_NAMES", "Workload", "make_decode_queue", "make_workload", "sub_forest"]
