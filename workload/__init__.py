"""Seeded synthetic inputs and workload shapes (no arithmetic of the method lives here).

Both the CPU oracle's callers and the CUDA path's callers draw their inputs from
this package; it imports neither of them.
"""
from .synth import (LAYER_ELEMS, Workload, baseline_workloads, grad_slab, normal_f32, theta0_slab,
                    scaled)

__all__ = ["LAYER_ELEMS", "Workload", "baseline_workloads", "grad_slab", "normal_f32", "theta0_slab",
           "scaled"]
