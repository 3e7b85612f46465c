"""Seeded synthetic scheduler workloads.

This package only draws inputs (loss histories, iteration-time samples,
cluster sizes).  It contains none of the scheduler's arithmetic and is the one
module that both the CPU oracle's tests and the CUDA library's tests import.
"""

from .synthetic import (CONFIGS, Workload, make_workload, make_time_samples, make_unfittable_histories,
                        true_curve)

__all__ = ["CONFIGS", "Workload", "make_workload", "make_time_samples", "make_unfittable_histories",
           "true_curve"]
