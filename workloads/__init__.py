"""Seeded synthetic input generators shared by the CUDA tests, the bench and the oracle tests.

Holds no part of the recall method's arithmetic.
"""
from .recall_inputs import (CONFIGS, PAPER_DEFAULT_MAX_SIZES, PAPER_DEFAULT_WIN_SIZES,
                            RecallInputs, RecallWorkload, layer_sweep_workloads, make_inputs,
                            small_workload)

__all__ = ["CONFIGS", "PAPER_DEFAULT_MAX_SIZES", "PAPER_DEFAULT_WIN_SIZES", "RecallInputs",
           "RecallWorkload", "layer_sweep_workloads", "make_inputs", "small_workload"]
