"""Seeded synthetic input generators shared by the oracle's tests and the CUDA path's tests."""
from .gen import (C1, C2, C3, C4_5, C4_10, C4_20, C5, WORKLOADS, Workload, decode_inputs,
                  directions, head_budgets, prompt)

__all__ = ["C1", "C2", "C3", "C4_5", "C4_10", "C4_20", "C5", "WORKLOADS", "Workload",
           "decode_inputs", "directions", "head_budgets", "prompt"]
