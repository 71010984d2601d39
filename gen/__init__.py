"""Seeded synthetic input generators shared by the oracle tests and the CUDA path."""
from .workloads import (BASE_SEED, CONFIGS, Inputs, Workload, distinct_positions, hash_u64,
                        make_inputs, normal_f64, normal_tensor, sample_rows, scaled, uniform_int)

__all__ = ["BASE_SEED", "CONFIGS", "Inputs", "Workload", "distinct_positions", "hash_u64",
           "make_inputs", "normal_f64", "normal_tensor", "sample_rows", "scaled", "uniform_int"]
