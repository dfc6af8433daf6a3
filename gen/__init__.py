"""Seeded synthetic input generators shared by the tests, the benchmark and the CPU oracle's callers."""
from .workloads import (CONFIGS, LayerInputs, Workload, bf16_bits_to_f32, concentration_to_logit_std, config,
                        f32_to_bf16_bits, make_layer, small_workload)

__all__ = ["CONFIGS", "LayerInputs", "Workload", "bf16_bits_to_f32", "concentration_to_logit_std", "config",
           "f32_to_bf16_bits", "make_layer", "small_workload"]
