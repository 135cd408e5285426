"""Seeded synthetic workloads (shapes + input generators) shared by all tests and benches."""
from .configs import (CONFIGS, SWEEP_BATCHES, SWEEP_BUDGETS, VScanConfig, schedule_points, sweep_config,
                      tiny_config)
from .generate import (attention_rows_one, features_one, redraw_token, round_to_dtype,
                       stage1_inputs, stage2_inputs)

__all__ = ["CONFIGS", "SWEEP_BATCHES", "SWEEP_BUDGETS", "VScanConfig", "schedule_points", "sweep_config",
           "tiny_config", "attention_rows_one", "features_one", "redraw_token", "round_to_dtype",
           "stage1_inputs", "stage2_inputs"]
