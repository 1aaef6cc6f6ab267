"""Seeded synthetic inputs shared by the oracle-side tests and the CUDA-side tests (no method arithmetic)."""
from .gen import normal_bf16, f32_to_bf16_bits, bf16_bits_to_f32, bf16_bits_to_f64, rng  # noqa: F401
from .workloads import CONFIGS, DraftConfig, Workload, make_workload, scaled, sweep_configs, seq_lens, head_scales  # noqa: F401
from .workloads import Q_ALONG, recency_column, profile_window_mass, calibrate_delta  # noqa: F401
