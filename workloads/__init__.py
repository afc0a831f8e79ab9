"""Seeded synthetic inputs for the Slim-DP round: shapes, sizes and value
distributions only.  Nothing in this package scores, selects, samples,
packs or merges; both the CPU oracle's tests and the CUDA library's tests
and benchmark draw their inputs from here."""
from .configs import CONFIGS, Config, Segment, get_config, scaled_config
from .generate import weights, grads, all_inputs

__all__ = ["CONFIGS", "Config", "Segment", "get_config", "scaled_config",
           "weights", "grads", "all_inputs"]
