"""Seeded synthetic input generators (no method arithmetic lives here)."""
from .configs import (CONFIGS, RDKConfig, embeddings, kept_ids, make_inputs, tiny_config, to_f64,
                      token_ranks)
from .philox import philox4x32_10, uniforms

__all__ = ["CONFIGS", "RDKConfig", "embeddings", "kept_ids", "make_inputs", "tiny_config",
           "to_f64", "token_ranks", "philox4x32_10", "uniforms"]
