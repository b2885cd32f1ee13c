"""B200 (sm_100a) library for the hot path of the Redistributing-Drafter-Kernels sampler.

`binding` wraps the C ABI declared in include/rdk.h; `build` compiles the CUDA sources in-tree.
"""
from . import binding  # noqa: F401
from .binding import (KeptIndex, RdkError, rdk_build_affinity, rdk_emit_sequences, rdk_prepare_ids, rdk_redistribute_exact,
                      rdk_redistribute_exact_static,
                      rdk_redistribute_linear, rdk_sample_and_verify, rdk_sample_and_verify_host,
                      rdk_stream_geometry, rdk_version, rdk_sample_and_verify_prior, rdk_redistribute_linear_prior,
                      rdk_sample_route, rdk_test_set_spin_limit)

__all__ = ["binding", "KeptIndex", "RdkError", "rdk_build_affinity", "rdk_emit_sequences", "rdk_prepare_ids",
           "rdk_redistribute_exact", "rdk_redistribute_linear", "rdk_sample_and_verify",
           "rdk_sample_and_verify_host", "rdk_stream_geometry", "rdk_version", "rdk_sample_and_verify_prior",
           "rdk_redistribute_linear_prior", "rdk_redistribute_exact_static", "rdk_sample_route",
           "rdk_test_set_spin_limit"]
