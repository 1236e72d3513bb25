"""Nested gradient code (arXiv 2212.08580) hot path for B200: thin ctypes binding over libngc.so.

All arithmetic of the path runs inside the CUDA library; this package only marshals
arguments.  Importing it fails loudly if the library has not been built.
"""
from .binding import (NGC_BF16, NGC_F32, NGC_F64, NGC_LOGISTIC, NGC_LSQ, NGC_MLP, NGC_SOFTMAX, Model, NgcError, Plan,
                      StepInfo, dense_schedule, gd_update, latency_cdf_gc, latency_cdf_ngc, lib_path, load_library, sample_times)

__all__ = ["Plan", "Model", "StepInfo", "NgcError", "load_library", "lib_path", "sample_times", "dense_schedule", "gd_update", "latency_cdf_gc", "latency_cdf_ngc",
           "NGC_LSQ", "NGC_LOGISTIC", "NGC_SOFTMAX", "NGC_MLP", "NGC_F32", "NGC_BF16", "NGC_F64"]
