"""Compressed-sensing-guided sparse FFN step for B200: thin Python binding over the C library.

The functions here only marshal arguments (torch tensors -> device pointers) into the
``extern "C"`` entry points declared in ``include/cs.h``; every step of the path runs in the
CUDA kernels under ``csrc/``.  There is no CPU implementation: loading fails loudly if the
shared library is missing and calls fail on non-CUDA tensors.
"""
from .binding import (  # noqa: F401
    CSError, Layer, Plan, StepOptions, cs_bucket, cs_ffn_exec, cs_ffn_exec_shared, cs_ffn_exec_static, cs_layer_step,
    cs_layer_step_ex, cs_layer_step_fallback, cs_layer_step_host, cs_prompt_support, cs_recover, cs_recover_ex,
    cs_recover_warm, cs_sketch, cs_sketch_srht, cs_support_drift, cs_support_drift_ratio, cs_uds_budget,
    exported_symbols, library_path, load_library,
)
