"""Few-bit stochastic rounding on B200: thin Python binding over libfbsr.so.

Every function here only marshals arguments (torch tensors -> device pointers,
current stream -> cudaStream_t) and calls the C-ABI entry point of the same
name; all arithmetic runs in the CUDA kernels.  There is no CPU fallback: if
the shared library is missing, importing :mod:`paper_2504_20634_b200.binding`
raises.
"""
from .binding import (  # noqa: F401
    FMT, VARIANT, CODE_DTYPE, FbsrError, fbsr_round, fbsr_round_bits, fbsr_round_stats,
    fbsr_sgd_update, fbsr_adam_update, fbsr_accumulate, fbsr_round_host, fbsr_tile_elements,
    fbsr_launch_count, fbsr_stats_workspace_bytes, fbsr_round_host_min_workspace,
    fbsr_version, fbsr_status_string, library_path,
)
