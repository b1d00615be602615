"""Few-bit stochastic rounding on B200: thin Python binding over libfbsr.so.

Every function here only marshals arguments (torch tensors -> device pointers,
current stream -> cudaStream_t) and calls the C-ABI entry point of the same
name; all arithmetic runs in the CUDA kernels.  There is no CPU fallback: the
first use of any entry point loads ``libfbsr.so`` and raises ImportError if it
has not been built (``python -m paper_2504_20634_b200.build``).
"""
import importlib

_BINDING_NAMES = (
    "FMT", "VARIANT", "CODE_DTYPE", "VIEW_DTYPE", "FbsrError", "fbsr_round", "fbsr_round_bits", "fbsr_round_lp", "fbsr_round_mx",
    "fbsr_round_desc", "fbsr_format_desc_valid", "FbsrFormatDesc", "format_desc",
    "fbsr_round_stats", "fbsr_round_stats_noalloc", "stats_from_bytes", "fbsr_sgd_update", "fbsr_adam_update", "fbsr_accumulate", "fbsr_qat_update", "fbsr_qat_adamw_step", "fbsr_round_host",
    "fbsr_tile_elements", "fbsr_launch_count", "fbsr_stats_workspace_bytes",
    "fbsr_round_host_min_workspace", "fbsr_version", "fbsr_status_string", "library_path",
)


def __getattr__(name):
    # Loaded on first use so that the build module can be imported before the library exists.
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(".binding", __name__), name)
    raise AttributeError("module %r has no attribute %r" % (__name__, name))


def __dir__():
    return sorted(list(globals()) + list(_BINDING_NAMES))
