"""B200-native verify step of speculative decoding for autoregressive image generation.

Three hand-written sm_100a kernels behind a C-ABI shared library (see include/hawk.h):
hawk_verify_attn, hawk_head_proj, hawk_cfg_accept.  The Python names below only marshal torch
tensors into pointers and sizes; the shared library is loaded on first use and a missing build
raises instead of falling back to anything.
"""
__version__ = "0.1.0"

_BINDING_NAMES = (
    "load_library", "library_path", "HawkError", "status_string", "version",
    "verify_attn", "verify_attn_workspace_bytes", "head_proj",
    "cfg_accept", "cfg_accept_workspace_bytes",
    "verify_step_host", "StepHostArgs",
    "cfg_accept_noalloc", "cfg_accept_noalloc_max_rows", "tree_accept", "verify_attn_tree",
    "spec_cache_slots", "spec_cache_slot", "spec_cache_new", "spec_cache_clear", "spec_cache_put",
    "pool_build", "pool_sample", "pool_sample_workspace_bytes",
    "head_proj_cfg", "cfg_accept_guided", "tree_accept_guided",
)


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
