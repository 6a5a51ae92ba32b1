"""B200-native kernel-halving compression + weighted attention (arXiv 2606.10944 hot path).

``compress`` / ``attend`` and friends are thin argument-marshalling wrappers over the C-ABI
CUDA library in ``csrc/``; they are loaded on first use so that the input generators in
``workloads`` stay importable on machines without the built library.
"""
_BINDING_NAMES = {
    "compress", "compress_ragged", "compress_ragged_count", "express_compress", "express_prefill", "attend_workspace_bytes", "Stream", "ElmStream", "attend", "compress_status", "attend_status", "attend_static", "attend_static_status", "ATTEND_STATIC_SCRATCH_BYTES", "compress_attend_host", "workspace_bytes", "default_delta_levels",
    "ElmParams", "ElmError", "library_path", "load_library", "make_params", "profile_enable",
    "profile_read", "version", "debug_round_check", "EXPORTED_SYMBOLS", "STAGE_NAMES", "launch_count", "host_call_scratch_bytes",
}


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
