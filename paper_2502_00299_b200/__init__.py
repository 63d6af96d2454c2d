"""ChunkKV prefill-time KV-cache compression on B200 (sm_100a): thin Python binding.

All work runs in the CUDA kernels of ``libchunkkv.so`` (see ``include/chunkkv.h``); the
functions here only marshal ``torch`` tensors into pointers. There is no CPU fallback: the
first use of any function raises ImportError if the shared library has not been built
(``python -m paper_2502_00299_b200.build``). The binding is loaded on first attribute access
so that the build module itself can be imported before the library exists.
"""
_EXPORTS = (
    "ChunkKVError", "LIB_PATH", "Lane", "Pipe", "budget_from_ratio", "compress_layer", "compress_layer_alg1",
    "compress_layer_host", "compress_layer_paged", "compress_layer_strided", "compress_model", "compress_model_paged", "compress_model_strided", "gather_paged", "window_queries", "out_len_alg1", "select_alg1",
    "device_status", "ensure_workspace", "gather", "jaccard", "lib", "num_chunks", "num_kept_chunks", "out_len", "profile_enable",
    "profile_read", "score", "select", "set_workspace", "strerror", "workspace_bytes",
)
__all__ = list(_EXPORTS)


def __getattr__(name):
    if name in _EXPORTS:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
