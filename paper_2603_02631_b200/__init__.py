"""Speculative-prefill token scoring, chunk selection and span compaction for NVIDIA B200.

Thin Python binding over the C-ABI library ``libspf.so`` (see ``include/spf.h``).  Every step of the
path runs in the library's CUDA kernels; PyTorch only provides device memory and streams.
The first use of any name below loads the library and raises ImportError if it has not been built
(``python -m paper_2603_02631_b200.build``): there is no CPU fallback.  Only the ``build`` submodule
can be imported without the library, since it is what produces it.
"""
import importlib

_BINDING_NAMES = (
    "LIB_PATH", "SpfError", "Selection", "Selector", "PromptBuffers", "PagedPromptBuffers", "spf_score_paged", "spf_score_paged_workspace_bytes", "lib", "spf_chunk_pool", "spf_chunk_pool_edge", "spf_select_topk_forced", "spf_compact_spans",
    "spf_keep_count", "spf_keep_rate", "spf_snap_budget", "spf_concat_with_delim", "spf_last_error", "spf_score", "spf_score_extra", "spf_score_shard_lse", "spf_score_shard_apply", "spf_selftest_bounded_wait", "spf_set_score_path", "spf_score_static", "spf_score_workspace_bytes", "spf_select_topk",
    "spf_status_string", "spf_version", "spf_compress_host", "spf_compress_host_arena_bytes", "Fp8PromptBuffers", "spf_select_compact", "spf_score_shard_lse_ex", "spf_score_shard_apply_ex", "BatchSelector", "spf_chunk_pool_batch", "spf_select_topk_batch", "spf_compact_spans_batch", "spf_score_fp8", "spf_score_fp8_workspace_bytes",
)
__all__ = list(_BINDING_NAMES) + ["binding"]


def __getattr__(name):
    if name == "binding" or name in _BINDING_NAMES:
        binding = importlib.import_module(".binding", __name__)
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
