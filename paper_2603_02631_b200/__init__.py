"""Speculative-prefill token scoring, chunk selection and span compaction for NVIDIA B200.

Thin Python binding over the C-ABI library ``libspf.so`` (see ``include/spf.h``).  Every step of the
path runs in the library's CUDA kernels; PyTorch only provides device memory and streams.
Importing this package loads the library and raises if it has not been built
(``python -m paper_2603_02631_b200.build``): there is no CPU fallback.
"""
from .binding import (  # noqa: F401
    LIB_PATH,
    SpfError,
    Selection,
    Selector,
    lib,
    spf_chunk_pool,
    spf_compact_spans,
    spf_keep_count,
    spf_last_error,
    spf_score,
    spf_score_workspace_bytes,
    spf_select_topk,
    spf_status_string,
    spf_version,
)
