"""CPU oracle (test infrastructure only; never imported by the CUDA path)."""
from .spf_oracle import (  # noqa: F401
    attention_logits,
    avg_pool,
    bf16_to_f64,
    chunk_means,
    compact,
    compress,
    concat_with_delim,
    keep_count,
    keep_rate,
    merge_adjacent,
    select_topk,
    select_topk_forced,
    snap_budget,
    softmax_rows,
    token_importance,
)
