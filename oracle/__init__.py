"""CPU oracle (test infrastructure only; never imported by the CUDA path)."""
from .spf_oracle import (  # noqa: F401
    attention_logits,
    avg_pool,
    bf16_to_f64,
    chunk_means,
    compact,
    compress,
    keep_count,
    merge_adjacent,
    select_topk,
    softmax_rows,
    token_importance,
)
