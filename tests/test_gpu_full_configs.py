"""Parity at the full sizes of the five workload configurations, in the launch configuration bench.py times.

Inputs are generated on the GPU and the same bytes are copied to the host for the oracle.  Both scoring paths
(fused single kernel, general two-sweep) are checked against one oracle run per prompt; of the ragged batch every
prompt is checked on the fused path (the one the bench times), the shortest and the longest on both.
"""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits, make_prompt

from parity_util import IMPORTANCE_RTOL, assert_importance_close, assert_selection_matches

pytestmark = pytest.mark.gpu

CASES = [
    ("small32k", [0]),
    ("wide64k", [0]),
    ("long128k", [0]),
    ("ragged8", None),      # all prompts of the batch
]


def _prompt_indices(name, idx):
    return idx if idx is not None else list(range(len(CONFIGS[name].lengths)))


def _paths(name, index):
    """Kernel paths to check for this prompt: both, except the middle prompts of the ragged batch (fused only)."""
    lengths = CONFIGS[name].lengths
    if len(lengths) == 1 or index in (int(np.argmin(lengths)), int(np.argmax(lengths))):
        return (2, 1)
    return (2,)


@pytest.mark.parametrize("name,idx", CASES)
def test_full_size_config(name, idx):
    import paper_2603_02631_b200 as spf
    cfg = CONFIGS[name]
    for index in _prompt_indices(name, idx):
        prompt = make_prompt(cfg, index, "cuda")
        n = prompt.n_tokens
        host_q = bf16_bits(prompt.q)
        host_k = [bf16_bits(x) for x in prompt.k]
        ids, cs, ce = (t.cpu().numpy().astype(np.int64) for t in (prompt.token_ids, prompt.char_start, prompt.char_end))
        want_imp, want_lse = oracle.token_importance(host_q, host_k)
        del host_k
        want_scores = oracle.chunk_means(oracle.avg_pool(want_imp, cfg.pool_kernel), cfg.chunk)
        sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n,
                           chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)
        for path in _paths(name, index):
            previous = spf.spf_set_score_path(path)
            try:
                for keep in cfg.keep:
                    sel.dev_status.zero_()
                    got = sel.run(prompt.q, prompt.k, prompt.token_ids, prompt.char_start, prompt.char_end, keep)
                    torch.cuda.synchronize()
                    assert int(sel.dev_status.item()) == 0
                    got = got.host()
                    assert_importance_close(got["importance"], want_imp)
                    np.testing.assert_allclose(got["lse"], want_lse, rtol=0, atol=2e-4)
                    np.testing.assert_allclose(got["chunk_scores"], want_scores, rtol=IMPORTANCE_RTOL)
                    k = oracle.keep_count(len(want_scores), keep)
                    kept = oracle.select_topk(want_scores, k)
                    o_ids, o_pos, o_tok, o_ch = oracle.compact(kept, cfg.chunk, n, ids, cs, ce)
                    ref = dict(k=k, kept=kept, chunk_scores=want_scores, ids=o_ids, pos=o_pos, tok_spans=o_tok, char_spans=o_ch)
                    assert_selection_matches(got, ref, prompt)
                    # strong needle spans must be kept (their chunks lie far above the boundary)
                    kept_set = set(got["kept"].tolist())
                    if keep >= 0.10:
                        for start, length, strong in prompt.needles:
                            if strong:
                                for j in range((start + cfg.chunk - 1) // cfg.chunk, (start + length) // cfg.chunk):
                                    assert j in kept_set, f"{name}: chunk {j} of a strong needle span was dropped"
            finally:
                spf.spf_set_score_path(previous)
        del prompt, sel
        torch.cuda.empty_cache()
