"""GPU parity in the regimes the paper ran beyond the five workload configurations: chunk 128 (its code
setting, Appendix A.3), prompts of a quarter of a million tokens (its LongBench-v2 lengths, Section 4), and
keep rates from 3 % to 50 % (Tables 1 and 2).  Few layers and heads, so that the fp64 oracle stays within
seconds; the lengths, chunk counts and keep counts are the paper's.
"""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, small_config

from parity_util import IMPORTANCE_RTOL, assert_importance_close, assert_selection_matches

pytestmark = pytest.mark.gpu


def _check(cfg, keeps, paths=(2, 1)):
    import paper_2603_02631_b200 as spf
    prompt = make_prompt(cfg, 0, "cuda")
    n = prompt.n_tokens
    want_imp, want_lse = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k])
    want_scores = oracle.chunk_means(oracle.avg_pool(want_imp, cfg.pool_kernel), cfg.chunk)
    ids, cs, ce = (t.cpu().numpy().astype(np.int64) for t in (prompt.token_ids, prompt.char_start, prompt.char_end))
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n,
                       chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)
    for path in paths:
        previous = spf.spf_set_score_path(path)
        try:
            for keep in keeps:
                sel.dev_status.zero_()
                got = sel.run(prompt.q, prompt.k, prompt.token_ids, prompt.char_start, prompt.char_end, keep)
                torch.cuda.synchronize()
                assert int(sel.dev_status.item()) == 0
                got = got.host()
                assert_importance_close(got["importance"], want_imp)
                np.testing.assert_allclose(got["lse"], want_lse, rtol=0, atol=2e-4)
                np.testing.assert_allclose(got["chunk_scores"], want_scores, rtol=IMPORTANCE_RTOL)
                k = oracle.keep_count(len(want_scores), keep)
                assert got["k"] == k
                kept = oracle.select_topk(want_scores, k)
                ref = dict(k=k, kept=kept, chunk_scores=want_scores)
                assert_selection_matches(got, ref, prompt)
                # the invariants of the selection, at any size
                assert len(got["ids"]) == sum(min(cfg.chunk, n - int(j) * cfg.chunk) for j in got["kept"])
                spans = got["tok_spans"]
                assert (spans[:, 0] < spans[:, 1]).all() and (spans[1:, 0] > spans[:-1, 1]).all()
        finally:
            spf.spf_set_score_path(previous)


def test_quarter_million_tokens_chunk_32():
    """N = 262144: 8192 chunks in the top-k, 14 key tiles per CTA in the fused kernel."""
    cfg = small_config("v2len", n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(262144,),
                       chunk=32, keep=(0.03, 0.06, 0.10), rank=8, n_needles=32, n_strong=8, needle_len=(16, 128), seed=11)
    _check(cfg, cfg.keep)


def test_code_setting_chunk_128():
    """Chunk 128 at the length of the paper's code-debugging prompts (about 110k tokens, not a multiple of the chunk)."""
    cfg = small_config("code", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=128, n_lookahead=8, lengths=(110003,),
                       chunk=128, keep=(0.15, 0.20, 0.30), rank=8, n_needles=24, n_strong=6, needle_len=(32, 256), seed=12)
    _check(cfg, cfg.keep)


def test_keep_rates_from_three_to_fifty_percent():
    cfg = small_config("rates", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(40000,),
                       chunk=32, keep=(0.03, 0.06, 0.10, 0.25, 0.45, 0.50), rank=8, n_needles=16, n_strong=4,
                       needle_len=(16, 128), recency=True, seed=13)
    _check(cfg, cfg.keep)


def test_two_accumulator_stages_when_the_running_maxima_need_the_room():
    """64 query rows per kv-head and 9 key tiles per CTA: the running maxima take 144 tensor-memory columns, which
    leaves room for two accumulator stages only (the fused kernel picks that layout by itself)."""
    cfg = small_config("deep", n_layers=1, n_q_heads=4, n_kv_heads=1, head_dim=64, n_lookahead=16, lengths=(160001,),
                       chunk=32, keep=(0.10,), rank=8, n_needles=16, n_strong=4, needle_len=(16, 128), seed=14)
    _check(cfg, cfg.keep, paths=(2,))


def test_prompt_beyond_the_fused_kernels_capacity_takes_the_general_path():
    """17 key tiles per CTA at 64 query rows do not fit next to two accumulator stages: pinned to the fused kernel the
    call is refused, left on automatic it is scored by the general path."""
    import paper_2603_02631_b200 as spf
    cfg = small_config("huge", n_layers=1, n_q_heads=4, n_kv_heads=1, head_dim=64, n_lookahead=16, lengths=(310000,),
                       chunk=32, keep=(0.06,), rank=8, n_needles=16, n_strong=4, needle_len=(16, 128), seed=15)
    prompt = make_prompt(cfg, 0, "cuda")
    imp = torch.empty(prompt.n_tokens, dtype=torch.float32, device="cuda")
    bufs = spf.PromptBuffers(prompt.q, prompt.k, imp, None)
    ws = torch.empty(spf.spf_score_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
    previous = spf.spf_set_score_path(2)
    try:
        with pytest.raises(spf.SpfError) as err:
            spf.spf_score([bufs], ws)
        assert err.value.status == -2
    finally:
        spf.spf_set_score_path(previous)
    _check(cfg, cfg.keep, paths=(0,))
