"""spf_compress_host: the whole path for host buffers through one C call, against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits, make_prompt, small_config

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("pinned", [True, False])
def test_compress_host_matches_the_oracle(pinned):
    import paper_2603_02631_b200 as spf
    cfg = small_config("hostpath", n_layers=3, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(5003,),
                       chunk=32, keep=(0.2,), rank=4, n_needles=3, n_strong=2, seed=77)
    prompt = make_prompt(cfg)                             # host tensors
    keep = 0.2
    ref = oracle.compress(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k], prompt.token_ids.numpy(),
                          prompt.char_start.numpy(), prompt.char_end.numpy(), chunk=cfg.chunk, keep=keep,
                          pool_kernel=cfg.pool_kernel)
    pin = (lambda t: t.contiguous().pin_memory()) if pinned else (lambda t: t.contiguous())
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, prompt.n_tokens,
                       chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)
    for _ in range(2):                                    # the second call reuses the arena and the result buffers
        got = sel.run_host(pin(prompt.q), [pin(x) for x in prompt.k], pin(prompt.token_ids), pin(prompt.char_start),
                           pin(prompt.char_end), keep)
        assert got["ids"].tolist() == ref["ids"].tolist()
        assert got["pos"].tolist() == ref["pos"].tolist()
        assert got["tok_spans"].tolist() == ref["tok_spans"].tolist()
        assert got["char_spans"].tolist() == ref["char_spans"].tolist()


def test_compress_host_reports_a_small_arena():
    import paper_2603_02631_b200 as spf
    prompt = make_prompt(CONFIGS["tiny"])
    cfg = prompt.cfg
    k = spf.spf_keep_count(prompt.n_tokens // cfg.chunk, 0.25)
    arena = torch.empty(1024, dtype=torch.uint8, device="cuda")
    out = [torch.empty(k * cfg.chunk, dtype=torch.int32), torch.empty(k * cfg.chunk, dtype=torch.int32),
           torch.empty((k, 2), dtype=torch.int32), torch.empty((k, 2), dtype=torch.int32), torch.empty(2, dtype=torch.int64)]
    with pytest.raises(spf.SpfError) as err:
        spf.spf_compress_host(prompt.q, prompt.k, prompt.token_ids, prompt.char_start, prompt.char_end, cfg.chunk,
                              cfg.pool_kernel, 0.25, arena, *out)
    assert err.value.status == -3
