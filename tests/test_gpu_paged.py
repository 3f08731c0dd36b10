"""Paged key cache (the paper's serving system keeps KV caches in 4k-token blocks, Section 3.1): spf_score_paged on a
shuffled block pool against the oracle on the logical keys, and bit for bit against spf_score on the gathered copy."""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, small_config

pytestmark = pytest.mark.gpu


def _paged_copy(k_layers, n, block_tokens, n_spare, seed):
    """Scatters [Hkv, N, d] keys over a pool of shuffled blocks; spare and tail rows hold NaN patterns."""
    Hkv, _, d = k_layers[0].shape
    n_blocks = (n + block_tokens - 1) // block_tokens
    g = torch.Generator().manual_seed(seed)
    perm = torch.randperm(n_blocks + n_spare, generator=g)[:n_blocks].to(torch.int32)
    pools = []
    for k in k_layers:
        pool = torch.full((n_blocks + n_spare, Hkv, block_tokens, d), float("nan"), dtype=torch.bfloat16, device=k.device)
        for b in range(n_blocks):
            lo, hi = b * block_tokens, min((b + 1) * block_tokens, n)
            pool[int(perm[b]), :, :hi - lo] = k[:, lo:hi]
        pools.append(pool)
    return pools, perm.to(k_layers[0].device)


@pytest.mark.parametrize("L,Hq,Hkv,d,m,N,bt", [
    (2, 8, 2, 64, 8, 20000, 4096),      # the paper's block size; the last block is partly filled
    (2, 4, 2, 128, 8, 9001, 1024),
    (1, 4, 1, 64, 16, 50000, 128),      # one tile per block
    (1, 2, 1, 64, 8, 100, 256),         # a single, partly filled block
])
@pytest.mark.parametrize("path", [2, 1])
def test_paged_scoring(L, Hq, Hkv, d, m, N, bt, path):
    import paper_2603_02631_b200 as spf
    outer = spf.spf_set_score_path(path)
    try:
        _paged_case(spf, L, Hq, Hkv, d, m, N, bt, path)
    finally:
        spf.spf_set_score_path(outer)


def _paged_case(spf, L, Hq, Hkv, d, m, N, bt, path):
    cfg = small_config("paged", n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, n_lookahead=m, lengths=(N,),
                       rank=4, n_needles=2 if N >= 300 else 0, n_strong=1, needle_len=(4, 40), seed=N + bt)
    prompt = make_prompt(cfg, 0, "cuda")
    pools, table = _paged_copy(prompt.k, N, bt, n_spare=3, seed=N)
    want_imp, want_lse = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k])
    imp = torch.empty(N, dtype=torch.float32, device="cuda")
    lse = torch.empty(L * Hq * m, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    bufs = spf.PagedPromptBuffers(prompt.q, pools, table, N, imp, lse)
    ws = torch.empty(spf.spf_score_paged_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
    spf.spf_score_paged([bufs], ws, 0.0, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    got = imp.cpu().numpy()
    assert np.isfinite(got).all()
    rel = np.abs(got - want_imp) / np.maximum(want_imp, 1e-30)
    assert rel.max() <= 1e-3, rel.max()
    np.testing.assert_allclose(lse.cpu().numpy().reshape(L, Hq, m), want_lse, rtol=0, atol=2e-4)
    # the same kernels on the contiguous keys: identical bits
    previous = spf.spf_set_score_path(path)
    try:
        imp2 = torch.empty_like(imp)
        flat = spf.PromptBuffers(prompt.q, prompt.k, imp2, None)
        ws2 = torch.empty(spf.spf_score_workspace_bytes([flat]), dtype=torch.uint8, device="cuda")
        spf.spf_score([flat], ws2, 0.0, st)
        torch.cuda.synchronize()
        assert torch.equal(imp, imp2)
    finally:
        spf.spf_set_score_path(previous)


def test_paged_argument_checks():
    import paper_2603_02631_b200 as spf
    cfg = small_config("paged", n_layers=1, n_q_heads=2, n_kv_heads=1, head_dim=64, n_lookahead=8, lengths=(300,), seed=1)
    prompt = make_prompt(cfg, 0, "cuda")
    imp = torch.empty(300, dtype=torch.float32, device="cuda")
    for bt in (100, 64):                   # not multiples of 128
        pools = [torch.zeros((4, 1, bt, 64), dtype=torch.bfloat16, device="cuda")]
        table = torch.zeros(8, dtype=torch.int32, device="cuda")
        with pytest.raises(spf.SpfError):
            spf.spf_score_paged_workspace_bytes([spf.PagedPromptBuffers(prompt.q, pools, table, 300, imp)])


def test_paged_selection_end_to_end():
    """The chained path on a paged cache gives the selection the contiguous cache gives."""
    import paper_2603_02631_b200 as spf
    cfg = small_config("paged", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(12345,),
                       rank=4, n_needles=4, n_strong=2, needle_len=(8, 64), seed=31)
    prompt = make_prompt(cfg, 0, "cuda")
    n = prompt.n_tokens
    pools, table = _paged_copy(prompt.k, n, 4096, n_spare=2, seed=5)
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n)
    a = sel.run(prompt.q, prompt.k, prompt.token_ids, prompt.char_start, prompt.char_end, 0.1).host()
    b = sel.run_paged(prompt.q, pools, table, n, prompt.token_ids, prompt.char_start, prompt.char_end, 0.1).host()
    assert int(sel.dev_status.item()) == 0
    for key in ("importance", "kept", "ids", "pos", "tok_spans", "char_spans"):
        assert np.array_equal(a[key], b[key]), key
    ref = oracle.compress(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k], prompt.token_ids.cpu().numpy(),
                          prompt.char_start.cpu().numpy(), prompt.char_end.cpu().numpy(), chunk=32, keep=0.1, pool_kernel=13)
    assert np.array_equal(b["kept"], ref["kept"]) and np.array_equal(b["ids"], ref["ids"])
