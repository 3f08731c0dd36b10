"""Key-sharded scoring on the GPU: the two entry points (log-sum-exp of a key range, importance given the whole prompt's
log-sum-exps) on the ranges of two and three would-be ranks, run one after the other on this GPU and combined on the
host exactly as the ranks would combine them; and the library-backed orchestration in a one-rank process group."""
import os

import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, small_config

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["general", "fused"])
def kernel_path(request):
    """The shard calls on the general two-sweep kernels, and on the fused kernel run one visit at a time."""
    import paper_2603_02631_b200 as mod
    previous = mod.spf_set_score_path({"general": 1, "fused": 2}[request.param])
    yield request.param
    mod.spf_set_score_path(previous)


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("L,Hq,Hkv,d,m,N", [(2, 8, 2, 64, 8, 5000), (2, 4, 2, 128, 16, 3333), (1, 4, 4, 64, 5, 777),
                                            (3, 8, 2, 64, 16, 60001)])
def test_shard_entry_points(kernel_path, world, L, Hq, Hkv, d, m, N):
    import paper_2603_02631_b200 as spf
    from paper_2603_02631_b200.sharded import LibraryOps, Shard, shard_bounds
    cfg = small_config("shard", n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, n_lookahead=m, lengths=(N,),
                       rank=4, n_needles=2, n_strong=1, needle_len=(4, 40), seed=N + world)
    prompt = make_prompt(cfg, 0, "cuda")
    want_imp, want_lse = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k])
    ops = LibraryOps()
    shards = [Shard(lo, hi, prompt.q, [k[:, lo:hi].contiguous() for k in prompt.k], prompt.token_ids[lo:hi],
                    prompt.char_start[lo:hi], prompt.char_end[lo:hi]) for lo, hi in shard_bounds(N, world, 32)]
    lses = torch.stack([ops.shard_lse(s) for s in shards])
    # each shard's value is the log-sum-exp over its own keys
    for s, l in zip(shards, lses):
        _, own = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(k) for k in s.k_layers])
        np.testing.assert_allclose(l.cpu().numpy(), own, rtol=0, atol=2e-4)
    lse_all = torch.logsumexp(lses.double(), dim=0).float()
    np.testing.assert_allclose(lse_all.cpu().numpy(), want_lse, rtol=0, atol=2e-4)
    imp = torch.cat([ops.shard_importance(s, lse_all) for s in shards])
    torch.cuda.synchronize()
    rel = np.abs(imp.cpu().numpy() - want_imp) / np.maximum(want_imp, 1e-30)
    assert rel.max() <= 1e-3, rel.max()


def test_orchestration_on_the_library_in_a_one_rank_group():
    import torch.distributed as dist
    import paper_2603_02631_b200 as spf
    from paper_2603_02631_b200.sharded import LibraryOps, Shard, sharded_select
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29561")
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    try:
        cfg = small_config("one", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(6001,),
                           rank=4, n_needles=4, n_strong=2, needle_len=(8, 64), seed=41)
        prompt = make_prompt(cfg, 0, "cuda")
        n = prompt.n_tokens
        k = spf.spf_keep_count((n + 31) // 32, 0.1)
        got = sharded_select(Shard(0, n, prompt.q, prompt.k, prompt.token_ids, prompt.char_start, prompt.char_end), n, k,
                             LibraryOps(), chunk=32, pool_kernel=13)
        ref = oracle.compress(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k], prompt.token_ids.cpu().numpy(),
                              prompt.char_start.cpu().numpy(), prompt.char_end.cpu().numpy(), chunk=32, keep=0.1, pool_kernel=13)
        assert got.kept.tolist() == ref["kept"].tolist()
        assert got.ids.tolist() == ref["ids"].tolist() and got.pos.tolist() == ref["pos"].tolist()
        assert got.tok_spans.tolist() == ref["tok_spans"].tolist() and got.char_spans.tolist() == ref["char_spans"].tolist()
    finally:
        if created:
            dist.destroy_process_group()
