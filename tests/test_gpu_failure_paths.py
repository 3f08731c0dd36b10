"""Device-side conditions are reported through dev_status; nothing traps, hangs or poisons the context."""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits

from parity_util import assert_importance_close

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_and_context_survives():
    import paper_2603_02631_b200 as spf
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    spf.spf_selftest_bounded_wait(status)
    torch.cuda.synchronize()
    assert int(status.item()) == -5                       # SPF_ERR_TIMEOUT
    # the context is still usable
    x = torch.arange(1000, device="cuda", dtype=torch.float32)
    assert float(x.sum().item()) == 499500.0


def _overflow_case():
    """One key whose logits exceed those of the sample key (index N // 2) by far more than 2^187."""
    L, Hq, Hkv, d, m, N = 1, 2, 1, 64, 8, 300
    g = torch.Generator().manual_seed(11)
    q = torch.randn(L, Hq, m, d, generator=g)
    q[..., 0] = 64.0
    k = torch.randn(Hkv, N, d, generator=g) * 0.1
    k[0, N // 2] = 0.0                                     # the sample key: logit 0
    k[0, 7, 0] = 256.0                                     # q.k = 16384 -> about 2950 in base-2 units
    return q.to(torch.bfloat16), [k.to(torch.bfloat16)]


def test_fused_path_reports_range_overflow_and_general_path_is_exact():
    import paper_2603_02631_b200 as spf
    q, k = _overflow_case()
    n = k[0].shape[1]
    want, _ = oracle.token_importance(bf16_bits(q), [bf16_bits(x) for x in k])
    results = {}
    for path in (2, 1):
        previous = spf.spf_set_score_path(path)
        try:
            imp = torch.zeros(n, dtype=torch.float32, device="cuda")
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            bufs = spf.PromptBuffers(q.cuda(), [x.cuda() for x in k], imp, None)
            ws = torch.empty(spf.spf_score_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
            spf.spf_score([bufs], ws, 0.0, status)
            torch.cuda.synchronize()
            results[path] = (int(status.item()), imp.cpu().numpy())
        finally:
            spf.spf_set_score_path(previous)
    assert results[2][0] == -6                            # SPF_ERR_RANGE from the fused path
    assert results[1][0] == 0
    assert_importance_close(results[1][1], want)          # the general path handles any finite logits
    assert abs(results[1][1][7] - 1.0) < 1e-3            # logits near 3000 (base 2): fp32 spacing there is 2.4e-4


def test_selector_checked_run_falls_back_to_the_general_path():
    import paper_2603_02631_b200 as spf
    q, k = _overflow_case()
    n = k[0].shape[1]
    sel = spf.Selector(1, 2, 1, 64, 8, max_tokens=n, chunk=32)
    ids = torch.arange(n, dtype=torch.int32, device="cuda")
    starts = ids * 3
    res = sel.run_checked(q.cuda(), [x.cuda() for x in k], ids, starts, starts + 3, keep=0.2)
    want, _ = oracle.token_importance(bf16_bits(q), [bf16_bits(x) for x in k])
    assert_importance_close(res.importance.cpu().numpy(), want)
    assert 0 in res.kept_chunks[:res.k].cpu().tolist()     # the dominant key 7 lives in chunk 0


def _offset_case(offsets_nats, seed=5, n=3000):
    """One kv-head with a group of four query heads whose logits carry constant offsets (in nats): every key has
    16 in coordinate 0 and head g has offsets[g] / 2 there, so head g's logits are shifted by offsets[g] (scale
    1/8).  The softmax does not see a constant shift; a per-slab reference does."""
    L, Hq, Hkv, d, m = 2, 4, 1, 64, 8
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(L, Hq, m, d, generator=g)
    k = [torch.randn(Hkv, n, d, generator=g) for _ in range(L)]
    for layer in range(L):
        k[layer][..., 0] = 16.0
        for h, off in enumerate(offsets_nats):
            q[layer, h, :, 0] = off / 2.0
    return q.to(torch.bfloat16), [x.to(torch.bfloat16) for x in k]


def _score(spf, q, k, path):
    n = k[0].shape[1]
    previous = spf.spf_set_score_path(path)
    try:
        imp = torch.zeros(n, dtype=torch.float32, device="cuda")
        lse = torch.zeros(q.shape[0] * q.shape[1] * q.shape[2], dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        bufs = spf.PromptBuffers(q.cuda(), [x.cuda() for x in k], imp, lse)
        ws = torch.empty(spf.spf_score_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
        spf.spf_score([bufs], ws, 0.0, status)
        torch.cuda.synchronize()
        return int(status.item()), imp.cpu().numpy(), lse.cpu().numpy()
    finally:
        spf.spf_set_score_path(previous)


@pytest.mark.parametrize("offsets", [(0.0, -30.0, -45.0, 10.0), (0.0, -70.0, 20.0, -80.0), (60.0, 0.0, 0.0, 0.0)])
def test_fused_path_is_exact_when_heads_of_a_group_differ_in_scale(offsets):
    """Heads that share a kv-head, tens of nats apart: the fused path's single reference per kv-head must not cost
    the low heads any part of their row sums (importance and lse against the oracle, status 0)."""
    import paper_2603_02631_b200 as spf
    q, k = _offset_case(offsets)
    want, want_lse = oracle.token_importance(bf16_bits(q), [bf16_bits(x) for x in k])
    status, imp, lse = _score(spf, q, k, 2)
    assert status == 0
    assert_importance_close(imp, want)
    # logits reach 80 nats here: fp32 spacing there is 8e-6, the accumulated error a few 1e-4
    np.testing.assert_allclose(lse.reshape(want_lse.shape), want_lse, rtol=0, atol=1e-3)


def test_fused_path_range_limit_is_on_the_high_side_only():
    """A head 150 nats (216 base-2 units) above the lowest head of its group overflows the fp32 row sums of the
    fused path: status SPF_ERR_RANGE, nothing else; 80 nats below is fine (previous test).  The checked run
    recovers on the general path and matches the oracle."""
    import paper_2603_02631_b200 as spf
    q, k = _offset_case((0.0, 150.0, 0.0, 0.0))
    want, _ = oracle.token_importance(bf16_bits(q), [bf16_bits(x) for x in k])
    status, _, _ = _score(spf, q, k, 2)
    assert status == -6
    status, imp, _ = _score(spf, q, k, 1)
    assert status == 0
    assert_importance_close(imp, want)
    n = k[0].shape[1]
    sel = spf.Selector(2, 4, 1, 64, 8, max_tokens=n, chunk=32)
    ids = torch.arange(n, dtype=torch.int32, device="cuda")
    previous = spf.spf_set_score_path(2)
    try:
        res = sel.run_checked(q.cuda(), [x.cuda() for x in k], ids, ids * 2, ids * 2 + 2, keep=0.1)
    finally:
        spf.spf_set_score_path(previous)
    assert_importance_close(res.importance.cpu().numpy(), want)
