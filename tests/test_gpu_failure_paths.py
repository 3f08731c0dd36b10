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
