"""Batched selection calls: one launch for several prompts must give exactly what the single-prompt calls give, and the
whole batched path must match the oracle per prompt."""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, small_config

from parity_util import assert_importance_close, assert_selection_matches, oracle_run

pytestmark = pytest.mark.gpu


def test_batched_selection_equals_single_calls_bit_for_bit():
    import paper_2603_02631_b200 as spf
    g = torch.Generator().manual_seed(17)
    lengths = [31, 1000, 4097, 10007, 1, 2500] + [333 + 17 * i for i in range(34)]       # 40 prompts: two launches
    chunk, w, keep = 32, 13, 0.25
    imps = [torch.rand(n, generator=g).cuda() for n in lengths]
    for t in imps[:3]:
        t[::5] = 0.5                                      # heavy ties
    ncs = [(n + chunk - 1) // chunk for n in lengths]
    ks = [spf.spf_keep_count(c, keep) for c in ncs]
    ids = [torch.randint(0, 32000, (n,), generator=g, dtype=torch.int32).cuda() for n in lengths]
    starts = [torch.arange(n, dtype=torch.int32, device="cuda") * 3 for n in lengths]
    ends = [s + 2 for s in starts]

    def outputs():
        return dict(scores=[torch.zeros(c, device="cuda") for c in ncs],
                    kept=[torch.full((k,), -1, dtype=torch.int32, device="cuda") for k in ks],
                    out_ids=[torch.full((min(k * chunk, n),), -1, dtype=torch.int32, device="cuda") for k, n in zip(ks, lengths)],
                    out_pos=[torch.full((min(k * chunk, n),), -1, dtype=torch.int32, device="cuda") for k, n in zip(ks, lengths)],
                    tok=[torch.full((k, 2), -1, dtype=torch.int32, device="cuda") for k in ks],
                    ch=[torch.full((k, 2), -1, dtype=torch.int32, device="cuda") for k in ks],
                    counts=[torch.zeros(2, dtype=torch.int64, device="cuda") for _ in ks])
    one, many = outputs(), outputs()
    for i, n in enumerate(lengths):
        spf.spf_chunk_pool(imps[i], w, chunk, one["scores"][i])
        spf.spf_select_topk(one["scores"][i], ncs[i], ks[i], one["kept"][i])
        spf.spf_compact_spans(one["kept"][i], ks[i], chunk, n, ids[i], starts[i], ends[i], one["out_ids"][i], one["out_pos"][i],
                              one["tok"][i], one["ch"][i], one["counts"][i])
    spf.spf_chunk_pool_batch(imps, w, chunk, many["scores"])
    spf.spf_select_topk_batch(many["scores"], ncs, ks, many["kept"])
    spf.spf_compact_spans_batch(many["kept"], ks, chunk, lengths, ids, starts, ends, many["out_ids"], many["out_pos"], many["tok"],
                                many["ch"], many["counts"])
    torch.cuda.synchronize()
    for name in one:
        for i in range(len(lengths)):
            assert torch.equal(one[name][i], many[name][i]), f"{name}[{i}] differs between the single and the batched call"
    # and the single calls are the oracle's
    i = 3
    want = oracle.chunk_means(oracle.avg_pool(imps[i].cpu().numpy().astype(np.float64), w), chunk)
    np.testing.assert_allclose(many["scores"][i].cpu().numpy(), want, rtol=1e-5)


def test_batch_selector_matches_the_oracle_per_prompt():
    import paper_2603_02631_b200 as spf
    cfg = small_config("batch", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8,
                       lengths=(3001, 777, 5000, 129), chunk=32, keep=(0.2,), rank=4, n_needles=2, n_strong=1, seed=21)
    prompts = [make_prompt(cfg, i) for i in range(len(cfg.lengths))]
    dev = [p.to("cuda") for p in prompts]
    sel = spf.BatchSelector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, cfg.lengths,
                            chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)
    results = sel.run(dev, 0.2)
    torch.cuda.synchronize()
    assert int(sel.dev_status.item()) == 0
    for p, res in zip(prompts, results):
        ref = oracle_run(p, 0.2)
        got = res.host()
        assert_importance_close(got["importance"], ref["importance"])
        assert_selection_matches(got, ref, p)


def test_batched_calls_validate_every_item_before_launching():
    import paper_2603_02631_b200 as spf
    good = torch.rand(100).cuda()
    out = torch.zeros(4).cuda()
    with pytest.raises(spf.SpfError) as err:
        spf.spf_select_topk_batch([out, out], [4, 4], [2, 9], [torch.zeros(2, dtype=torch.int32).cuda(), torch.zeros(9, dtype=torch.int32).cuda()])
    assert err.value.status == -1 and "item 1" in str(err.value)
    with pytest.raises(spf.SpfError):
        spf.spf_chunk_pool_batch([good], 12, 32, [out])   # even pooling kernel


@pytest.mark.parametrize("n,chunk,keep", [(10007, 32, 0.3), (131072, 32, 0.1), (262144, 32, 0.5), (5000, 128, 0.03), (31, 32, 1.0),
                                          (300000, 32, 0.25)])
def test_select_compact_equals_the_two_calls(n, chunk, keep):
    """Top-k and compaction chained in one launch: bit-identical to spf_select_topk + spf_compact_spans (with ties, with the
    score array cached in registers and, for the longest prompt, re-read per pass), and to the oracle's selection."""
    import paper_2603_02631_b200 as spf
    g = torch.Generator().manual_seed(n)
    imp = torch.rand(n, generator=g)
    imp[::7] = 0.25
    imp = imp.cuda()
    n_chunks = (n + chunk - 1) // chunk
    k = spf.spf_keep_count(n_chunks, keep)
    scores = torch.zeros(n_chunks, device="cuda")
    spf.spf_chunk_pool(imp, 13, chunk, scores)
    scores[::3] = scores[min(1, n_chunks - 1)].item()      # heavy ties across chunk scores
    ids = torch.randint(0, 32000, (n,), generator=g, dtype=torch.int32).cuda()
    starts = torch.arange(n, dtype=torch.int32, device="cuda") * 2
    ends = starts + 1

    def outs():
        rows = min(k * chunk, n)
        return [torch.full((k,), -1, dtype=torch.int32, device="cuda"), torch.full((rows,), -1, dtype=torch.int32, device="cuda"),
                torch.full((rows,), -1, dtype=torch.int32, device="cuda"), torch.full((k, 2), -1, dtype=torch.int32, device="cuda"),
                torch.full((k, 2), -1, dtype=torch.int32, device="cuda"), torch.zeros(2, dtype=torch.int64, device="cuda")]
    a, b = outs(), outs()
    spf.spf_select_topk(scores, n_chunks, k, a[0])
    spf.spf_compact_spans(a[0], k, chunk, n, ids, starts, ends, a[1], a[2], a[3], a[4], a[5])
    spf.spf_select_compact(scores, n_chunks, k, chunk, n, ids, starts, ends, b[0], b[1], b[2], b[3], b[4], b[5])
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    want = oracle.select_topk(scores.cpu().numpy().astype(np.float64), k)
    assert b[0].cpu().tolist() == want.tolist()
