"""Switches for two points the paper leaves open: the pooling edge rule and chunks that are always kept.
CPU part: the oracle's versions against library routines, hand examples and brute force.  GPU part: the
library's entry points against the oracle."""
import itertools

import numpy as np
import pytest
import torch

import oracle


# ------------------------------------------------------------------------------------------- oracle pins (CPU)
def test_oracle_pool_in_range_divisor_matches_torch_and_keeps_constants():
    rng = np.random.default_rng(0)
    x = rng.random(200)
    want = torch.nn.functional.avg_pool1d(torch.from_numpy(x)[None, None], 13, 1, 6, count_include_pad=False)[0, 0].numpy()
    np.testing.assert_allclose(oracle.avg_pool(x, 13, count_include_pad=False), want, rtol=1e-13)
    # a constant signal stays constant up to the ends under this rule, and is damped to 7/13 at the ends under the default
    c = np.full(50, 3.0)
    np.testing.assert_allclose(oracle.avg_pool(c, 13, count_include_pad=False), c, rtol=1e-14)
    assert abs(oracle.avg_pool(c, 13)[0] - 3.0 * 7 / 13) < 1e-14


def test_oracle_forced_topk_hand_example_and_brute_force():
    s = np.array([0.1, 0.9, 0.5, 0.5, 0.2, 0.8])
    assert oracle.select_topk_forced(s, 3, True, True).tolist() == [0, 1, 5]      # 0 and 5 forced, best of the rest: 1
    assert oracle.select_topk_forced(s, 3, True, False).tolist() == [0, 1, 5]     # 0 forced, then 0.9 and 0.8
    assert oracle.select_topk_forced(s, 4, False, True).tolist() == [1, 2, 3, 5]  # 5 forced, then 0.9, 0.5 (index 2), 0.5 (index 3)
    assert oracle.select_topk_forced(s, 2, True, True).tolist() == [0, 5]
    assert oracle.select_topk_forced(np.array([0.3]), 1, True, True).tolist() == [0]
    with pytest.raises(ValueError):
        oracle.select_topk_forced(s, 1, True, True)
    # brute force on tiny inputs with ties: the kept set maximises (sum of scores of the unforced kept, then lowest indices)
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(1, 8)); k = int(rng.integers(1, n + 1))
        sc = rng.integers(0, 3, n).astype(np.float64)
        ff, fl = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        forced = ({0} if ff else set()) | ({n - 1} if fl else set())
        if k < len(forced):
            continue
        best = None
        for comb in itertools.combinations(range(n), k):
            if not forced <= set(comb):
                continue
            rest = [j for j in comb if j not in forced]
            cand = (-sum(sc[j] for j in rest), sorted(rest))
            if best is None or cand < best[0]:
                best = (cand, comb)
        assert oracle.select_topk_forced(sc, k, ff, fl).tolist() == list(best[1])
    # no flags: the plain selection
    for _ in range(50):
        sc = rng.random(40)
        assert oracle.select_topk_forced(sc, 7).tolist() == oracle.select_topk(sc, 7).tolist()


# ------------------------------------------------------------------------------------------- library (GPU)
@pytest.mark.gpu
@pytest.mark.parametrize("n,chunk,w", [(1000, 32, 13), (4097, 64, 13), (50, 8, 5), (7, 32, 13), (131072, 32, 13)])
def test_chunk_pool_edge_rule(n, chunk, w):
    import paper_2603_02631_b200 as spf
    rng = np.random.default_rng(n)
    imp = rng.random(n).astype(np.float32)
    d_imp = torch.from_numpy(imp).cuda()
    n_chunks = (n + chunk - 1) // chunk
    out = torch.empty(n_chunks, dtype=torch.float32, device="cuda")
    for rule, include_pad in ((0, True), (1, False)):
        spf.spf_chunk_pool_edge(d_imp, w, chunk, rule, out)
        want = oracle.chunk_means(oracle.avg_pool(imp.astype(np.float64), w, count_include_pad=include_pad), chunk)
        np.testing.assert_allclose(out.cpu().numpy(), want, rtol=1e-5)
    # rule 0 is the plain entry point, bit for bit
    ref = torch.empty_like(out)
    spf.spf_chunk_pool(d_imp, w, chunk, ref)
    spf.spf_chunk_pool_edge(d_imp, w, chunk, 0, out)
    assert torch.equal(out, ref)
    with pytest.raises(spf.SpfError):
        spf.spf_chunk_pool_edge(d_imp, w, chunk, 2, out)


@pytest.mark.gpu
def test_select_topk_forced_is_exact():
    import paper_2603_02631_b200 as spf
    rng = np.random.default_rng(9)
    for n, k in [(1, 1), (2, 2), (64, 16), (1024, 103), (4096, 410), (8192, 246), (5000, 2)]:
        # coarse scores so that ties abound, the forced ends among the lowest
        sc = (rng.integers(0, 50, n) / 50).astype(np.float32)
        sc[0] = 0.0; sc[-1] = 0.0
        d_sc = torch.from_numpy(sc).cuda()
        kept = torch.empty(k, dtype=torch.int32, device="cuda")
        for ff, fl in itertools.product((False, True), repeat=2):
            n_forced = len(({0} if ff else set()) | ({n - 1} if fl else set()))
            if k < n_forced:
                with pytest.raises(spf.SpfError):
                    spf.spf_select_topk_forced(d_sc, n, k, ff, fl, kept)
                continue
            spf.spf_select_topk_forced(d_sc, n, k, ff, fl, kept)
            want = oracle.select_topk_forced(sc.astype(np.float64), k, ff, fl)
            assert kept.cpu().numpy().tolist() == want.tolist(), (n, k, ff, fl)


# ------------------------------------------------------------------------------------------- extra denominator term
def _tiny_inputs(seed=0, L=2, Hq=4, Hkv=2, d=64, m=3, N=40):
    from workloads import bf16_bits
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(L, Hq, m, d, generator=g).to(torch.bfloat16)
    k = [torch.randn(Hkv, N, d, generator=g).to(torch.bfloat16) for _ in range(L)]
    return q, k, bf16_bits(q), [bf16_bits(x) for x in k]


def test_oracle_extra_denominator_equals_appended_keys_and_closed_forms():
    """A per-row extra term is what extra keys seen by that row alone would contribute: for one (layer, head, query)
    row, append explicit extra logits to the row and take a library softmax over the lot."""
    from scipy.special import logsumexp, softmax
    q, k, qb, kb = _tiny_inputs()
    L, Hq, m, d = q.shape
    rng = np.random.default_rng(0)
    n_extra = 5
    extra_logits = rng.normal(size=(L, Hq, m, n_extra)) * 2.0
    extra = logsumexp(extra_logits, axis=-1)
    imp, lse = oracle.token_importance(qb, kb, extra_lse=extra)
    # brute force: the definition, row by row, with the extra logits appended as further softmax inputs
    G = Hq // k[0].shape[0]
    N = k[0].shape[1]
    A = np.zeros((m, N))
    for l in range(L):
        for h in range(Hq):
            for i in range(m):
                z = (k[l][h // G].double() @ q[l, h, i].double()).numpy() / np.sqrt(d)
                p = softmax(np.concatenate([z, extra_logits[l, h, i]]))[:N]
                A[i] = np.maximum(A[i], p)
                assert abs(lse[l, h, i] - logsumexp(np.concatenate([z, extra_logits[l, h, i]]))) < 1e-12
    np.testing.assert_allclose(imp, A.mean(axis=0), rtol=1e-12)
    # closed forms: an extra term equal to the prompt's own log-sum-exp halves every probability; -inf changes nothing
    imp0, lse0 = oracle.token_importance(qb, kb)
    imp_half, lse_half = oracle.token_importance(qb, kb, extra_lse=lse0)
    np.testing.assert_allclose(imp_half, imp0 / 2, rtol=1e-13)
    np.testing.assert_allclose(lse_half, lse0 + np.log(2.0), rtol=0, atol=1e-12)
    imp_same, _ = oracle.token_importance(qb, kb, extra_lse=np.full_like(lse0, -np.inf))
    np.testing.assert_allclose(imp_same, imp0, rtol=0, atol=0)


@pytest.mark.gpu
@pytest.mark.parametrize("path", [1, 2])
def test_score_extra_matches_oracle(path):
    import paper_2603_02631_b200 as spf
    from workloads import bf16_bits, make_prompt, small_config
    previous = spf.spf_set_score_path(path)
    try:
        for (L, Hq, Hkv, d, m, N) in [(2, 8, 2, 64, 8, 3001), (3, 4, 2, 128, 8, 2049), (1, 4, 1, 64, 16, 40000)]:
            cfg = small_config("extra", n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, n_lookahead=m, lengths=(N,),
                               rank=4, n_needles=2, n_strong=1, needle_len=(4, 40), seed=N)
            prompt = make_prompt(cfg, 0, "cuda")
            qb, kb = bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k]
            _, lse0 = oracle.token_importance(qb, kb)
            rng = np.random.default_rng(N)
            # around the prompt's own denominators: from negligible to dominant
            extra = lse0 + rng.uniform(-6.0, 3.0, size=lse0.shape)
            want_imp, want_lse = oracle.token_importance(qb, kb, extra_lse=extra)
            imp = torch.empty(N, dtype=torch.float32, device="cuda")
            lse = torch.empty(L * Hq * m, dtype=torch.float32, device="cuda")
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            bufs = spf.PromptBuffers(prompt.q, prompt.k, imp, lse)
            ws = torch.empty(spf.spf_score_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
            d_extra = torch.from_numpy(extra.astype(np.float32)).cuda().contiguous()
            spf.spf_score_extra([bufs], [d_extra], ws, 0.0, st)
            torch.cuda.synchronize()
            assert int(st.item()) == 0
            # the oracle sees the extra term in fp64, the device in fp32: compare against the fp32-rounded input
            want_imp, want_lse = oracle.token_importance(qb, kb, extra_lse=d_extra.cpu().numpy().astype(np.float64).reshape(L, Hq, m))
            rel = np.abs(imp.cpu().numpy() - want_imp) / np.maximum(want_imp, 1e-30)
            assert rel.max() <= 1e-3, rel.max()
            np.testing.assert_allclose(lse.cpu().numpy().reshape(L, Hq, m), want_lse, rtol=0, atol=2e-4)
            # without the term (NULL entry) the call is spf_score, bit for bit
            imp2 = torch.empty_like(imp)
            spf.spf_score_extra([spf.PromptBuffers(prompt.q, prompt.k, imp2, None)], [None], ws, 0.0, st)
            imp3 = torch.empty_like(imp)
            spf.spf_score([spf.PromptBuffers(prompt.q, prompt.k, imp3, None)], ws, 0.0, st)
            torch.cuda.synchronize()
            assert torch.equal(imp2, imp3)
    finally:
        spf.spf_set_score_path(previous)


@pytest.mark.gpu
def test_selector_with_all_switches_on():
    """The chained path with the in-range pooling divisor and both ends forced, against the oracle's steps."""
    import paper_2603_02631_b200 as spf
    from workloads import bf16_bits, make_prompt, small_config
    cfg = small_config("switches", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(6000,),
                       chunk=32, rank=4, n_needles=4, n_strong=2, needle_len=(8, 64), seed=21)
    prompt = make_prompt(cfg, 0, "cuda")
    n = prompt.n_tokens
    imp, _ = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k])
    scores = oracle.chunk_means(oracle.avg_pool(imp, 13, count_include_pad=False), 32)
    k = oracle.keep_count(len(scores), 0.1)
    kept = oracle.select_topk_forced(scores, k, True, True)
    ids, pos, tok, ch = oracle.compact(kept, 32, n, *(t.cpu().numpy().astype(np.int64) for t in
                                                     (prompt.token_ids, prompt.char_start, prompt.char_end)))
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n, chunk=32,
                       pool_edge_rule=1, force_first=True, force_last=True)
    got = sel.run(prompt.q, prompt.k, prompt.token_ids, prompt.char_start, prompt.char_end, 0.1).host()
    np.testing.assert_allclose(got["chunk_scores"], scores, rtol=1e-3)
    assert 0 in got["kept"] and len(scores) - 1 in got["kept"]
    # the kept set may differ from the oracle's only inside the tie band of the k-th score among the unforced chunks
    differ = np.setxor1d(got["kept"], kept)
    if len(differ):
        rest = np.sort(np.delete(scores, [0, len(scores) - 1]))[::-1]
        tau = rest[k - 3]
        assert (np.abs(scores[differ] - tau) <= 1e-3 * abs(tau)).all()
    else:
        assert np.array_equal(got["ids"], ids) and np.array_equal(got["char_spans"], ch)
