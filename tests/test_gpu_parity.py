"""GPU parity: the CUDA path through the C ABI against the CPU oracle on the same seeded bytes."""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits, make_prompt, small_config

from parity_util import (assert_importance_close, assert_selection_matches, compare_full, gpu_run, oracle_run)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["general", "fused"])
def spf(request):
    """The package with spf_score pinned to one of its two kernel paths (restored afterwards)."""
    import paper_2603_02631_b200 as mod
    previous = mod.spf_set_score_path({"general": 1, "fused": 2}[request.param])
    yield mod
    mod.spf_set_score_path(previous)


def test_tiny_config_end_to_end(spf):
    prompt = make_prompt(CONFIGS["tiny"])
    ref, gpu, err, n_diff = compare_full(prompt, 0.25)
    assert n_diff == 0
    kept = set(gpu["kept"].tolist())
    for start, _, _ in prompt.needles:
        assert start // 32 in kept


SHAPES = [
    # L, Hq, Hkv, d, m, N, chunk          (several key tiles, ragged tails, every tile-shape template)
    (2, 4, 2, 64, 8, 1000, 32),            # G=2, rows 16
    (1, 8, 2, 64, 8, 4097, 32),            # G=4, rows 32, N = 1 mod 32
    (2, 8, 1, 64, 8, 2500, 64),            # G=8, rows 64
    (2, 8, 2, 64, 16, 3001, 32),           # m=16, rows 64 (long-context geometry)
    (3, 16, 8, 128, 8, 2049, 32),          # d=128, G=2 (wide-head geometry)
    (1, 4, 4, 128, 16, 777, 16),           # G=1, m=16
    (2, 2, 2, 64, 1, 333, 8),              # m=1
    (2, 6, 2, 64, 5, 1234, 32),            # m=5 (padded to 8), G=3 -> rows 24 padded to 32
    (1, 4, 2, 128, 12, 1500, 128),         # m=12 padded to 16, chunk 128
    (1, 2, 1, 64, 20, 900, 32),            # m=20 padded to 24
    (1, 2, 1, 64, 32, 650, 32),            # m=32
    (1, 2, 1, 128, 8, 60001, 32),          # d=128, four one-tile pipeline stages per CTA in the fused path
    (1, 4, 1, 64, 16, 50000, 32),          # d=64, 64 query rows, three tiles (two stages, the second half full) per CTA
    (2, 4, 2, 64, 8, 31, 32),              # a single partial key tile and a single chunk
    (1, 1, 1, 64, 8, 1, 32),               # one token
]


@pytest.mark.parametrize("L,Hq,Hkv,d,m,N,chunk", SHAPES)
def test_random_small_shapes(spf, L, Hq, Hkv, d, m, N, chunk):
    cfg = small_config("rand", n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, n_lookahead=m, lengths=(N,),
                       chunk=chunk, keep=(0.2,), rank=4, n_needles=2 if N >= 300 else 0, n_strong=1,
                       needle_len=(4, 40), seed=N + m)
    prompt = make_prompt(cfg)
    compare_full(prompt, 0.2)


def test_layer_scale_and_recency_inputs(spf):
    cfg = small_config("scaled", n_layers=4, n_q_heads=8, n_kv_heads=4, head_dim=128, n_lookahead=8, lengths=(5000,),
                       chunk=64, keep=(0.05, 0.5), rank=8, n_needles=6, n_strong=2, needle_len=(16, 128),
                       layer_scale=True, recency=True, seed=77)
    prompt = make_prompt(cfg)
    for keep in (0.05, 0.10, 0.25, 0.50):
        compare_full(prompt, keep)


def test_custom_softmax_scale_and_strided_keys(spf):
    cfg = small_config("strided", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(1500,),
                       seed=5)
    prompt = make_prompt(cfg)
    n = prompt.n_tokens
    # keys stored token-major [N, Hkv, d] and viewed as [Hkv, N, d]: token stride Hkv*d, head stride d
    k_dev = [x.cuda().permute(1, 0, 2).contiguous().permute(1, 0, 2) for x in prompt.k]
    assert k_dev[0].stride() == (64, 128, 1)
    imp = torch.empty(n, dtype=torch.float32, device="cuda")
    lse = torch.empty(2 * 4 * 8, dtype=torch.float32, device="cuda")
    bufs = spf.binding.PromptBuffers(prompt.q.cuda(), k_dev, imp, lse)
    ws = torch.empty(spf.spf_score_workspace_bytes([bufs], 0.2), dtype=torch.uint8, device="cuda")
    spf.spf_score([bufs], ws, softmax_scale=0.2)
    torch.cuda.synchronize()
    want, want_lse = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k], scale=0.2)
    assert_importance_close(imp.cpu().numpy(), want)
    np.testing.assert_allclose(lse.cpu().numpy().reshape(want_lse.shape), want_lse, atol=2e-4, rtol=0)


def test_ragged_batch_in_one_call(spf):
    cfg = small_config("batch", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=128, n_lookahead=8,
                       lengths=(700, 1531, 64, 2222), seed=9)
    prompts = [make_prompt(cfg, i) for i in range(4)]
    bufs = []
    for p in prompts:
        dp = p.to("cuda")
        bufs.append(spf.binding.PromptBuffers(dp.q, dp.k, torch.empty(p.n_tokens, dtype=torch.float32, device="cuda"),
                                              torch.empty(2 * 4 * 8, dtype=torch.float32, device="cuda")))
    ws = torch.empty(spf.spf_score_workspace_bytes(bufs), dtype=torch.uint8, device="cuda")
    spf.spf_score(bufs, ws)
    torch.cuda.synchronize()
    for p, b in zip(prompts, bufs):
        want, _ = oracle.token_importance(bf16_bits(p.q), [bf16_bits(x) for x in p.k])
        assert_importance_close(b.importance.cpu().numpy(), want)


def test_identical_keys_give_uniform_importance(spf):
    L, Hq, Hkv, d, m, N = 2, 4, 2, 64, 8, 515
    g = torch.Generator().manual_seed(3)
    q = torch.randn(L, Hq, m, d, generator=g).to(torch.bfloat16).cuda()
    k = [torch.randn(Hkv, 1, d, generator=g).to(torch.bfloat16).expand(Hkv, N, d).contiguous().cuda() for _ in range(L)]
    imp = torch.empty(N, dtype=torch.float32, device="cuda")
    bufs = spf.binding.PromptBuffers(q, k, imp, None)
    ws = torch.empty(spf.spf_score_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
    spf.spf_score([bufs], ws)
    np.testing.assert_allclose(imp.cpu().numpy(), 1.0 / N, rtol=1e-4)


def test_rows_sum_to_one_through_gpu_lse(spf):
    cfg = small_config("lse", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(3000,), seed=12)
    prompt = make_prompt(cfg)
    gpu = gpu_run(prompt, 0.25)
    qv = oracle.bf16_to_f64(bf16_bits(prompt.q))
    for l in range(2):
        for h in range(4):
            kv = oracle.bf16_to_f64(bf16_bits(prompt.k[l][h // 2]))
            z = (qv[l, h] @ kv.T) / 8.0
            total = np.exp(z - gpu["lse"][l, h][:, None].astype(np.float64)).sum(axis=1)
            np.testing.assert_allclose(total, 1.0, atol=1e-5)


# ------------------------------------------------------------------ the selection calls on their own
def test_chunk_pool_alone(spf):
    rng = np.random.default_rng(0)
    for n, w, c in [(1000, 13, 32), (1, 13, 32), (77, 1, 8), (4096, 13, 128), (333, 5, 7), (5000, 255, 64)]:
        x = rng.random(n).astype(np.float32) ** 8
        out = torch.empty((n + c - 1) // c, dtype=torch.float32, device="cuda")
        spf.spf_chunk_pool(torch.from_numpy(x).cuda(), w, c, out)
        want = oracle.chunk_means(oracle.avg_pool(x.astype(np.float64), w), c)
        np.testing.assert_allclose(out.cpu().numpy(), want, rtol=2e-6)


def test_select_topk_alone_is_exact_with_ties(spf):
    rng = np.random.default_rng(1)
    cases = []
    for _ in range(30):
        C = int(rng.integers(1, 5000))
        kind = rng.integers(0, 3)
        if kind == 0:
            cs = rng.random(C).astype(np.float32)
        elif kind == 1:
            cs = rng.integers(0, 4, size=C).astype(np.float32)          # heavy ties
        else:
            cs = (rng.normal(size=C) * 10.0 ** rng.integers(-20, 20)).astype(np.float32)   # signs and scales
        cases.append((cs, int(rng.integers(1, C + 1))))
    cases.append((np.zeros(100, dtype=np.float32), 7))
    cases.append((np.array([0.0, -0.0, 0.0, -0.0], dtype=np.float32), 2))
    cases.append((np.arange(3000, dtype=np.float32), 3000))
    cases.append((rng.random(70000).astype(np.float32), 6999))
    for cs, k in cases:
        kept = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        spf.spf_select_topk(torch.from_numpy(cs).cuda(), len(cs), k, kept)
        assert kept.cpu().numpy().tolist() == oracle.select_topk(cs.astype(np.float64), k).tolist()


def test_compact_spans_alone(spf):
    rng = np.random.default_rng(2)
    for n, c in [(1000, 32), (1003, 32), (50, 64), (4096, 128), (9999, 1), (131072, 32)]:
        C = (n + c - 1) // c
        ids = rng.integers(0, 32000, size=n, dtype=np.int32)
        lens = rng.integers(0, 9, size=n)
        ends = np.cumsum(lens).astype(np.int32)
        starts = (ends - lens).astype(np.int32)
        for k in sorted({1, max(1, C // 10), max(1, C // 2), C}):
            patterns = [np.sort(rng.choice(C, size=k, replace=False))]
            if k < C:
                patterns.append(np.arange(C - k, C))                   # one run ending at the (maybe short) last chunk
            for kept in patterns:
                d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
                out_ids = torch.full((min(k * c, n),), -1, dtype=torch.int32, device="cuda")
                out_pos = torch.full_like(out_ids, -1)
                tok = torch.full((k, 2), -1, dtype=torch.int32, device="cuda")
                ch = torch.full((k, 2), -1, dtype=torch.int32, device="cuda")
                counts = torch.zeros(2, dtype=torch.int64, device="cuda")
                spf.spf_compact_spans(d(kept.astype(np.int32)), k, c, n, d(ids), d(starts), d(ends), out_ids, out_pos,
                                      tok, ch, counts)
                w_ids, w_pos, w_tok, w_ch = oracle.compact(kept, c, n, ids.astype(np.int64), starts.astype(np.int64),
                                                           ends.astype(np.int64))
                n_kept, n_spans = counts.cpu().tolist()
                assert n_kept == len(w_ids) and n_spans == len(w_tok)
                assert np.array_equal(out_ids.cpu().numpy()[:n_kept], w_ids)
                assert np.array_equal(out_pos.cpu().numpy()[:n_kept], w_pos)
                assert np.array_equal(tok.cpu().numpy()[:n_spans], w_tok)
                assert np.array_equal(ch.cpu().numpy()[:n_spans], w_ch)
                assert (tok.cpu().numpy()[n_spans:] == -1).all()       # rows beyond n_spans untouched


def test_compact_without_positions(spf):
    n, c, k = 100, 10, 3
    d = lambda a: torch.tensor(a, dtype=torch.int32, device="cuda")
    ids = torch.arange(n, dtype=torch.int32, device="cuda") + 500
    starts = torch.arange(n, dtype=torch.int32, device="cuda") * 2
    out_ids = torch.empty(k * c, dtype=torch.int32, device="cuda")
    tok = torch.empty((k, 2), dtype=torch.int32, device="cuda")
    ch = torch.empty((k, 2), dtype=torch.int32, device="cuda")
    counts = torch.zeros(2, dtype=torch.int64, device="cuda")
    spf.spf_compact_spans(d([1, 2, 7]), k, c, n, ids, starts, starts + 2, out_ids, None, tok, ch, counts)
    assert counts.cpu().tolist() == [30, 2]
    assert tok.cpu().numpy()[:2].tolist() == [[10, 30], [70, 80]] and ch.cpu().numpy()[:2].tolist() == [[20, 60], [140, 160]]
    assert out_ids.cpu().numpy().tolist() == list(range(510, 530)) + list(range(570, 580))


def test_determinism_across_runs(spf):
    prompt = make_prompt(small_config("det", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=16,
                                      lengths=(5000,), seed=4))
    first = gpu_run(prompt, 0.1)
    for _ in range(3):
        again = gpu_run(prompt, 0.1)
        assert np.array_equal(first["importance"], again["importance"])
        assert np.array_equal(first["kept"], again["kept"])


def test_host_buffer_entry_matches_device_entry(spf):
    """Selector.run_host (pinned host tensors in, host arrays out) gives what Selector.run gives on device tensors."""
    cfg = small_config("host", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(3000,), seed=8)
    prompt = make_prompt(cfg)
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, prompt.n_tokens,
                       chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)
    pin = lambda t: t.pin_memory()
    host = sel.run_host(pin(prompt.q), [pin(x) for x in prompt.k], pin(prompt.token_ids), pin(prompt.char_start),
                        pin(prompt.char_end), 0.2)
    dev = gpu_run(prompt, 0.2, sel)
    for key in ("ids", "pos", "tok_spans", "char_spans"):
        assert np.array_equal(host[key], dev[key])
