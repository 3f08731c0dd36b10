"""8-bit key caches (spf_score_fp8) against the oracle on the same bytes, on both kernel paths: small shapes with ragged
tails, every row-count template, strided caches, and the long-context geometry at full size.  The fused path feeds the
tensor cores E4M3 keys and queries split into two E4M3 terms (exact but for elements 2^9 below a slab's largest), so
the same tolerances hold on both paths."""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, bf16_bits, make_prompt, quantize_keys_e4m3, small_config

from parity_util import IMPORTANCE_RTOL, assert_importance_close, assert_selection_matches

pytestmark = pytest.mark.gpu

SHAPES = [
    # L, Hq, Hkv, d, m, N
    (2, 4, 2, 64, 8, 1000),
    (1, 8, 2, 64, 8, 4097),
    (2, 8, 1, 64, 8, 2500),
    (2, 8, 2, 64, 16, 3001),
    (3, 16, 8, 128, 8, 2049),
    (2, 6, 2, 64, 5, 1234),
    (1, 2, 1, 128, 32, 650),
    (2, 4, 2, 64, 8, 31),
    (1, 1, 1, 64, 8, 1),
]


@pytest.fixture(params=["general", "fused"])
def kernel_path(request):
    """Pins the scoring path for one test; a shape the fused path refuses (status -2) turns into a skip (conftest)."""
    import paper_2603_02631_b200 as spf
    previous = spf.spf_set_score_path(1 if request.param == "general" else 2)
    yield request.param
    spf.spf_set_score_path(previous)


def _run(spf, q, k8, scales, n, lse_rows):
    imp = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((lse_rows,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bufs = spf.Fp8PromptBuffers(q, k8, scales, imp, lse)
    ws = torch.empty(spf.spf_score_fp8_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
    spf.spf_score_fp8([bufs], ws, 0.0, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return imp.cpu().numpy(), lse.cpu().numpy()


@pytest.mark.parametrize("L,Hq,Hkv,d,m,N", SHAPES)
def test_fp8_small_shapes(kernel_path, L, Hq, Hkv, d, m, N):
    import paper_2603_02631_b200 as spf
    cfg = small_config("fp8", n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, n_lookahead=m, lengths=(N,),
                       rank=4, n_needles=2 if N >= 300 else 0, n_strong=1, needle_len=(4, 40), seed=N + m)
    prompt = make_prompt(cfg)
    k8, scales = quantize_keys_e4m3(prompt.k)
    want, want_lse = oracle.token_importance_fp8(bf16_bits(prompt.q), [x.numpy() for x in k8], scales.numpy())
    got, got_lse = _run(spf, prompt.q.cuda(), [x.cuda() for x in k8], scales.cuda(), N, L * Hq * m)
    assert_importance_close(got, want)
    np.testing.assert_allclose(got_lse.reshape(want_lse.shape), want_lse, rtol=0, atol=2e-4)


def test_fp8_every_byte_value_is_decoded_exactly(kernel_path):
    """A cache that holds every finite E4M3 byte: one head, d = 64, query = a unit vector along each coordinate in turn, so
    each logit is one decoded key value times the scale (exact in fp32): checks the kernel's decoder bit for bit through
    the log-sum-exp and the importance."""
    import paper_2603_02631_b200 as spf
    finite = [b for b in range(256) if b not in (0x7F, 0xFF)]
    n, d = 508, 64                                        # 254 finite bytes x 2
    rng = np.random.default_rng(0)
    kb = rng.choice(finite, size=(1, n, d)).astype(np.uint8)
    kb[0, :254, 0] = finite                                # coordinate 0 of the first 254 keys: every finite byte once
    q = torch.zeros(1, 1, 8, d)
    for i in range(8):
        q[0, 0, i, i] = 1.0 if i else 0.125               # lookahead 0 reads coordinate 0 with a small weight
    q = q.to(torch.bfloat16)
    scales = torch.tensor([[0.0625]], dtype=torch.float32)
    want, want_lse = oracle.token_importance_fp8(bf16_bits(q), [kb], scales.numpy())
    got, got_lse = _run(spf, q.cuda(), [torch.from_numpy(kb).cuda()], scales.cuda(), n, 8)
    assert_importance_close(got, want)
    np.testing.assert_allclose(got_lse.reshape(want_lse.shape), want_lse, rtol=0, atol=2e-4)


@pytest.mark.parametrize("row,first", [(136, 8), (144, 16)])
def test_fp8_strided_cache(kernel_path, row, first):
    """Keys interleaved with other data (a fused KV layout): strides in bytes.  Rows 8-byte aligned are enough for the
    general path; the fused path wants 16 (and refuses the other case, which the automatic choice hands to the general path)."""
    import paper_2603_02631_b200 as spf
    cfg = small_config("fp8s", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(777,), rank=4, seed=9)
    prompt = make_prompt(cfg)
    k8, scales = quantize_keys_e4m3(prompt.k)
    wide = [torch.full((2, 777, row), 0x7E, dtype=torch.uint8, device="cuda") for _ in k8]   # 448s around the keys
    for w, x in zip(wide, k8):
        w[:, :, first:first + 64] = x.cuda()
    views = [w[:, :, first:first + 64] for w in wide]
    want, _ = oracle.token_importance_fp8(bf16_bits(prompt.q), [x.numpy() for x in k8], scales.numpy())
    got, _ = _run(spf, prompt.q.cuda(), views, scales.cuda(), 777, 2 * 4 * 8)
    assert_importance_close(got, want)


def test_fp8_long_context_full_size(kernel_path):
    """The long-context configuration with its key cache in 8 bits, end to end (score -> pool -> top-k -> spans)."""
    import paper_2603_02631_b200 as spf
    cfg = CONFIGS["long128k"]
    prompt = make_prompt(cfg, 0, "cuda")
    k8, scales = quantize_keys_e4m3(prompt.k)
    n = prompt.n_tokens
    want_imp, want_lse = oracle.token_importance_fp8(bf16_bits(prompt.q), [x.cpu().numpy() for x in k8], scales.cpu().numpy())
    want_scores = oracle.chunk_means(oracle.avg_pool(want_imp, cfg.pool_kernel), cfg.chunk)
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n, chunk=cfg.chunk,
                       pool_kernel=cfg.pool_kernel)
    keep = cfg.keep[0]
    got = sel.run_fp8(prompt.q, k8, scales, prompt.token_ids, prompt.char_start, prompt.char_end, keep)
    torch.cuda.synchronize()
    got = got.host()
    assert_importance_close(got["importance"], want_imp)
    np.testing.assert_allclose(got["lse"], want_lse, rtol=0, atol=2e-4)
    np.testing.assert_allclose(got["chunk_scores"], want_scores, rtol=IMPORTANCE_RTOL)
    ids, cs, ce = (t.cpu().numpy().astype(np.int64) for t in (prompt.token_ids, prompt.char_start, prompt.char_end))
    k = oracle.keep_count(len(want_scores), keep)
    kept = oracle.select_topk(want_scores, k)
    o_ids, o_pos, o_tok, o_ch = oracle.compact(kept, cfg.chunk, n, ids, cs, ce)
    assert_selection_matches(got, dict(k=k, kept=kept, chunk_scores=want_scores, ids=o_ids, pos=o_pos, tok_spans=o_tok,
                                       char_spans=o_ch), prompt)


def test_fp8_queries_with_a_wide_dynamic_range(kernel_path):
    """Query elements spread over 2^-14 .. 1 of their slab's largest: on the fused path the small ones pass the two-term
    split inexactly (by at most 2^-17 of the largest), which must stay far inside the tolerance."""
    import paper_2603_02631_b200 as spf
    cfg = small_config("fp8w", n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=8, lengths=(1500,), rank=4,
                       n_needles=2, n_strong=1, needle_len=(4, 40), seed=77)
    prompt = make_prompt(cfg)
    g = torch.Generator().manual_seed(5)
    expo = torch.randint(-14, 1, prompt.q.shape, generator=g).to(torch.float32)
    q = (prompt.q.to(torch.float32) * torch.exp2(expo) * 8.0).to(torch.bfloat16)
    k8, scales = quantize_keys_e4m3(prompt.k)
    want, want_lse = oracle.token_importance_fp8(bf16_bits(q), [x.numpy() for x in k8], scales.numpy())
    got, got_lse = _run(spf, q.cuda(), [x.cuda() for x in k8], scales.cuda(), 1500, 2 * 8 * 8)
    assert_importance_close(got, want)
    np.testing.assert_allclose(got_lse.reshape(want_lse.shape), want_lse, rtol=0, atol=2e-4)


def test_fp8_unaligned_cache_goes_to_the_general_path_by_itself():
    """Rows that start 8 bytes into a 16-byte unit: the fused path cannot read them, the automatic choice must not try."""
    import paper_2603_02631_b200 as spf
    cfg = small_config("fp8u", n_layers=1, n_q_heads=2, n_kv_heads=1, head_dim=64, n_lookahead=8, lengths=(300,), seed=1)
    prompt = make_prompt(cfg)
    k8, scales = quantize_keys_e4m3(prompt.k)
    wide = torch.zeros((1, 300, 136), dtype=torch.uint8, device="cuda")
    wide[:, :, 8:72] = k8[0].cuda()
    want, _ = oracle.token_importance_fp8(bf16_bits(prompt.q), [k8[0].numpy()], scales.numpy())
    assert spf.spf_set_score_path(0) == 0
    got, _ = _run(spf, prompt.q.cuda(), [wide[:, :, 8:72]], scales.cuda(), 300, 2 * 8)
    assert_importance_close(got, want)
