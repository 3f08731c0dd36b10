"""Helpers shared by the GPU parity tests: run the CUDA path and the oracle on the same bytes and compare."""
import numpy as np
import torch

import oracle
from workloads import bf16_bits

IMPORTANCE_RTOL = 1e-3   # relative error allowed on token importance (fp32 path vs fp64 oracle)
BOUNDARY_BAND = 1e-3     # chunks whose oracle score is this close (relative) to the k-th score may differ


def oracle_run(prompt, keep):
    cfg = prompt.cfg
    return oracle.compress(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k], prompt.token_ids.cpu().numpy(),
                           prompt.char_start.cpu().numpy(), prompt.char_end.cpu().numpy(), chunk=cfg.chunk, keep=keep,
                           pool_kernel=cfg.pool_kernel)


def gpu_run(prompt, keep, selector=None):
    """Runs the whole CUDA path; a non-zero device status (timeout, range) fails the test."""
    import paper_2603_02631_b200 as spf
    cfg = prompt.cfg
    dp = prompt.to("cuda")
    sel = selector or spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead,
                                   max_tokens=prompt.n_tokens, chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)
    res = sel.run(dp.q, dp.k, dp.token_ids, dp.char_start, dp.char_end, keep)
    torch.cuda.synchronize()
    assert int(sel.dev_status.item()) == 0
    return res.host()


def assert_importance_close(got, want, rtol=IMPORTANCE_RTOL):
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == want.shape
    assert np.isfinite(got).all()
    rel = np.abs(got - want) / np.maximum(np.abs(want), 1e-30)
    worst = int(rel.argmax())
    assert rel[worst] <= rtol, f"importance[{worst}] = {got[worst]!r}, oracle {want[worst]!r}, rel err {rel[worst]:.3e}"
    return float(rel.max())


def assert_selection_matches(gpu, ref, prompt):
    """Kept chunks equal the oracle's except inside the tie band; compaction is bit-exact given the kept set."""
    cfg = prompt.cfg
    n = prompt.n_tokens
    assert gpu["k"] == ref["k"]
    k = ref["k"]
    g_kept, o_kept = gpu["kept"].astype(np.int64), ref["kept"]
    assert len(g_kept) == k and (np.diff(g_kept) > 0).all() and g_kept.min() >= 0 and g_kept.max() < len(ref["chunk_scores"])
    cs = ref["chunk_scores"]
    tau = np.sort(cs)[::-1][k - 1]
    differ = np.setxor1d(g_kept, o_kept)
    if len(differ):
        assert (np.abs(cs[differ] - tau) <= BOUNDARY_BAND * abs(tau)).all(), \
            f"chunks {differ.tolist()} differ outside the tie band (tau={tau}, scores={cs[differ].tolist()})"
    # compaction of the GPU's own kept set must be exact
    ids, pos, tok, ch = oracle.compact(g_kept, cfg.chunk, n, prompt.token_ids.cpu().numpy().astype(np.int64),
                                       prompt.char_start.cpu().numpy().astype(np.int64),
                                       prompt.char_end.cpu().numpy().astype(np.int64))
    assert np.array_equal(gpu["ids"], ids) and np.array_equal(gpu["pos"], pos)
    assert np.array_equal(gpu["tok_spans"], tok) and np.array_equal(gpu["char_spans"], ch)
    return len(differ)


def compare_full(prompt, keep, selector=None):
    ref = oracle_run(prompt, keep)
    gpu = gpu_run(prompt, keep, selector)
    err = assert_importance_close(gpu["importance"], ref["importance"])
    np.testing.assert_allclose(gpu["lse"], ref["lse"], rtol=0, atol=2e-4)
    np.testing.assert_allclose(gpu["chunk_scores"], ref["chunk_scores"], rtol=IMPORTANCE_RTOL)
    n_diff = assert_selection_matches(gpu, ref, prompt)
    return ref, gpu, err, n_diff
