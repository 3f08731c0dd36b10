"""spf_score writes only where it may: importance[0:N], lse and its workspace.

compute-sanitizer is not available where these tests run, so the check is done with guard bands: every output and
the workspace sit inside one large buffer between 4 KB bands of a known byte pattern, and the bands must be intact
after the call.  Both kernel paths, shapes with ragged tails, a prompt batch, and the paged entry point.
"""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, small_config

from parity_util import assert_importance_close

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


class Arena:
    """One device buffer; carve() hands out regions separated by guard bands."""

    def __init__(self, nbytes):
        self.buf = torch.full((nbytes,), PATTERN, dtype=torch.uint8, device="cuda")
        self.used = []          # (start, stop) of every carved region
        self.pos = GUARD

    def carve(self, nbytes, dtype):
        start = (self.pos + 4095) // 4096 * 4096
        stop = start + nbytes
        assert stop + GUARD <= self.buf.numel()
        self.used.append((start, stop))
        self.pos = stop + GUARD
        return self.buf[start:stop].view(dtype)

    def assert_guards_intact(self):
        mask = torch.ones(self.buf.numel(), dtype=torch.bool, device="cuda")
        for start, stop in self.used:
            mask[start:stop] = False
        bad = (self.buf[mask] != PATTERN).nonzero()
        assert bad.numel() == 0, f"{bad.numel()} guard bytes were overwritten (first at guard index {int(bad[0])})"


SHAPES = [
    # L, Hq, Hkv, d, m, N
    (2, 8, 2, 64, 16, 3001),
    (3, 16, 8, 128, 8, 2049),
    (1, 4, 1, 64, 16, 50000),
    (2, 4, 2, 64, 8, 31),
    (1, 2, 1, 64, 20, 900),
]


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("L,Hq,Hkv,d,m,N", SHAPES)
def test_score_stays_inside_its_buffers(path, L, Hq, Hkv, d, m, N):
    import paper_2603_02631_b200 as spf
    cfg = small_config("canary", n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, n_lookahead=m, lengths=(N,),
                       rank=4, n_needles=0, seed=N)
    prompt = make_prompt(cfg)
    dp = prompt.to("cuda")
    previous = spf.spf_set_score_path(path)
    try:
        probe = spf.PromptBuffers(dp.q, dp.k, torch.empty(N, dtype=torch.float32, device="cuda"), None)
        ws_bytes = spf.spf_score_workspace_bytes([probe])
        arena = Arena(4 * N + 4 * L * Hq * m + ws_bytes + 16 * GUARD)
        imp = arena.carve(4 * N, torch.float32)
        lse = arena.carve(4 * L * Hq * m, torch.float32)
        ws = arena.carve(ws_bytes, torch.uint8)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        spf.spf_score([spf.PromptBuffers(dp.q, dp.k, imp, lse)], ws, 0.0, status)
        torch.cuda.synchronize()
    except spf.SpfError as err:
        if err.status == -2 and path == 2:
            pytest.skip("shape outside the fused path")
        raise
    finally:
        spf.spf_set_score_path(previous)
    assert int(status.item()) == 0
    arena.assert_guards_intact()
    want, _ = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k])
    assert_importance_close(imp.cpu().numpy(), want)


def test_selection_calls_stay_inside_their_buffers():
    """chunk pool -> top-k -> compaction with every output between guard bands (sizes as include/spf.h states them)."""
    import paper_2603_02631_b200 as spf
    n, chunk, keep = 10007, 32, 0.3
    g = torch.Generator().manual_seed(3)
    importance = torch.rand(n, generator=g).cuda()
    n_chunks = (n + chunk - 1) // chunk
    k = spf.spf_keep_count(n_chunks, keep)
    arena = Arena(4 * n_chunks + 4 * k + 2 * 4 * min(k * chunk, n) + 2 * 8 * k + 16 + 16 * GUARD)
    scores = arena.carve(4 * n_chunks, torch.float32)
    kept = arena.carve(4 * k, torch.int32)
    out_ids = arena.carve(4 * min(k * chunk, n), torch.int32)
    out_pos = arena.carve(4 * min(k * chunk, n), torch.int32)
    tok = arena.carve(8 * k, torch.int32)
    ch = arena.carve(8 * k, torch.int32)
    counts = arena.carve(16, torch.int64)
    ids = torch.arange(n, dtype=torch.int32, device="cuda")
    spf.spf_chunk_pool(importance, 13, chunk, scores)
    spf.spf_select_topk(scores, n_chunks, k, kept)
    spf.spf_compact_spans(kept, k, chunk, n, ids, ids * 3, ids * 3 + 3, out_ids, out_pos, tok, ch, counts)
    torch.cuda.synchronize()
    arena.assert_guards_intact()
    want_scores = oracle.chunk_means(oracle.avg_pool(importance.cpu().numpy().astype(np.float64), 13), chunk)
    np.testing.assert_allclose(scores.cpu().numpy(), want_scores, rtol=1e-5)
