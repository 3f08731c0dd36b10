"""spf_score_static: the scoring entry point for callers that cannot allocate device memory.

A serving engine that has handed all free HBM to its KV-cache pool, or code that must not trigger
the device-wide synchronisation of cudaMalloc, cannot provide the workspace spf_score asks for.
spf_score_static uses a fixed scratch array inside the library instead.  These tests call it through
the C ABI and require the importance and log-sum-exp of the CPU oracle, and of spf_score with a caller-owned
workspace, on two calls in a row (the second one sees whatever the first left in the shared array); and they
require that the call leaves the amount of free device memory exactly as it found it, which is the property the
entry point exists for.

This file is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, small_config

from parity_util import IMPORTANCE_RTOL, assert_importance_close


def _score_both(spf, prompt):
    """Runs spf_score (own workspace) and spf_score_static on one prompt; returns both results on the host."""
    cfg = prompt.cfg
    dp = prompt.to("cuda")
    n = prompt.n_tokens
    n_rows = cfg.n_layers * cfg.n_q_heads * cfg.n_lookahead
    out = []
    for static in (False, True):
        imp = torch.full((n,), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((n_rows,), float("nan"), dtype=torch.float32, device="cuda")
        bufs = spf.PromptBuffers(dp.q, dp.k, imp, lse)
        if static:
            # everything the call touches is allocated by now; the call itself must not change what the device has free
            # (measured at the driver, below torch's caching allocator) nor what torch has handed out
            torch.cuda.synchronize()
            free_before, _ = torch.cuda.mem_get_info()
            torch_before = torch.cuda.memory_allocated()
            spf.spf_score_static([bufs])
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info()
            assert free_after == free_before, f"spf_score_static changed free device memory by {free_before - free_after} bytes"
            assert torch.cuda.memory_allocated() == torch_before
        else:
            ws = torch.empty(spf.spf_score_workspace_bytes([bufs]), dtype=torch.uint8, device="cuda")
            spf.spf_score([bufs], ws)
        torch.cuda.synchronize()
        out.append((imp.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)))
    return out


@pytest.mark.gpu
def test_static_scratch_matches_workspace_path_twice_in_a_row():
    import paper_2603_02631_b200 as spf
    # a larger prompt first, then a smaller one of another geometry: the second call finds the
    # first call's leftovers in the shared scratch array and must not be affected by them
    shapes = [
        small_config("noalloc_a", n_layers=4, n_q_heads=8, n_kv_heads=2, head_dim=64, n_lookahead=16, lengths=(6001,), seed=31),
        small_config("noalloc_b", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=128, n_lookahead=8, lengths=(1500,), seed=32),
    ]
    # the first call on a device looks the scratch array up (and loads the module that holds it): done here, outside
    # the calls whose memory footprint is checked
    warm = make_prompt(small_config("noalloc_warm", n_layers=1, n_q_heads=2, n_kv_heads=1, head_dim=64, n_lookahead=8,
                                    lengths=(200,), seed=30)).to("cuda")
    spf.spf_score_static([spf.PromptBuffers(warm.q, warm.k, torch.empty(200, dtype=torch.float32, device="cuda"), None)])
    torch.cuda.synchronize()
    for cfg in shapes:
        prompt = make_prompt(cfg)
        (imp_ws, lse_ws), (imp_st, lse_st) = _score_both(spf, prompt)
        want_imp, want_lse = oracle.token_importance(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k])
        assert_importance_close(imp_st, want_imp)
        np.testing.assert_allclose(lse_st, want_lse.reshape(-1), rtol=0, atol=2e-4)
        assert np.isfinite(imp_st).all() and np.isfinite(lse_st).all()
        rel = np.abs(imp_st - imp_ws) / np.maximum(np.abs(imp_ws), 1e-30)
        assert rel.max() <= IMPORTANCE_RTOL, f"{cfg.name}: importance differs by {rel.max():.3e}"
        np.testing.assert_allclose(lse_st, lse_ws, rtol=0, atol=2e-4)


def test_static_scratch_rejects_prompts_that_do_not_fit():
    # host-side check only: nothing is launched and no device is touched
    import paper_2603_02631_b200 as spf
    from paper_2603_02631_b200.binding import _Prompt, _Shape
    n_layers = 128
    layers = (ctypes.c_void_p * n_layers)(*([4096] * n_layers))
    lp = ctypes.cast(layers, ctypes.POINTER(ctypes.c_void_p))
    prompt = (_Prompt * 1)(_Prompt(100000, lp, 100000 * 128, 128, 4096, 4096, None))
    shape = _Shape(n_layers, 32, 8, 128, 16, 0.0)            # 1024 slabs x 64 rows x 128 dims of packed queries alone = 16 MiB
    assert spf.lib.spf_score_static(ctypes.byref(shape), prompt, 1, None) == -3
    assert "built-in array" in spf.spf_last_error()
    assert spf.lib.spf_score_static(None, None, 0, None) == -1
