"""Pins of the oracle's 8-bit key-cache functions (CPU only): the E4M3 decoder against the format's definition,
against torch's own conversion for all 256 bytes and against hand values; the fp8 importance against the bf16
oracle on inputs where the two must agree exactly."""
import numpy as np
import pytest
import torch

import oracle
from workloads import bf16_bits, make_prompt, quantize_keys_e4m3, small_config


def test_e4m3_hand_values():
    dec = oracle.fp8_e4m3_to_f64
    cases = {0x00: 0.0, 0x38: 1.0, 0xB8: -1.0, 0x3C: 1.5, 0x40: 2.0, 0x7E: 448.0, 0xFE: -448.0, 0x01: 2.0 ** -9,
             0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x0F: 1.875 * 2.0 ** -6, 0x78: 256.0, 0x30: 0.5, 0x29: 0.28125}
    got = dec(np.array(list(cases), dtype=np.uint8))
    assert got.tolist() == list(cases.values())
    assert np.signbit(dec(np.array([0x80], dtype=np.uint8))[0]) and dec(np.array([0x80], dtype=np.uint8))[0] == 0.0
    assert np.isnan(dec(np.array([0x7F, 0xFF], dtype=np.uint8))).all()


def test_e4m3_matches_torch_for_every_byte():
    bits = np.arange(256, dtype=np.uint8)
    want = torch.from_numpy(bits.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = oracle.fp8_e4m3_to_f64(bits)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])


def test_e4m3_is_monotone_and_symmetric():
    pos = oracle.fp8_e4m3_to_f64(np.arange(0x00, 0x7F, dtype=np.uint8))
    assert (np.diff(pos) > 0).all()                        # bit patterns of one sign order like their values
    neg = oracle.fp8_e4m3_to_f64(np.arange(0x80, 0xFF, dtype=np.uint8))
    assert np.array_equal(neg, -pos)


def _case(seed=3, n=700):
    cfg = small_config("fp8pin", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=4, lengths=(n,),
                       rank=4, n_needles=2, seed=seed)
    p = make_prompt(cfg)
    k8, scales = quantize_keys_e4m3(p.k)
    return p, [x.numpy() for x in k8], scales.numpy()


def test_fp8_importance_equals_bf16_importance_when_the_scale_is_a_power_of_two():
    """With a power-of-two scale every decoded key is a bf16 number, so the 8-bit oracle must reproduce the bf16 oracle
    on those keys exactly (same products, same sums)."""
    p, k8, _ = _case()
    scales = np.array([[0.25, 2.0], [1.0, 0.0625]], dtype=np.float32)
    k_bf16 = []
    for l, kb in enumerate(k8):
        vals = oracle.fp8_e4m3_to_f64(kb) * scales[l][:, None, None].astype(np.float64)
        t = torch.from_numpy(vals).to(torch.bfloat16)
        assert np.array_equal(t.to(torch.float64).numpy(), vals)          # exactly representable
        k_bf16.append(bf16_bits(t))
    want, want_lse = oracle.token_importance(bf16_bits(p.q), k_bf16)
    got, got_lse = oracle.token_importance_fp8(bf16_bits(p.q), k8, scales)
    np.testing.assert_allclose(got, want, rtol=1e-13, atol=0)
    np.testing.assert_allclose(got_lse, want_lse, rtol=0, atol=1e-12)


def test_fp8_scale_and_softmax_scale_trade_off():
    """Multiplying every key scale by s and dividing the softmax scale by s changes no logit."""
    p, k8, scales = _case(seed=4)
    a, a_lse = oracle.token_importance_fp8(bf16_bits(p.q), k8, scales, scale=0.125)
    b, b_lse = oracle.token_importance_fp8(bf16_bits(p.q), k8, scales * np.float32(4.0), scale=0.125 / 4.0)
    np.testing.assert_allclose(a, b, rtol=1e-12)
    np.testing.assert_allclose(a_lse, b_lse, rtol=0, atol=1e-12)


def test_fp8_importance_uses_the_scale_of_its_own_kv_head():
    """A wrong index into the scales (layer and kv-head swapped, or one scale for all) must show: permuting the kv-heads
    of keys and scales together, and the query heads with them, changes nothing; permuting only the scales does."""
    p, k8, scales = _case(seed=5)
    base, _ = oracle.token_importance_fp8(bf16_bits(p.q), k8, scales)
    q = bf16_bits(p.q)                                     # [L, Hq=4, m, d], G = 2: heads (0,1) -> kv 0, (2,3) -> kv 1
    q_sw = q[:, [2, 3, 0, 1]]
    k_sw = [kb[[1, 0]] for kb in k8]
    same, _ = oracle.token_importance_fp8(q_sw, k_sw, scales[:, [1, 0]])
    np.testing.assert_allclose(same, base, rtol=1e-12)
    other, _ = oracle.token_importance_fp8(q_sw, k_sw, scales)
    assert np.abs(other - base).max() > 1e-6 * base.max()


def test_quantised_keys_stay_close_to_the_originals():
    """The generator's 8-bit copy is a faithful stand-in (relative error of a 4-bit significand), so the workload keeps
    its structure: the planted needles still stand out."""
    p, k8, scales = _case(seed=6)
    for l, kb in enumerate(k8):
        dec = oracle.fp8_e4m3_to_f64(kb) * scales[l][:, None, None]
        ref = p.k[l].to(torch.float64).numpy()
        assert np.abs(dec - ref).max() <= 0.07 * np.abs(ref).max()
