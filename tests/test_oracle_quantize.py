"""Pins for the oracle's per-head absmax quantizer (Eq. 2)."""
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f64, f32_to_bf16_bits, read_golden_table
from paper_2609_13031_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")
CONST = {k: float(v) for k, v in read_golden_table(os.path.join(GOLD, "paper_constants.txt"))}


def torch_reference_quantize(bits, scale=None):
    """Third-party route: torch CPU fp32 division + float8_e4m3fn cast."""
    x = torch.from_numpy(bits.astype(np.int16)).view(torch.bfloat16).float()
    if scale is None:
        amax = x.abs().amax(dim=(2, 3), keepdim=True)
        s = torch.where(amax == 0, torch.ones_like(amax), amax / 448.0)
    else:
        s = torch.from_numpy(scale).float()[:, :, None, None]
    y = (x / s).clamp(-448.0, 448.0)
    return y.to(torch.float8_e4m3fn).view(torch.uint8).numpy(), s[:, :, 0, 0].numpy()


@pytest.mark.parametrize("cfg", ["C1", "C2"])
def test_matches_torch_cast_route(cfg):
    w = W.CONFIGS[cfg]
    if cfg == "C2":
        w = w.scaled(2048, 512)
    g = W.generate(w)
    for name in ("q_train", "k", "v"):
        codes, s = oracle.quantize(g[name])
        rc, rs = torch_reference_quantize(g[name])
        assert np.array_equal(s, rs)
        assert np.array_equal(codes, rc)
    _, sq = oracle.quantize(g["q_train"])
    codes, s = oracle.quantize(g["q_test"], scale_in=sq)
    rc, _ = torch_reference_quantize(g["q_test"], sq)
    assert np.array_equal(s, sq) and np.array_equal(codes, rc)


def test_largest_entry_maps_to_448_and_codes_on_grid():
    # Method section: "the largest entry of each head maps to +-448"
    g = W.generate(W.CONFIGS["C1"])
    for name in ("q_train", "k", "v"):
        codes, s = oracle.quantize(g[name])
        x = bf16_bits_to_f64(g[name])
        assert not np.any((codes & 0x7F) == 0x7F)
        for b in range(codes.shape[0]):
            for h in range(codes.shape[1]):
                i = np.argmax(np.abs(x[b, h]))
                assert (codes[b, h].ravel()[i] & 0x7F) == 0x7E
                # scale = amax/448, recomputed in fp64 and rounded to fp32
                assert s[b, h] == np.float32(np.abs(x[b, h]).max() / CONST["e4m3_max"])


def test_relative_error_matches_paper_constant():
    # Appendix (noise experiment): quantization error is typically 0.0265
    tab = oracle.e4m3_decode_table()
    for cfg in ("C1",):
        g = W.generate(W.CONFIGS[cfg].scaled(4096, 128))
        for name in ("q_train", "k", "v"):
            codes, s = oracle.quantize(g[name])
            x = bf16_bits_to_f64(g[name])
            xh = tab[codes] * s[:, :, None, None].astype(np.float64)
            rel = np.sqrt(((xh - x) ** 2).sum(axis=(2, 3)) / (x ** 2).sum(axis=(2, 3)))
            assert np.all(np.abs(rel - CONST["typical_quant_rel_error"]) < 1e-3), rel


def test_idempotent_on_quantized_data():
    tab = oracle.e4m3_decode_table()
    g = W.generate(W.CONFIGS["C1"])
    codes, s = oracle.quantize(g["v"])
    # dequantize with a power-of-two-free scale is not exactly bf16, so use the
    # grid values themselves (scale 1 after requantization: amax = 448)
    grid_vals = tab[codes].astype(np.float32)
    bits = f32_to_bf16_bits(grid_vals)          # every e4m3 value is a bf16 value
    assert np.array_equal(bf16_bits_to_f64(bits), tab[codes])
    codes2, s2 = oracle.quantize(bits)
    assert np.all(s2 == 1.0)
    assert np.array_equal(codes2 & 0x7F, codes & 0x7F)
    nz = (codes & 0x7F) != 0
    assert np.array_equal(codes2[nz], codes[nz])


def test_zero_head_and_saturating_shared_scale():
    x = np.zeros((1, 2, 4, 64), dtype=np.float32)
    x[0, 1] = np.linspace(-2, 2, 256, dtype=np.float32).reshape(4, 64)
    bits = f32_to_bf16_bits(x)
    codes, s = oracle.quantize(bits)
    assert s[0, 0] == 1.0 and np.all((codes[0, 0] & 0x7F) == 0)
    assert s[0, 1] == np.float32(2.0) / np.float32(448.0)
    # test queries larger than the train range saturate at +-448
    big = f32_to_bf16_bits(np.full((1, 2, 1, 64), 1000.0, dtype=np.float32))
    big[0, 1, 0, 1::2] |= 0x8000
    c2, s2 = oracle.quantize(big, scale_in=s)
    assert np.array_equal(s2, s)
    assert np.all(c2[0, :, 0, 0::2] == 0x7E) and np.all(c2[0, 1, 0, 1::2] == 0xFE)


def test_heads_are_independent_and_shift_moves_scale():
    w = W.CONFIGS["C4"].scaled(256, 64)
    g = W.generate(w)
    codes, s = oracle.quantize(g["k"])
    x = bf16_bits_to_f64(g["k"])
    # K carries a constant mean of 3: amax ~ 3 + max z
    assert np.all(s * 448.0 > 5.0) and np.all(s * 448.0 < 9.0)
    assert abs(x.mean() - 3.0) < 0.05
    # scaling one head by 1000 leaves every other head's codes and scale unchanged
    y = g["k"].copy()
    xf = W.bf16_bits_to_f32(y[1, 2]) * np.float32(1024.0)
    y[1, 2] = f32_to_bf16_bits(xf)
    codes2, s2 = oracle.quantize(y)
    mask = np.ones((w.B, w.H), dtype=bool); mask[1, 2] = False
    assert np.array_equal(codes2[mask], codes[mask]) and np.array_equal(s2[mask], s[mask])
    assert np.array_equal(codes2[1, 2], codes[1, 2]) and s2[1, 2] == s[1, 2] * 1024
