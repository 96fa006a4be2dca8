"""Pins of the oracle's IEEE fp16 input path (the paper's kernel benchmark table runs in
float16): the decoder against numpy's float16 on every bit pattern, the quantizer against
the torch CPU cast, and the 16-bit attention reference against an fp64 brute force."""
import numpy as np
import torch

import oracle
from helpers import numpy_attention_f64


def test_half_decode_matches_numpy_on_every_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.half_to_float(int(b)) for b in bits])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))     # -0.0 keeps its sign


def test_quantize_fp16_matches_torch_cpu_route():
    rng = np.random.default_rng(11)
    x = rng.standard_normal((2, 3, 37, 64)).astype(np.float32)
    x[:, :, :, 5] *= 20.0                                   # an outlier channel
    x[0, 0] *= 1e-4                                         # a head whose values are fp16 subnormals after rounding
    h = x.astype(np.float16)
    codes, s = oracle.quantize(h.view(np.uint16), dtype16="fp16")
    xt = torch.from_numpy(h.astype(np.float32))
    st = xt.abs().amax(dim=(2, 3), keepdim=True) / 448.0
    ct = (xt / st).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(s, st.numpy().reshape(2, 3))
    assert np.array_equal(codes, ct)
    # the largest entry of every head maps to +-448
    flat = codes.reshape(6, -1) & 0x7F
    assert (flat.max(axis=1) == 0x7E).all()
    # shared scale: values outside its range saturate
    t = (rng.standard_normal((2, 3, 9, 64)) * 3).astype(np.float16)
    tc, ts = oracle.quantize(t.view(np.uint16), scale_in=s / 4, dtype16="fp16")
    tt = (torch.from_numpy(t.astype(np.float32)) / torch.from_numpy(s / 4).reshape(2, 3, 1, 1)).clamp(-448, 448)
    assert np.array_equal(tc, tt.to(torch.float8_e4m3fn).view(torch.uint8).numpy())
    assert np.array_equal(ts, s / 4)


def test_fp16_reads_differ_from_bf16_reads_of_the_same_bits():
    """Guards the dtype switch itself: the same bit patterns mean different numbers."""
    bits = np.full((1, 1, 2, 64), 0x3C00, dtype=np.uint16)          # 1.0 in fp16, 0.0078125 in bf16
    bits[0, 0, 0, 0] = 0x4000                                        # 2.0 in fp16, 2.0 in bf16 (same)
    _, s16 = oracle.quantize(bits, dtype16="fp16")
    _, sbf = oracle.quantize(bits)
    assert s16[0, 0] == np.float32(2.0) / np.float32(448.0) and sbf[0, 0] == s16[0, 0]
    c16, _ = oracle.quantize(bits, dtype16="fp16")
    cbf, _ = oracle.quantize(bits)
    assert c16[0, 0, 0, 1] != cbf[0, 0, 0, 1]


def test_fp16_attention_matches_fp64_brute_force():
    rng = np.random.default_rng(3)
    B, H, N, M, d = 1, 2, 45, 7, 64
    mk = lambda r: rng.standard_normal((B, H, r, d)).astype(np.float16)
    q, k, v = mk(M), mk(N), mk(N)
    A, Abs, _ = oracle.icl_attention_rows(q.view(np.uint16), k.view(np.uint16), v.view(np.uint16),
                                          np.arange(M), dtype16="fp16")
    for h in range(H):
        ref, p = numpy_attention_f64(q[0, h].astype(np.float64), k[0, h].astype(np.float64),
                                     v[0, h].astype(np.float64), 1.0 / np.sqrt(d))
        assert np.abs(A[0, h] - ref).max() <= 1e-12
        assert np.abs(Abs[0, h] - p @ np.abs(v[0, h].astype(np.float64))).max() <= 1e-12
