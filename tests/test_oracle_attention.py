"""Pins for the oracle's attention: fp64 brute force over the dequantized
tensors, closed forms, softmax invariants, the ICL structure (test rows see
train rows only), the 2^8 lift of the FP8 probability tile, and the validity of
the P-quantization error bound."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f64, f32_to_bf16_bits, numpy_attention_f64
from paper_2609_13031_b200 import workloads as W


def quantized_c1(n_train=192, n_test=40):
    w = W.CONFIGS["C1"].scaled(n_train, n_test)
    g = W.generate(w)
    q8, sq = oracle.quantize(g["q_train"])
    k8, sk = oracle.quantize(g["k"])
    v8, sv = oracle.quantize(g["v"])
    t8, _ = oracle.quantize(g["q_test"], scale_in=sq)
    return w, g, dict(q8=q8, k8=k8, v8=v8, t8=t8, sq=sq, sk=sk, sv=sv)


def dequant(codes, s):
    return oracle.e4m3_decode_table()[codes] * s.astype(np.float64)[:, :, None, None]


def test_exact_mode_vs_numpy_fp64_brute_force():
    w, g, z = quantized_c1()
    alpha = 1 / np.sqrt(w.d)
    kh, vh = dequant(z["k8"], z["sk"]), dequant(z["v8"], z["sv"])
    for qname, nq in (("q8", w.n_train), ("t8", w.n_test)):
        rows = np.arange(nq)
        A, Abs, _ = oracle.icl_attention_rows(z[qname], z["k8"], z["v8"], rows,
                                              sq=z["sq"], sk=z["sk"], sv=z["sv"])
        qh = dequant(z[qname], z["sq"])
        for b in range(w.B):
            for h in range(w.H):
                ref, p = numpy_attention_f64(qh[b, h], kh[b, h], vh[b, h], alpha)
                refabs = p @ np.abs(vh[b, h])
                assert np.max(np.abs(A[b, h] - ref) / np.maximum(1, refabs)) < 1e-12
                assert np.max(np.abs(Abs[b, h] - refabs)) < 1e-12


def test_bf16_inputs_vs_numpy_fp64_brute_force():
    w = W.CONFIGS["C1"].scaled(130, 7)
    g = W.generate(w)
    alpha = 0.2
    A, Abs, _ = oracle.icl_attention_rows(g["q_test"], g["k"], g["v"], np.arange(7), alpha=alpha)
    q, k, v = (bf16_bits_to_f64(g[n]) for n in ("q_test", "k", "v"))
    for h in range(w.H):
        ref, _ = numpy_attention_f64(q[0, h], k[0, h], v[0, h], alpha)
        assert np.max(np.abs(A[0, h] - ref)) < 1e-12


def test_softmax_rows_sum_to_one_and_cover_train_rows_only():
    w, g, z = quantized_c1()
    for row in (0, 5, w.n_test - 1):
        p = oracle.softmax_row(z["t8"], z["k8"], bh=1, row=row, sq=z["sq"][0, 1], sk=z["sk"][0, 1])
        assert p.shape == (w.n_train,)          # one weight per TRAIN row, none for test rows
        assert abs(p.sum() - 1.0) < 1e-12 and np.all(p >= 0)


def test_closed_forms():
    rng = np.random.default_rng(3)
    B, H, N, d = 1, 2, 37, 64
    v = f32_to_bf16_bits(rng.standard_normal((B, H, N, d)).astype(np.float32))
    vf = bf16_bits_to_f64(v)
    q = f32_to_bf16_bits(rng.standard_normal((B, H, 5, d)).astype(np.float32))
    rows = np.arange(5)
    # all keys identical -> uniform weights -> mean of the value rows
    k_same = np.broadcast_to(f32_to_bf16_bits(rng.standard_normal((B, H, 1, d)).astype(np.float32)),
                             (B, H, N, d)).copy()
    A, _, _ = oracle.icl_attention_rows(q, k_same, v, rows)
    assert np.max(np.abs(A - vf.mean(axis=2, keepdims=True))) < 1e-12
    # zero queries -> uniform average as well
    A, _, _ = oracle.icl_attention_rows(np.zeros_like(q), f32_to_bf16_bits(
        rng.standard_normal((B, H, N, d)).astype(np.float32)), v, rows)
    assert np.max(np.abs(A - vf.mean(axis=2, keepdims=True))) < 1e-12
    # a single key -> its value row
    A, _, _ = oracle.icl_attention_rows(q, k_same[:, :, :1], v[:, :, :1], rows)
    assert np.max(np.abs(A - vf[:, :, :1])) == 0
    # very large softmax scale -> value row of the best-matching key
    k = f32_to_bf16_bits(rng.standard_normal((B, H, N, d)).astype(np.float32))
    A, _, _ = oracle.icl_attention_rows(q, k, v, rows, alpha=1e4)
    qf, kf = bf16_bits_to_f64(q), bf16_bits_to_f64(k)
    for h in range(H):
        best = np.argmax(qf[0, h] @ kf[0, h].T, axis=1)
        assert np.max(np.abs(A[0, h] - vf[0, h][best])) < 1e-9


def test_key_shift_invariance_on_exact_inputs():
    # softmax is invariant to adding a constant vector c to every key
    # (q.(k+c) = q.k + q.c shifts every score of the row equally)
    rng = np.random.default_rng(5)
    B, H, N, d = 1, 1, 50, 64
    k = rng.integers(-4, 5, (B, H, N, d)).astype(np.float32)
    q = rng.integers(-2, 3, (B, H, 9, d)).astype(np.float32)
    v = rng.standard_normal((B, H, N, d)).astype(np.float32)
    rows = np.arange(9)
    A0, _, _ = oracle.icl_attention_rows(f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v), rows)
    A1, _, _ = oracle.icl_attention_rows(f32_to_bf16_bits(q), f32_to_bf16_bits(k + 3.0), f32_to_bf16_bits(v), rows)
    assert np.max(np.abs(A0 - A1)) < 1e-12


def test_icl_structure_batch_invariance_and_shared_kv():
    w, g, z = quantized_c1()
    kw = dict(sq=z["sq"], sk=z["sk"], sv=z["sv"])
    full, _, _ = oracle.icl_attention_rows(z["t8"], z["k8"], z["v8"], np.arange(w.n_test), **kw)
    # a test row's output does not depend on which other test rows are present
    one = z["t8"][:, :, 7:8]
    single, _, _ = oracle.icl_attention_rows(one, z["k8"], z["v8"], np.arange(1), **kw)
    assert np.array_equal(single[:, :, 0], full[:, :, 7])
    perm = np.random.default_rng(0).permutation(w.n_test)
    shuffled, _, _ = oracle.icl_attention_rows(z["t8"][:, :, perm], z["k8"], z["v8"],
                                               np.arange(w.n_test), **kw)
    assert np.array_equal(shuffled, full[:, :, perm])
    # a test query equal to a train query gets the same output: both calls read the same K8/V8
    t8 = z["t8"].copy(); t8[:, :, 3] = z["q8"][:, :, 11]
    a_test, _, _ = oracle.icl_attention_rows(t8, z["k8"], z["v8"], np.array([3]), **kw)
    a_train, _, _ = oracle.icl_attention_rows(z["q8"], z["k8"], z["v8"], np.array([11]), **kw)
    assert np.array_equal(a_test, a_train)


def test_lifted_row_maximum_is_256():
    # Method section: the row maximum of P is lifted to 2^8 = 256 (< 448)
    w, g, z = quantized_c1()
    for row in range(0, w.n_train, 17):
        p8 = oracle.lifted_p8_row(z["q8"], z["k8"], bh=0, row=row, sq=z["sq"][0, 0], sk=z["sk"][0, 0])
        assert p8.max() == 0x78 and oracle.e4m3_decode(int(p8.max())) == 256.0
        assert np.all(p8 < 0x80)


def online_p8_emulation(qh, k8f, v8f, c, tile):
    """Independent numpy/torch emulation of the method's online softmax with an
    e4m3 P tile lifted against the RUNNING maximum (fp32 state), one row block."""
    x = (c * (qh @ k8f.T)).astype(np.float32)
    n = x.shape[1]
    m = np.full((x.shape[0], 1), -np.inf, dtype=np.float32)
    l = np.zeros((x.shape[0], 1), dtype=np.float32)
    acc = np.zeros((x.shape[0], v8f.shape[1]), dtype=np.float64)
    for j in range(0, n, tile):
        xs = x[:, j:j + tile]
        mn = np.maximum(m, xs.max(axis=1, keepdims=True))
        corr = np.exp2(m - mn)
        p = np.exp2(xs - mn + np.float32(8.0)).astype(np.float32)
        p8 = torch.from_numpy(p).to(torch.float8_e4m3fn).to(torch.float64).numpy()
        l = l * corr + p.sum(axis=1, keepdims=True)
        acc = acc * corr + p8 @ v8f[j:j + tile]
        m = mn
    return acc / l


@pytest.mark.parametrize("tile", [32, 128])
def test_p_quantization_bound_holds_and_faithful_mode_is_close(tile):
    w, g, z = quantized_c1(n_train=300, n_test=33)
    tab = oracle.e4m3_decode_table()
    kw = dict(sq=z["sq"], sk=z["sk"], sv=z["sv"])
    rows = np.arange(w.n_test)
    A, Abs, Bnd = oracle.icl_attention_rows(z["t8"], z["k8"], z["v8"], rows, **kw)
    O4 = oracle.icl_attention_rows(z["t8"], z["k8"], z["v8"], rows, mode="p8", **kw)
    assert np.all(Bnd >= 0) and np.all(Bnd <= Abs * (1 + 1e-12))
    # two-pass e4m3-P result (bf16-rounded) stays inside bound + bf16 half-ulp
    assert np.all(np.abs(O4 - A) <= Bnd + 2.0 ** -8 * np.abs(A) + 1e-9)
    assert np.mean(np.abs(O4 - A) / np.maximum(1, Abs)) < 2e-3
    # online emulation with a running maximum also stays inside the bound
    alpha = 1 / np.sqrt(w.d)
    for h in range(w.H):
        c = alpha * float(z["sq"][0, h]) * float(z["sk"][0, h]) * np.log2(np.e)
        O = online_p8_emulation(tab[z["t8"][0, h]], tab[z["k8"][0, h]], tab[z["v8"][0, h]], c, tile)
        O = O * float(z["sv"][0, h])
        assert np.all(np.abs(O - A[0, h]) <= 1.02 * Bnd[0, h] + 1e-4 * Abs[0, h] + 1e-9)
