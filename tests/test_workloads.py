"""The seeded input generator: determinism, slicing, and the structure each
configuration names."""
import numpy as np

from helpers import bf16_bits_to_f64
from paper_2609_13031_b200 import workloads as W


def test_deterministic_and_thread_count_independent():
    w = W.CONFIGS["C2"].scaled(300, 70)
    a = W.generate(w, nthreads=1)
    b = W.generate(w, nthreads=7)
    for k in a:
        assert np.array_equal(a[k], b[k])
    # a prefix of rows is a pure function of (seed, tensor, b, h, row, col)
    c = W.generate(w.scaled(100, 70))
    assert np.array_equal(c["k"], a["k"][:, :, :100])
    assert not np.array_equal(a["q_train"], a["k"])


def test_shapes_of_the_five_configurations():
    expect = {"C1": (1, 2, 64, 512, 128), "C2": (1, 8, 64, 8192, 2048),
              "C3": (1, 8, 128, 65536, 16384), "C4": (4, 4, 64, 262144, 65536),
              "C5": (1, 8, 64, 1048576, 131072)}
    for name, (B, H, d, N, M) in expect.items():
        w = W.CONFIGS[name]
        assert (w.B, w.H, w.d, w.n_train, w.n_test) == (B, H, d, N, M)
        assert w.flops == 4.0 * B * H * d * N * (N + M)


def test_standard_normal_statistics():
    g = W.generate(W.CONFIGS["C1"].scaled(8192, 128))
    x = bf16_bits_to_f64(g["v"])
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1) < 0.01
    assert abs(np.mean(x ** 4) - 3) < 0.1


def test_outlier_channels_row_gains_and_key_shift():
    w = W.CONFIGS["C2"].scaled(2048, 2048)
    g = W.generate(w)
    for bh in range(w.H):
        mask = W.outlier_mask(w, bh)
        assert mask.sum() == 4
        for name in ("q_train", "k", "v", "q_test"):
            std = bf16_bits_to_f64(g[name])[0, bh].std(axis=0)
            assert np.all(np.abs(std[mask] - 20) < 4) and np.all(np.abs(std[~mask] - 1) < 0.25)
    w = W.CONFIGS["C3"].scaled(4096, 64)
    x = bf16_bits_to_f64(W.generate(w)["k"])
    log_norm = np.log(np.sqrt((x ** 2).mean(axis=3)))
    assert abs(log_norm.std() - 0.5) < 0.05 and abs(log_norm.mean()) < 0.05
    w = W.CONFIGS["C4"].scaled(1024, 64)
    g = W.generate(w)
    assert abs(bf16_bits_to_f64(g["k"]).mean() - 3.0) < 0.02
    assert abs(bf16_bits_to_f64(g["v"]).mean()) < 0.02
