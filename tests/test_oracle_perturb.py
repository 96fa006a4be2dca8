"""Pins for the oracle's Gaussian perturbation (appendix Eq. 3): closed forms and the
statistics the equation fixes."""
import numpy as np

import oracle
from helpers import bf16_bits_to_f64, f32_to_bf16_bits
from paper_2609_13031_b200 import workloads as W


def test_zero_strength_is_identity_and_rho_is_the_head_rms():
    g = W.generate(W.CONFIGS["C4"].scaled(256, 0))
    x = g["k"]                                   # mean 3: RMS is not the standard deviation
    out, rho = oracle.perturb(x, 0.0, seed=1, stream_id=0)
    assert np.array_equal(out, x)
    xf = bf16_bits_to_f64(x)
    assert np.allclose(rho, np.sqrt((xf ** 2).mean(axis=(2, 3))), rtol=1e-12)
    const = f32_to_bf16_bits(np.full((1, 2, 8, 64), 2.0, dtype=np.float32))
    _, rho = oracle.perturb(const, 0.5, 3, 0)
    assert np.all(rho == 2.0)


def test_noise_is_standard_normal_scaled_by_epsilon_rho_per_head():
    # heads whose entries differ by orders of magnitude are perturbed equally in relative terms
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 3, 4096, 64)).astype(np.float32)
    x[0, 1] *= 1000.0
    x[0, 2] *= 0.001
    bits = f32_to_bf16_bits(x)
    eps = 5 * 0.0265                             # the paper's largest strength
    out, rho = oracle.perturb(bits, eps, seed=7, stream_id=2)
    noise = (bf16_bits_to_f64(out) - bf16_bits_to_f64(bits)) / (eps * rho[:, :, None, None])
    for h in range(3):
        z = noise[0, h].ravel()
        assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.02      # bf16 rounding adds ~1e-2 noise
        assert abs(np.mean(z ** 4) - 3) < 0.15
    # independent across heads, neighbouring elements and streams
    assert abs(np.corrcoef(noise[0, 0].ravel(), noise[0, 1].ravel())[0, 1]) < 0.01
    assert abs(np.corrcoef(noise[0, 0, :, 0::2].ravel(), noise[0, 0, :, 1::2].ravel())[0, 1]) < 0.01
    other, _ = oracle.perturb(bits, eps, seed=7, stream_id=3)
    n2 = (bf16_bits_to_f64(other) - bf16_bits_to_f64(bits)) / (eps * rho[:, :, None, None])
    assert abs(np.corrcoef(noise[0, 0].ravel(), n2[0, 0].ravel())[0, 1]) < 0.01


def test_reproducible_and_linear_in_epsilon():
    g = W.generate(W.CONFIGS["C1"].scaled(128, 0))
    a, _ = oracle.perturb(g["v"], 0.0265, 11, 5, nthreads=1)
    b, _ = oracle.perturb(g["v"], 0.0265, 11, 5, nthreads=4)
    assert np.array_equal(a, b)
    c, _ = oracle.perturb(g["v"], 0.0265, 12, 5)
    assert not np.array_equal(a, c)
    # the field z does not depend on epsilon: doubling epsilon doubles the displacement
    big, rho = oracle.perturb(g["v"], 2.0, 11, 5)
    bigger, _ = oracle.perturb(g["v"], 4.0, 11, 5)
    x = bf16_bits_to_f64(g["v"])
    d1, d2 = bf16_bits_to_f64(big) - x, bf16_bits_to_f64(bigger) - x
    assert np.max(np.abs(d2 - 2 * d1)) < 0.1     # up to bf16 rounding of values of size ~10
