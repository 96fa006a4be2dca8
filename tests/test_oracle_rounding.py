"""Pins for the oracle's rounding helpers that feed the parity criteria:

* the e4m3 rounding envelope behind the per-element bound ``Bnd`` (a bound that is valid
  AND tight: a looser envelope fails here),
* the two bf16 roundings (fp32 -> bf16 for the e4m3-P mode's output, fp64 -> bf16 for the
  perturbation), against torch's CPU cast on ties, neighbours and random values,
* the e4m3 encoder against a second third party: the host-side conversion of the CUDA
  toolkit's cuda_fp8.h, compiled with nvcc and run on the CPU.
"""
import os
import shutil
import subprocess
import struct

import numpy as np
import pytest
import torch

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def actual_rounding_error(x):
    return abs(x - oracle.e4m3_decode(oracle.e4m3_encode(x)))


def test_rounding_envelope_is_a_bound_everywhere():
    # dense grid over (0, 448]: geometric (every binade, subnormal range and flush range
    # included) plus every midpoint between neighbouring grid values and its neighbours
    xs = list(np.exp(np.linspace(np.log(2.0 ** -14), np.log(448.0), 20000)))
    grid = sorted(v for v in oracle.e4m3_decode_table() if v == v and v >= 0)
    for a, b in zip(grid[:-1], grid[1:]):
        mid = 0.5 * (a + b)
        xs += [mid, np.nextafter(mid, 0.0), np.nextafter(mid, 1e9), a, b]
    for x in xs:
        if 0.0 < x <= 448.0:
            assert oracle.rounding_envelope(x) >= actual_rounding_error(x) - 1e-300, x


def test_rounding_envelope_is_tight():
    # at the midpoint just above a power of two (17 between 16 and 18, 34, 272, ...) the
    # actual error is 2^-4 * 2^e; the envelope 2^-4 * x exceeds it by the factor 17/16 only.
    # An envelope of 2^-3 x (or any slack beyond 7 %) fails here.
    for e in range(-6, 9):
        x = 2.0 ** e * (1 + 1 / 16)
        if x > 448:
            continue
        err = actual_rounding_error(x)
        assert err == pytest.approx(2.0 ** e / 16)
        assert oracle.rounding_envelope(x) <= 1.07 * err, (x, oracle.rounding_envelope(x), err)
    # subnormal range: half the spacing 2^-9, exactly
    for k in range(1, 8):
        x = (k + 0.5) * 2.0 ** -9
        assert oracle.rounding_envelope(x) == pytest.approx(actual_rounding_error(x))
    # flush range: a value below 2^-10 rounds to zero, the envelope is the value itself
    for x in (2.0 ** -10 * 0.999, 2.0 ** -12, 1e-9):
        assert oracle.rounding_envelope(x) == pytest.approx(x) and actual_rounding_error(x) == pytest.approx(x)


def _bf16_cases():
    rng = np.random.default_rng(7)
    base = rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-20, 20, 4000).astype(np.float32)
    bits = base.view(np.uint32) & np.uint32(0xFFFF0000)
    lo = bits.view(np.float32)
    hi = (bits + np.uint32(0x10000)).view(np.float32)
    tie = ((lo.astype(np.float64) + hi.astype(np.float64)) / 2)       # exact ties (fp32-representable)
    cases = [base.astype(np.float64), lo.astype(np.float64), tie,
             np.nextafter(tie.astype(np.float32), np.float32(np.inf)).astype(np.float64),
             np.nextafter(tie.astype(np.float32), np.float32(-np.inf)).astype(np.float64)]
    return np.concatenate(cases + [np.array([0.0, -0.0, 1.0, -1.0, 3.3895313892515355e38, 1e-40])])


def test_round_to_bf16_matches_torch_cast():
    x = _bf16_cases().astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.round_to_bf16(float(v)) for v in x], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    # a truncating implementation fails on the ties and the values above them
    trunc = (x.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
    assert not np.array_equal(trunc.view(np.uint32), ref.view(np.uint32))


def test_double_to_bf16_bits_matches_torch_cast():
    x = _bf16_cases()
    x = x[np.abs(x) < 3.38e38]
    # fp64 inputs that are exactly fp32-representable: torch's fp32 -> bf16 cast is the reference
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.double_to_bf16_bits(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, ref)
    # fp64 values strictly between an exact tie and its neighbour round to the nearer side,
    # where a detour through fp32 would land on the tie and then on the even side
    lo, hi = 1.0, 1.0 + 2.0 ** -7
    tie = 0.5 * (lo + hi)
    assert oracle.double_to_bf16_bits(tie + 1e-12) == 0x3F81
    assert oracle.double_to_bf16_bits(tie - 1e-12) == 0x3F80
    assert oracle.double_to_bf16_bits(tie) == 0x3F80            # tie to even


CUDA_FP8_CHECK = r"""
#include <cuda_fp8.h>
#include <cstdio>
#include <cstdlib>
int main(int argc, char** argv) {
    // reads fp32 values (hex bit patterns) on stdin, prints the e4m3 code of each as the
    // toolkit's host-side conversion gives it (saturating, round to nearest even)
    unsigned u;
    while (scanf("%x", &u) == 1) {
        float f; __builtin_memcpy(&f, &u, 4);
        __nv_fp8_storage_t c = __nv_cvt_float_to_fp8(f, __NV_SATFINITE, __NV_E4M3);
        printf("%02x\n", (unsigned)c);
    }
    return 0;
}
"""


@pytest.mark.skipif(shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"),
                    reason="needs the CUDA toolkit's nvcc for the host-side cuda_fp8.h conversion")
def test_encode_matches_cuda_fp8_host_conversion(tmp_path):
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    src = tmp_path / "cvt.cu"
    src.write_text(CUDA_FP8_CHECK)
    exe = tmp_path / "cvt"
    subprocess.run([nvcc, "-O1", "-o", str(exe), str(src)], check=True, capture_output=True, timeout=300)
    rng = np.random.default_rng(3)
    vals = [rng.standard_normal(20000).astype(np.float32) * np.float32(100.0),
            (rng.standard_normal(20000).astype(np.float32) * np.float32(2.0) ** rng.integers(-12, 9, 20000).astype(np.float32))]
    grid = np.array(sorted(v for v in oracle.e4m3_decode_table() if v == v and v >= 0), dtype=np.float64)
    mids = (0.5 * (grid[:-1] + grid[1:])).astype(np.float32)      # every tie point is fp32-exact
    vals += [mids, -mids, np.nextafter(mids, np.float32(np.inf)), np.nextafter(mids, np.float32(-np.inf)),
             np.array([0.0, -0.0, 448.0, -448.0, 464.0, 1e9, -1e9, 2.0 ** -10, 2.0 ** -11], dtype=np.float32)]
    x = np.concatenate(vals).astype(np.float32)
    text = "\n".join(f"{b:08x}" for b in x.view(np.uint32)) + "\n"
    out = subprocess.run([str(exe)], input=text, check=True, capture_output=True, text=True, timeout=120).stdout
    theirs = np.array([int(t, 16) for t in out.split()], dtype=np.uint8)
    clipped = np.clip(x, -448.0, 448.0)                            # Eq. 2 clamps, the oracle's encoder takes |y| <= 448
    ours = oracle.e4m3_encode_array(clipped)
    assert theirs.size == x.size
    assert np.array_equal(ours, theirs), np.flatnonzero(ours != theirs)[:10]
