"""The allocation-free quantizer entry point against the regular one.

fp8attn_quantize_noalloc is for hosts that can pass only inputs and outputs and
may not allocate device memory (no workspace argument in their plugin interface,
or a memory pool that already owns the GPU).  Its scratch is a fixed array inside
the library that every call shares and that keeps the previous call's contents,
so the check runs two different tensors back to back: stale maxima left by the
first call would corrupt the scales of the second.  Results must equal the
regular entry point's bit for bit, which is the bar all quantizer tests use, and
they are compared with the CPU oracle directly as well.

This file is named to be collected last; it also passes when run on its own.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row():
    w = W.CONFIGS["C2"].scaled(3000, 500)      # 8 heads, outlier channels: large, distinct maxima
    g = W.generate(w)
    big = to_dev(g["k"])
    small = (to_dev(g["v"]).float() * 0.01).to(torch.bfloat16)   # far smaller maxima than `big`
    q_test = to_dev(g["q_test"])
    ws = api.new_workspace(w.B, w.H)
    ref_big, ref_big_s = api.quantize(big, ws)
    ref_small, ref_small_s = api.quantize(small, ws)
    ref_test, _ = api.quantize(q_test, ws, scale_in=ref_big_s)

    out = torch.empty_like(ref_big)
    scale = torch.empty_like(ref_big_s)
    out2 = torch.empty_like(ref_small)
    scale2 = torch.empty_like(ref_small_s)
    out3 = torch.empty_like(ref_test)
    scale3 = torch.empty_like(ref_big_s)
    # two calls in a row on one stream, large maxima first
    api.quantize_noalloc(big, out, scale)
    api.quantize_noalloc(small, out2, scale2)
    api.quantize_noalloc(q_test, out3, scale3, scale_in=scale)
    torch.cuda.synchronize()
    assert torch.equal(scale, ref_big_s) and torch.equal(out, ref_big)
    assert torch.equal(scale2, ref_small_s) and torch.equal(out2, ref_small)
    assert torch.equal(scale3, ref_big_s) and torch.equal(out3, ref_test)
    # the oracle itself, not only the other GPU entry point
    small_bits = small.view(torch.int16).cpu().numpy().view(np.uint16)
    for got, got_s, bits, s_in in ((out, scale, g["k"], None), (out2, scale2, small_bits, None),
                                   (out3, scale3, g["q_test"], scale.cpu().numpy())):
        want, want_s = oracle.quantize(bits, scale_in=s_in)
        assert np.array_equal(got.cpu().numpy(), want) and np.array_equal(got_s.cpu().numpy(), want_s)
    # and once more in the opposite order
    api.quantize_noalloc(small, out2, scale2)
    api.quantize_noalloc(big, out, scale)
    torch.cuda.synchronize()
    assert torch.equal(scale, ref_big_s) and torch.equal(out, ref_big)
    assert torch.equal(scale2, ref_small_s) and torch.equal(out2, ref_small)


def test_noalloc_rejects_more_heads_than_its_scratch_holds():
    lib = api.load()
    x = torch.zeros((1, 1, 1, 64), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros((1, 1, 1, 64), dtype=torch.uint8, device="cuda")
    s = torch.zeros((1, 1), dtype=torch.float32, device="cuda")
    too_many = api.NOALLOC_MAX_HEADS + 1
    rc = lib.fp8attn_quantize_noalloc(x.data_ptr(), 1, too_many, 1, 64, None, o.data_ptr(), s.data_ptr(), None)
    assert rc == api.ERR_TOO_LARGE
    assert "scratch" in api.status_string(rc)
    rc = lib.fp8attn_quantize_noalloc(x.data_ptr(), 1, 1, 1, 96, None, o.data_ptr(), s.data_ptr(), None)
    assert rc == api.ERR_UNSUPPORTED
