"""The three-tile kernels (d = 64, launches of at least eight rounds of 384-row blocks): both
data types, fp16 tensors, the forward flags and ragged sizes, on a shape that is large in heads
rather than in rows so that the oracle can follow.  The named workloads C4 and C5 take this
path at full size in test_gpu_attention.py (FP8 only)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from helpers import Guarded, bf16_bits_to_f64, check_bf16_attention, check_fp8_attention, sample_rows
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu

# 64 heads x (16 + 3) blocks of 384 rows = 1216 CTAs >= 8 x 148; rows are not multiples of 128
SHAPE = dict(B=4, H=16, n_train=6100, n_test=1001)


def workload(cfg="C2", **kw):
    return dataclasses.replace(W.CONFIGS[cfg], **{**SHAPE, **kw})


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def head0(x, H):
    """K / V (or their scales) of head 0 of each table, broadcast over the table's heads."""
    return np.ascontiguousarray(np.broadcast_to(x[:, :1], x.shape))


@pytest.mark.parametrize("half,gqa,test_only", [(False, False, False), (True, True, False), (False, True, True)])
def test_fp8_three_tile_launch(half, gqa, test_only):
    w = workload()
    flags = (api.TEST_ROWS_USE_KV_HEAD0 if gqa else 0) | (api.TEST_ROWS_ONLY if test_only else 0)
    assert api.attention_rows_per_cta(w.B, w.H, w.n_train, w.n_test, w.d, flags) == (384 if not test_only else 256)
    if test_only:
        # the test call alone has too few blocks for three tiles here: make it wide enough
        w = workload(n_test=8000)
        assert api.attention_rows_per_cta(w.B, w.H, w.n_train, w.n_test, w.d, flags) == 384
    g = W.generate(w)
    if half:
        g = {k: np.ascontiguousarray(bf16_bits_to_f64(v).astype(np.float16)).view(np.uint16) for k, v in g.items()}
    dtype16 = "fp16" if half else "bf16"
    tdt = torch.float16 if half else torch.bfloat16
    q8, sq = oracle.quantize(g["q_train"], dtype16=dtype16)
    k8, sk = oracle.quantize(g["k"], dtype16=dtype16)
    v8, sv = oracle.quantize(g["v"], dtype16=dtype16)
    t8, _ = oracle.quantize(g["q_test"], scale_in=sq, dtype16=dtype16)
    dev = lambda a: torch.from_numpy(a).cuda()
    ws = api.new_workspace(w.B, w.H)
    g_tr = Guarded((w.B, w.H, w.n_train, w.d), tdt)
    g_te = Guarded((w.B, w.H, w.n_test, w.d), tdt)
    before = api.launch_count()
    o_tr, o_te = api.icl_forward_fp8(None if test_only else dev(q8), dev(t8), dev(k8), dev(v8), dev(sq), dev(sk),
                                     dev(sv), ws, flags=flags, out_train=None if test_only else g_tr.t,
                                     out_test=g_te.t)
    assert api.launch_count() - before == 1
    assert api.last_device_status(ws) == (0, 0)
    g_tr.check("three tiles out_train")
    g_te.check("three tiles out_test")
    for name, out, q, nq in (("train", o_tr, q8, w.n_train), ("test", o_te, t8, w.n_test)):
        if name == "train" and test_only:
            assert out is None
            continue
        assert out.dtype == tdt
        kv0 = gqa and name == "test"
        kk, vv, ssk, ssv = (head0(k8, w.H), head0(v8, w.H), head0(sk, w.H), head0(sv, w.H)) if kv0 else (k8, v8, sk, sv)
        # the ragged last block of a head (one or two of its three tiles in use) and a stratified sample
        rows = np.unique(np.concatenate([sample_rows(nq, 12, 7), np.arange(max(0, nq - 400), nq, 37)]))
        A, Abs, Bnd = oracle.icl_attention_rows(q, kk, vv, rows, sq=sq, sk=ssk, sv=ssv)
        check_fp8_attention(f64(out[:, :, torch.from_numpy(rows).cuda()]), A, Abs, Bnd, diffuse=False,
                            label=f"three tiles fp8 half={half} gqa={gqa} test_only={test_only}/{name}",
                            named_config=False)


@pytest.mark.parametrize("half", [False, True])
def test_16bit_three_tile_launch(half):
    w = workload(cfg="C4")
    assert api.attention_rows_per_cta(w.B, w.H, w.n_train, w.n_test, w.d) == 384
    g = W.generate(w)
    if half:
        g = {k: np.ascontiguousarray(bf16_bits_to_f64(v).astype(np.float16)).view(np.uint16) for k, v in g.items()}
    tdt = torch.float16 if half else torch.bfloat16
    x = {k: torch.from_numpy(v.view(np.int16)).cuda().view(tdt) for k, v in g.items()}
    ws = api.new_workspace(w.B, w.H)
    o_tr, o_te = api.icl_forward_bf16(x["q_train"], x["q_test"], x["k"], x["v"], ws)
    assert api.last_device_status(ws) == (0, 0)
    for name, out, q, nq in (("train", o_tr, g["q_train"], w.n_train), ("test", o_te, g["q_test"], w.n_test)):
        rows = np.unique(np.concatenate([sample_rows(nq, 12, 9), np.arange(max(0, nq - 400), nq, 37)]))
        A, Abs, _ = oracle.icl_attention_rows(q, g["k"], g["v"], rows, dtype16="fp16" if half else "bf16")
        check_bf16_attention(f64(out[:, :, torch.from_numpy(rows).cuda()]), A, Abs,
                             label=f"three tiles 16-bit half={half}/{name}",
                             rounding=2.0 ** -12 if half else 2.0 ** -9)


def test_tile_count_follows_the_launch_size():
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    # just below and at eight rounds of 384-row blocks (one head, train rows only)
    blocks = 8 * sms
    assert api.attention_rows_per_cta(1, 1, 384 * blocks, 0, 64) == 384
    assert api.attention_rows_per_cta(1, 1, 384 * (blocks - 1), 0, 64) == 256
    assert api.attention_rows_per_cta(1, 1, 384 * blocks, 0, 128) == 256
    assert api.attention_rows_per_cta(1, 1, 384 * blocks, 0, 64, api.TEST_ROWS_ONLY) == 256
