"""Variant switches of the attention call: the test->train call alone
(FP8ATTN_TEST_ROWS_ONLY) with the precision-ablation arms it makes possible, and
IEEE fp16 tensors instead of bf16 (FP8ATTN_INPUT_FP16 / FP8ATTN_IO_FP16)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f64, check_bf16_attention, check_fp8_attention
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def fp16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.float16)


def to_fp16_bits(bf16_bits):
    """The workload's values rounded to IEEE fp16, as bit patterns."""
    return np.ascontiguousarray(bf16_bits_to_f64(bf16_bits).astype(np.float16)).view(np.uint16)


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def quantized(g, dtype16="bf16"):
    q8, sq = oracle.quantize(g["q_train"], dtype16=dtype16)
    k8, sk = oracle.quantize(g["k"], dtype16=dtype16)
    v8, sv = oracle.quantize(g["v"], dtype16=dtype16)
    t8, _ = oracle.quantize(g["q_test"], scale_in=sq, dtype16=dtype16)
    return q8, t8, k8, v8, sq, sk, sv


# ---- the test->train call alone, and the ablation arms -------------------------------

@pytest.mark.parametrize("cfg,n,m", [("C1", 512, 128), ("C3", 700, 300), ("C4", 520, 257)])
def test_test_rows_only_matches_the_combined_call(cfg, n, m):
    w = W.CONFIGS[cfg].scaled(n, m)
    g = W.generate(w)
    dev = lambda a: torch.from_numpy(a).cuda()
    q8, t8, k8, v8, sq, sk, sv = (dev(a) for a in quantized(g))
    ws = api.new_workspace(w.B, w.H)
    _, both_te = api.icl_forward_fp8(q8, t8, k8, v8, sq, sk, sv, ws)
    none_tr, only_te = api.icl_forward_fp8(None, t8, k8, v8, sq, sk, sv, ws, flags=api.TEST_ROWS_ONLY)
    assert none_tr is None and torch.equal(only_te, both_te)
    x = {k: bf16_dev(g[k]) for k in ("q_train", "q_test", "k", "v")}
    _, both_te = api.icl_forward_bf16(x["q_train"], x["q_test"], x["k"], x["v"], ws)
    none_tr, only_te = api.icl_forward_bf16(None, x["q_test"], x["k"], x["v"], ws, flags=api.TEST_ROWS_ONLY)
    assert none_tr is None and torch.equal(only_te, both_te)
    # with the grouped-query flag as well
    _, both_te = api.icl_forward_fp8(q8, t8, k8, v8, sq, sk, sv, ws, flags=api.TEST_ROWS_USE_KV_HEAD0)
    _, only_te = api.icl_forward_fp8(None, t8, k8, v8, sq, sk, sv, ws,
                                     flags=api.TEST_ROWS_ONLY | api.TEST_ROWS_USE_KV_HEAD0)
    assert torch.equal(only_te, both_te)
    assert api.last_device_status(ws) == (0, 0)


def test_test_rows_only_argument_checks():
    lib = api.load()
    ws = api.new_workspace(1, 1)
    q = torch.zeros((1, 1, 8, 64), dtype=torch.uint8, device="cuda")
    o = torch.zeros((1, 1, 8, 64), dtype=torch.bfloat16, device="cuda")
    s = torch.ones((1, 1), dtype=torch.float32, device="cuda")
    p = lambda t: t.data_ptr()
    # no test rows to run
    rc = lib.fp8attn_icl_forward_ex(None, None, p(q), p(q), p(s), p(s), p(s), 1, 1, 8, 0, 64, 0.0,
                                    api.TEST_ROWS_ONLY, None, None, p(ws), ws.numel(), None)
    assert rc == api.ERR_INVALID_ARG
    # the plain call still needs its train queries
    rc = lib.fp8attn_icl_forward_ex(None, p(q), p(q), p(q), p(s), p(s), p(s), 1, 1, 8, 8, 64, 0.0,
                                    0, None, p(o), p(ws), ws.numel(), None)
    assert rc == api.ERR_INVALID_ARG


def test_precision_ablation_arms():
    """FP8 in one call and 16 bits in the other: each half is, bit for bit, what the
    all-FP8 and the all-16-bit runs give for those rows."""
    w = W.CONFIGS["C2"].scaled(900, 260)
    g = W.generate(w)
    x = {k: bf16_dev(g[k]) for k in ("q_train", "q_test", "k", "v")}
    args = (x["q_train"], x["q_test"], x["k"], x["v"])
    ws = api.new_workspace(w.B, w.H)
    f_tr, f_te = api.icl_attention_arms(*args, True, True, ws)
    b_tr, b_te = api.icl_attention_arms(*args, False, False, ws)
    tr, te = api.icl_attention_arms(*args, True, False, ws)
    assert torch.equal(tr, f_tr) and torch.equal(te, b_te)
    tr, te = api.icl_attention_arms(*args, False, True, ws)
    assert torch.equal(tr, b_tr) and torch.equal(te, f_te)
    assert not torch.equal(f_te, b_te)
    assert api.last_device_status(ws) == (0, 0)


# ---- IEEE fp16 tensors -----------------------------------------------------------

@pytest.mark.parametrize("cfg,n,m", [("C1", 512, 128), ("C2", 1031, 77), ("C4", 300, 48)])
def test_quantize_fp16_input_is_bit_exact(cfg, n, m):
    w = W.CONFIGS[cfg].scaled(n, m)
    g = {k: to_fp16_bits(v) for k, v in W.generate(w).items()}
    ws = api.new_workspace(w.B, w.H)
    ref = quantized(g, "fp16")
    # one tensor at a time ...
    q8, sq = api.quantize(fp16_dev(g["q_train"]), ws)
    t8, st = api.quantize(fp16_dev(g["q_test"]), ws, scale_in=sq)
    assert np.array_equal(q8.cpu().numpy(), ref[0]) and np.array_equal(sq.cpu().numpy(), ref[4])
    assert np.array_equal(t8.cpu().numpy(), ref[1]) and np.array_equal(st.cpu().numpy(), ref[4])
    # ... and all four in one call
    o = api.quantize_qkv(fp16_dev(g["q_train"]), fp16_dev(g["k"]), fp16_dev(g["v"]), fp16_dev(g["q_test"]), ws)
    for name, r in zip(("q8", "t8", "k8", "v8", "sq", "sk", "sv"), ref):
        assert np.array_equal(o[name].cpu().numpy(), r), name
    assert api.last_device_status(ws) == (0, 0)


def test_quantize_fp16_subnormals_and_extremes():
    """fp16 subnormals, the largest finite fp16 and signed zeros go through exactly."""
    rng = np.random.default_rng(5)
    bits = rng.integers(0, 0x0400, size=(1, 2, 40, 64), dtype=np.uint16)     # subnormals and zero
    bits |= (rng.integers(0, 2, size=bits.shape, dtype=np.uint16) << 15)
    ws = api.new_workspace(1, 2)
    got, s = api.quantize(fp16_dev(bits), ws)
    ref, rs = oracle.quantize(bits, dtype16="fp16")
    assert np.array_equal(got.cpu().numpy(), ref) and np.array_equal(s.cpu().numpy(), rs)
    bits[0, 0, 3, 5] = 0x7BFF                                                # 65504
    bits[0, 1, 7, 9] = 0xFBFF
    got, s = api.quantize(fp16_dev(bits), ws)
    ref, rs = oracle.quantize(bits, dtype16="fp16")
    assert np.array_equal(got.cpu().numpy(), ref) and np.array_equal(s.cpu().numpy(), rs)
    assert got.cpu().numpy()[0, 0, 3, 5] == 0x7E and got.cpu().numpy()[0, 1, 7, 9] == 0xFE


@pytest.mark.parametrize("cfg,n,m", [("C1", 512, 128), ("C3", 777, 130)])
def test_fp8_attention_fp16_output(cfg, n, m):
    w = W.CONFIGS[cfg].scaled(n, m)
    g = W.generate(w)
    ref = quantized(g)
    dev = lambda a: torch.from_numpy(a).cuda()
    ws = api.new_workspace(w.B, w.H)
    h_tr, h_te = api.icl_forward_fp8(*(dev(a) for a in ref), ws, out_dtype=torch.float16)
    b_tr, b_te = api.icl_forward_fp8(*(dev(a) for a in ref), ws)
    assert h_tr.dtype == torch.float16 and h_te.dtype == torch.float16
    assert api.last_device_status(ws) == (0, 0)
    q8, t8, k8, v8, sq, sk, sv = ref
    for out, other, q, rows in ((h_tr, b_tr, q8, w.n_train), (h_te, b_te, t8, w.n_test)):
        A, Abs, Bnd = oracle.icl_attention_rows(q, k8, v8, np.arange(rows), sq=sq, sk=sk, sv=sv)
        check_fp8_attention(f64(out), A, Abs, Bnd, diffuse=(cfg == "C1"), label=f"{cfg}/fp16-out",
                            named_config=False)
        # the same fp32 result, rounded to fp16 here and to bf16 there
        o16, o_b = f64(out), f64(other)
        assert np.all(np.abs(o16 - o_b) <= 2.0 ** -8 * np.abs(o16) + 2.0 ** -24)


@pytest.mark.parametrize("cfg,n,m", [("C1", 512, 128), ("C3", 300, 129), ("C4", 600, 200)])
def test_fp16_attention_twin(cfg, n, m):
    w = W.CONFIGS[cfg].scaled(n, m)
    g = {k: to_fp16_bits(v) for k, v in W.generate(w).items()}
    ws = api.new_workspace(w.B, w.H)
    o_tr, o_te = api.icl_forward_bf16(fp16_dev(g["q_train"]), fp16_dev(g["q_test"]), fp16_dev(g["k"]),
                                      fp16_dev(g["v"]), ws)
    assert o_tr.dtype == torch.float16 and api.last_device_status(ws) == (0, 0)
    for out, q, rows in ((o_tr, g["q_train"], w.n_train), (o_te, g["q_test"], w.n_test)):
        A, Abs, _ = oracle.icl_attention_rows(q, g["k"], g["v"], np.arange(rows), dtype16="fp16")
        check_bf16_attention(f64(out), A, Abs, label=f"{cfg}/fp16-twin", rounding=2.0 ** -12)


def test_fp16_flags_are_checked():
    lib = api.load()
    ws = api.new_workspace(1, 1)
    x = torch.zeros((1, 1, 8, 64), dtype=torch.float16, device="cuda")
    o = torch.zeros((1, 1, 8, 64), dtype=torch.uint8, device="cuda")
    s = torch.ones((1, 1), dtype=torch.float32, device="cuda")
    p = lambda t: t.data_ptr()
    rc = lib.fp8attn_quantize_ex(p(x), 1, 1, 8, 64, None, p(o), p(s), 0x40, p(ws), ws.numel(), None)
    assert rc == api.ERR_INVALID_ARG
    rc = lib.fp8attn_quantize_ex(p(x), 1, 1, 8, 64, None, p(o), p(s), api.INPUT_FP16, p(ws), ws.numel(), None)
    assert rc == api.OK


# ---- scales computed upstream ----------------------------------------------------------

def test_quantize_with_given_scales_is_one_launch_and_bit_exact():
    w = W.CONFIGS["C2"].scaled(1031, 77)
    g = W.generate(w)
    ref = quantized(g)
    ws = api.new_workspace(w.B, w.H)
    dev = lambda a: torch.from_numpy(a).cuda()
    x = {k: bf16_dev(g[k]) for k in ("q_train", "q_test", "k", "v")}
    # the scales the maximum pass would have found: identical codes, in one launch
    given = {"sq": dev(ref[4]), "sk": dev(ref[5]), "sv": dev(ref[6])}
    before = api.launch_count()
    o = api.quantize_qkv(x["q_train"], x["k"], x["v"], x["q_test"], ws, out=dict(given),
                         flags=api.SCALES_GIVEN)
    assert api.launch_count() - before == 1
    for name, r in zip(("q8", "t8", "k8", "v8"), ref[:4]):
        assert np.array_equal(o[name].cpu().numpy(), r), name
    for name, r in zip(("sq", "sk", "sv"), ref[4:]):
        assert np.array_equal(o[name].cpu().numpy(), r), name          # left as given
    # other scales: the oracle with the same scales, values out of range saturate
    half = {k: dev(v / 2) for k, v in zip(("sq", "sk", "sv"), ref[4:])}
    o = api.quantize_qkv(x["q_train"], x["k"], x["v"], x["q_test"], ws, out=dict(half),
                         flags=api.SCALES_GIVEN)
    for name, src, sc in (("q8", "q_train", 4), ("t8", "q_test", 4), ("k8", "k", 5), ("v8", "v", 6)):
        want, _ = oracle.quantize(g[src], scale_in=ref[sc] / 2)
        assert np.array_equal(o[name].cpu().numpy(), want), name
    assert (o["k8"].cpu().numpy() & 0x7F).max() == 0x7E
    assert api.last_device_status(ws) == (0, 0)
    lib = api.load()
    p = lambda t: t.data_ptr()
    rc = lib.fp8attn_quantize_qkv_ex(p(x["q_train"]), p(x["k"]), p(x["v"]), p(x["q_test"]), w.B, w.H,
                                     w.n_train, w.n_test, w.d, p(o["q8"]), p(o["k8"]), p(o["v8"]), p(o["t8"]),
                                     p(o["sq"]), p(o["sk"]), p(o["sv"]),
                                     api.SCALES_GIVEN | api.QUERY_SCALE_FROM_ALL_ROWS, p(ws), ws.numel(), None)
    assert rc == api.ERR_INVALID_ARG


def test_fp16_whole_path_at_size_sampled():
    """fp16 in, fp16 out at a size that spans many CTAs, steps and a ragged tail: the
    quantizer bit-exact, the FP8 attention and the fp16 twin against the oracle on
    sampled rows."""
    from helpers import sample_rows
    w = W.CONFIGS["C3"].scaled(20011, 3001)
    g = {k: to_fp16_bits(v) for k, v in W.generate(w).items()}
    x = {k: fp16_dev(v) for k, v in g.items()}
    ws = api.new_workspace(w.B, w.H)
    q8, t8, k8, v8, sq, sk, sv = quantized(g, "fp16")
    o = api.quantize_qkv(x["q_train"], x["k"], x["v"], x["q_test"], ws)
    for name, r in zip(("q8", "t8", "k8", "v8", "sq", "sk", "sv"), (q8, t8, k8, v8, sq, sk, sv)):
        assert np.array_equal(o[name].cpu().numpy(), r), name
    f_tr, f_te = api.icl_attention(x["q_train"], x["q_test"], x["k"], x["v"], ws)
    h_tr, h_te = api.icl_forward_bf16(x["q_train"], x["q_test"], x["k"], x["v"], ws)
    assert f_tr.dtype == torch.float16 and h_te.dtype == torch.float16
    assert api.last_device_status(ws) == (0, 0)
    for name, f_out, h_out, codes, bits, nq in (("train", f_tr, h_tr, q8, g["q_train"], w.n_train),
                                                ("test", f_te, h_te, t8, g["q_test"], w.n_test)):
        rows = sample_rows(nq, 40, 9)
        idx = torch.from_numpy(rows).cuda()
        A, Abs, Bnd = oracle.icl_attention_rows(codes, k8, v8, rows, sq=sq, sk=sk, sv=sv)
        check_fp8_attention(f64(f_out[:, :, idx]), A, Abs, Bnd, diffuse=False, label=f"fp16-io/{name}",
                            named_config=False)
        A, Abs, _ = oracle.icl_attention_rows(bits, g["k"], g["v"], rows, dtype16="fp16")
        check_bf16_attention(f64(h_out[:, :, idx]), A, Abs, label=f"fp16-twin/{name}", rounding=2.0 ** -12)
