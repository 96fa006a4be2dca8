"""GPU parity: fp8attn_quantize must match the oracle bit for bit (codes and scales)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import f32_to_bf16_bits
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def run_case(w):
    g = W.generate(w)
    ws = api.new_workspace(w.B, w.H)
    scales = {}
    for name in ("q_train", "k", "v"):
        codes, s = api.quantize(to_dev(g[name]), ws)
        rc, rs = oracle.quantize(g[name])
        assert np.array_equal(s.cpu().numpy(), rs), name
        got = codes.cpu().numpy()
        assert np.array_equal(got, rc), (name, int((got != rc).sum()))
        scales[name] = s
    if w.n_test:
        codes, s = api.quantize(to_dev(g["q_test"]), ws, scale_in=scales["q_train"])
        rc, rs = oracle.quantize(g["q_test"], scale_in=scales["q_train"].cpu().numpy())
        assert np.array_equal(s.cpu().numpy(), rs)
        assert np.array_equal(codes.cpu().numpy(), rc)
    assert api.last_device_status(ws) == (0, 0)


@pytest.mark.parametrize("cfg", ["C1", "C2"])
def test_full_configs_small(cfg):
    run_case(W.CONFIGS[cfg])


@pytest.mark.parametrize("cfg,n,m", [("C3", 8192, 2048), ("C4", 4096, 1000), ("C5", 16384, 4096),
                                      ("C1", 1, 0), ("C1", 3, 1), ("C2", 129, 77), ("C3", 500, 7)])
def test_scaled_and_ragged(cfg, n, m):
    run_case(W.CONFIGS[cfg].scaled(n, m))


@pytest.mark.parametrize("cfg", ["C3", "C4", "C5"])
def test_full_size(cfg):
    """Full-size tensors, one tensor at a time to bound host memory."""
    w = W.CONFIGS[cfg]
    ws = api.new_workspace(w.B, w.H)
    sq = None
    for name, tid, rows in (("q_train", W.Q_TRAIN, w.n_train), ("k", W.K, w.n_train),
                            ("v", W.V, w.n_train), ("q_test", W.Q_TEST, w.n_test)):
        bits = W.fill(np.empty((w.B, w.H, rows, w.d), dtype=np.uint16), w, tid)
        s_in = sq if name == "q_test" else None
        codes, s = api.quantize(to_dev(bits), ws, scale_in=s_in)
        rc, rs = oracle.quantize(bits, scale_in=None if s_in is None else s_in.cpu().numpy())
        if name == "q_train":
            sq = s
        assert np.array_equal(s.cpu().numpy(), rs), name
        got = codes.cpu().numpy()
        assert np.array_equal(got, rc), (name, int((got != rc).sum()))
        del bits, codes, got, rc
    assert api.last_device_status(ws) == (0, 0)


def test_special_values_and_edges():
    ws = api.new_workspace(1, 3)
    x = np.zeros((1, 3, 16, 64), dtype=np.float32)
    x[0, 1] = np.linspace(-3, 3, 1024, dtype=np.float32).reshape(16, 64)
    x[0, 2, :, :] = 1e-30                      # tiny magnitudes: scale is subnormal-adjacent
    x[0, 2, 3, 5] = -3e-30
    x[0, 1, 0, 0] = -0.0
    bits = f32_to_bf16_bits(x)
    codes, s = api.quantize(to_dev(bits), ws)
    rc, rs = oracle.quantize(bits)
    assert np.array_equal(s.cpu().numpy(), rs) and np.array_equal(codes.cpu().numpy(), rc)
    assert rs[0, 0] == 1.0
    # test queries beyond the train range saturate at +-448
    big = f32_to_bf16_bits(np.full((1, 3, 2, 64), 1e6, dtype=np.float32))
    big[0, :, 1] |= 0x8000
    codes, s2 = api.quantize(to_dev(big), ws, scale_in=s)
    rc, _ = oracle.quantize(big, scale_in=rs)
    assert np.array_equal(codes.cpu().numpy(), rc)
    assert set(np.unique(rc[0, 1])) == {0x7E, 0xFE}
    # heads are independent: scaling one head leaves the others' codes untouched
    y = x.copy(); y[0, 1] *= 1024
    c2, s3 = api.quantize(to_dev(f32_to_bf16_bits(y)), ws)
    c1, _ = api.quantize(to_dev(bits), ws)
    assert torch.equal(c1[0, 0], c2[0, 0]) and torch.equal(c1[0, 2], c2[0, 2]) and torch.equal(c1[0, 1], c2[0, 1])


def test_argument_errors_are_reported_on_the_host():
    lib = api.load()
    ws = api.new_workspace(1, 2)
    x = torch.zeros((1, 2, 4, 64), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros((1, 2, 4, 64), dtype=torch.uint8, device="cuda")
    s = torch.zeros((1, 2), dtype=torch.float32, device="cuda")
    p = lambda t: t.data_ptr()
    q = lib.fp8attn_quantize
    assert q(p(x), 1, 2, 4, 96, None, p(o), p(s), p(ws), ws.numel(), None) == api.ERR_UNSUPPORTED
    assert q(None, 1, 2, 4, 64, None, p(o), p(s), p(ws), ws.numel(), None) == api.ERR_INVALID_ARG
    assert q(p(x), 0, 2, 4, 64, None, p(o), p(s), p(ws), ws.numel(), None) == api.ERR_INVALID_ARG
    assert q(p(x), 1, 2, 4, 64, None, p(o), None, p(ws), ws.numel(), None) == api.ERR_INVALID_ARG
    assert q(p(x) + 2, 1, 2, 4, 64, None, p(o), p(s), p(ws), ws.numel(), None) == api.ERR_INVALID_ARG
    assert q(p(x), 1, 2, 4, 64, None, p(o), p(s), p(ws), 8, None) == api.ERR_WORKSPACE
    assert q(p(x), 1, 2, 4, 64, None, p(o), p(s), None, ws.numel(), None) == api.ERR_WORKSPACE
    assert q(p(x), 1, 2, 4, 64, None, p(o), p(s), p(ws), ws.numel(), None) == api.OK
    torch.cuda.synchronize()


@pytest.mark.parametrize("cfg,n,m", [("C1", 512, 128), ("C2", 8192, 2048), ("C4", 3000, 0), ("C3", 4096, 1),
                                      ("C5", 1, 0)])
def test_fused_qkv_quantize_matches_oracle(cfg, n, m):
    """fp8attn_quantize_qkv is bit-identical to the oracle, including the shared train-query
    scale for the test queries: as one launch (these sizes are small calls), and as two launches
    when asked for.  Twice in a row on one workspace: the one-launch path must leave its
    counters clean."""
    w = W.CONFIGS[cfg].scaled(n, m)
    g = W.generate(w)
    ws = api.new_workspace(w.B, w.H)
    rq, rsq = oracle.quantize(g["q_train"])
    rk, rsk = oracle.quantize(g["k"])
    rv, rsv = oracle.quantize(g["v"])
    dev = [to_dev(g["q_train"]), to_dev(g["k"]), to_dev(g["v"]), to_dev(g["q_test"]) if m else None]
    for flags, launches in ((0, 1), (0, 1), (api.QKV_TWO_LAUNCHES, 2), (0, 1)):
        before = api.launch_count()
        o = api.quantize_qkv(*dev, ws, flags=flags)
        assert api.launch_count() - before == launches
        for got, ref in ((o["q8"], rq), (o["k8"], rk), (o["v8"], rv), (o["sq"], rsq), (o["sk"], rsk), (o["sv"], rsv)):
            assert np.array_equal(got.cpu().numpy(), ref)
        if m:
            rt, _ = oracle.quantize(g["q_test"], scale_in=rsq)
            assert np.array_equal(o["t8"].cpu().numpy(), rt)
        assert api.last_device_status(ws) == (0, 0)


def test_fused_qkv_large_call_takes_two_launches():
    """Above the one-launch size (48 MB of 16-bit input) the call is a maximum pass and a
    conversion pass; bit-identical to the oracle all the same."""
    w = W.CONFIGS["C3"].scaled(20000, 3000)      # 8 heads x 128 x (3 x 20000 + 3000) x 2 B = 129 MB
    g = W.generate(w)
    ws = api.new_workspace(w.B, w.H)
    before = api.launch_count()
    o = api.quantize_qkv(to_dev(g["q_train"]), to_dev(g["k"]), to_dev(g["v"]), to_dev(g["q_test"]), ws)
    assert api.launch_count() - before == 2
    rq, rsq = oracle.quantize(g["q_train"])
    rt, _ = oracle.quantize(g["q_test"], scale_in=rsq)
    rv, rsv = oracle.quantize(g["v"])
    assert np.array_equal(o["q8"].cpu().numpy(), rq) and np.array_equal(o["t8"].cpu().numpy(), rt)
    assert np.array_equal(o["v8"].cpu().numpy(), rv) and np.array_equal(o["sv"].cpu().numpy(), rsv)
    assert api.last_device_status(ws) == (0, 0)


@pytest.mark.parametrize("extra", [0, api.QKV_TWO_LAUNCHES])
def test_fused_qkv_query_scale_from_all_rows(extra):
    """Single-call form: one query scale over train and test queries together (one-launch and
    two-launch paths)."""
    w = W.CONFIGS["C2"].scaled(700, 900)
    g = W.generate(w)
    g["q_test"] = f32_to_bf16_bits(W.bf16_bits_to_f32(g["q_test"]) * np.float32(3.0))   # test rows set the maximum
    ws = api.new_workspace(w.B, w.H)
    o = api.quantize_qkv(to_dev(g["q_train"]), to_dev(g["k"]), to_dev(g["v"]), to_dev(g["q_test"]), ws,
                         flags=api.QUERY_SCALE_FROM_ALL_ROWS | extra)
    _, s_all = oracle.quantize(np.concatenate([g["q_train"], g["q_test"]], axis=2))
    rq, _ = oracle.quantize(g["q_train"], scale_in=s_all)
    rt, _ = oracle.quantize(g["q_test"], scale_in=s_all)
    _, s_train = oracle.quantize(g["q_train"])
    assert np.all(s_all > s_train)
    assert np.array_equal(o["sq"].cpu().numpy(), s_all)
    assert np.array_equal(o["q8"].cpu().numpy(), rq) and np.array_equal(o["t8"].cpu().numpy(), rt)
    rk, rsk = oracle.quantize(g["k"])
    assert np.array_equal(o["k8"].cpu().numpy(), rk) and np.array_equal(o["sk"].cpu().numpy(), rsk)


@pytest.mark.parametrize("scale", [1e-38, 3e-31, 1e-30, 7.3e-12, 1.0, 6.5e11, 1e30, 3e30, 2.9e38])
def test_given_scales_across_the_exponent_range(scale):
    """A given scale anywhere in the fp32 range (the conversion takes its quotients from a
    per-mantissa table inside a safe scale range and divides per element outside it): codes
    equal the oracle's, for inputs that span the whole bf16 exponent range, subnormals, zeros
    and both signs included."""
    rng = np.random.default_rng(17)
    bits = rng.integers(0, 0x7F80, size=(1, 2, 64, 64), dtype=np.uint16)       # every finite magnitude
    bits[0, 0, 0, :8] = [0x0000, 0x0001, 0x007F, 0x0080, 0x7F7F, 0x3F80, 0x0040, 0x7F00]
    bits |= (rng.integers(0, 2, size=bits.shape, dtype=np.uint16) << 15)
    # values around the scale itself, where the codes are neither zero nor saturated
    near = np.clip(rng.standard_normal((1, 2, 64, 64)) * scale * 100, -3e38, 3e38).astype(np.float32)
    near_bits = f32_to_bf16_bits(near).reshape(1, 2, 64, 64)
    x = np.concatenate([bits, near_bits], axis=2)
    s_in = np.full((1, 2), scale, dtype=np.float32)
    ws = api.new_workspace(1, 2)
    codes, s_out = api.quantize(to_dev(x), ws, scale_in=torch.from_numpy(s_in).cuda())
    want, _ = oracle.quantize(x, scale_in=s_in)
    got = codes.cpu().numpy()
    assert np.array_equal(got, want), np.argwhere(got != want)[:5]
    assert np.array_equal(s_out.cpu().numpy(), s_in)
