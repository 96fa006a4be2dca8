"""GPU parity: fused ICL attention (FP8 and BF16 paths) against the oracle's exact
softmax attention over the dequantized / original operands."""
import numpy as np
import pytest
import torch

import oracle
from helpers import (Guarded, bf16_bits_to_f64, check_bf16_attention, check_fp8_attention,
                     f32_to_bf16_bits, sample_rows)
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def out_to_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def oracle_quantized(g):
    q8, sq = oracle.quantize(g["q_train"])
    k8, sk = oracle.quantize(g["k"])
    v8, sv = oracle.quantize(g["v"])
    t8 = None
    if g["q_test"].shape[2]:
        t8, _ = oracle.quantize(g["q_test"], scale_in=sq)
    return dict(q8=q8, k8=k8, v8=v8, t8=t8, sq=sq, sk=sk, sv=sv)


def gpu_fp8_forward(z, w, alpha=0.0):
    dev = lambda a: None if a is None else torch.from_numpy(a).cuda()
    ws = api.new_workspace(w.B, w.H)
    # outputs sit between canary bytes: a store past a ragged tile's last row would show
    g_tr = Guarded((w.B, w.H, w.n_train, w.d), torch.bfloat16)
    g_te = Guarded((w.B, w.H, w.n_test, w.d), torch.bfloat16) if w.n_test else None
    o_tr, o_te = api.icl_forward_fp8(dev(z["q8"]), dev(z["t8"]), dev(z["k8"]), dev(z["v8"]),
                                     dev(z["sq"]), dev(z["sk"]), dev(z["sv"]), ws, alpha,
                                     out_train=g_tr.t, out_test=None if g_te is None else g_te.t)
    assert api.last_device_status(ws) == (0, 0)
    g_tr.check(f"{w.name} out_train")
    if g_te is not None:
        g_te.check(f"{w.name} out_test")
    return o_tr, o_te


def check_fp8_case(w, n_sample=None, diffuse=False, alpha=None, named_config=False):
    g = W.generate(w)
    z = oracle_quantized(g)
    o_tr, o_te = gpu_fp8_forward(z, w, 0.0 if alpha is None else alpha)
    stats = {}
    for name, out, q8, nq in (("train", o_tr, z["q8"], w.n_train), ("test", o_te, z["t8"], w.n_test)):
        if nq == 0:
            assert out is None
            continue
        rows = np.arange(nq) if n_sample is None else sample_rows(nq, n_sample, w.seed)
        A, Abs, Bnd = oracle.icl_attention_rows(q8, z["k8"], z["v8"], rows, sq=z["sq"], sk=z["sk"],
                                                sv=z["sv"], alpha=alpha)
        got = out_to_f64(out[:, :, torch.from_numpy(rows).cuda()])
        stats[name] = check_fp8_attention(got, A, Abs, Bnd, diffuse, label=f"{w.name}/{name}",
                                          named_config=named_config)
        # raw figures next to the normalised ones (visible with pytest -s / -rP)
        print(f"parity {w.name}/{name}: rows/head {rows.size} max_abs {stats[name]['max_abs']:.4g} "
              f"mean_abs {stats[name]['mean_abs']:.4g} max_norm {stats[name]['max_norm']:.4g} "
              f"mean_norm {stats[name]['mean_norm']:.4g} rel_rms {stats[name]['rel_rms']:.4g} "
              f"bound_ratio {stats[name]['bound_ratio']:.3f}")
        # no worse than the method-faithful two-pass e4m3-P evaluation
        O4 = oracle.icl_attention_rows(q8, z["k8"], z["v8"], rows, sq=z["sq"], sk=z["sk"],
                                       sv=z["sv"], alpha=alpha, mode="p8")
        faithful = np.mean(np.abs(O4 - A) / np.maximum(1, Abs))
        assert stats[name]["mean_norm"] <= 1.25 * faithful + 1e-5, (stats[name], faithful)
    return stats


def check_bf16_case(w, n_sample=None):
    g = W.generate(w)
    ws = api.new_workspace(w.B, w.H)
    q_test = to_dev(g["q_test"]) if w.n_test else None
    g_tr = Guarded((w.B, w.H, w.n_train, w.d), torch.bfloat16)
    g_te = Guarded((w.B, w.H, w.n_test, w.d), torch.bfloat16) if w.n_test else None
    o_tr, o_te = api.icl_forward_bf16(to_dev(g["q_train"]), q_test, to_dev(g["k"]), to_dev(g["v"]), ws,
                                      out_train=g_tr.t, out_test=None if g_te is None else g_te.t)
    assert api.last_device_status(ws) == (0, 0)
    g_tr.check(f"{w.name} bf16 out_train")
    if g_te is not None:
        g_te.check(f"{w.name} bf16 out_test")
    for name, out, q, nq in (("train", o_tr, g["q_train"], w.n_train), ("test", o_te, g["q_test"], w.n_test)):
        if nq == 0:
            continue
        rows = np.arange(nq) if n_sample is None else sample_rows(nq, n_sample, w.seed)
        A, Abs, _ = oracle.icl_attention_rows(q, g["k"], g["v"], rows)
        got = out_to_f64(out[:, :, torch.from_numpy(rows).cuda()])
        st = check_bf16_attention(got, A, Abs, label=f"{w.name}/{name}")
        print(f"parity bf16 {w.name}/{name}: rows/head {rows.size} max_abs {st['max_abs']:.4g} mean_abs {st['mean_abs']:.4g} "
              f"max_norm {st['max_norm']:.4g} mean_norm {st['mean_norm']:.4g} rel_rms {st['rel_rms']:.4g} "
              f"bound_ratio {st['bound_ratio']:.3f}")


# ---- FP8 path ---------------------------------------------------------------------

def test_fp8_c1_full():
    check_fp8_case(W.CONFIGS["C1"], diffuse=True, named_config=True)


@pytest.mark.parametrize("n,m", [(1, 0), (1, 1), (5, 3), (127, 1), (128, 128), (129, 77), (255, 257),
                                 (500, 77), (640, 0), (1000, 300)])
def test_fp8_ragged_shapes(n, m):
    check_fp8_case(W.CONFIGS["C1"].scaled(n, m))


def test_fp8_d128_small():
    check_fp8_case(W.CONFIGS["C3"].scaled(700, 130))


def test_fp8_c2_sampled():
    check_fp8_case(W.CONFIGS["C2"], n_sample=96, named_config=True)


def test_fp8_c4_like_shifted_keys_diffuse():
    check_fp8_case(W.CONFIGS["C4"].scaled(2048, 300), n_sample=64, diffuse=True)


def test_fp8_c3_full_size_sampled():
    # 256 stratified rows per head and call, plus the tile-boundary rows
    check_fp8_case(W.CONFIGS["C3"], n_sample=256, named_config=True)


def test_fp8_c4_full_size_sampled():
    # B=4 independent tables, 262,144 train rows each, keys with mean 3: diffuse softmax
    check_fp8_case(W.CONFIGS["C4"], n_sample=64, diffuse=True, named_config=True)


def test_fp8_c5_full_size_sampled():
    # 1,048,576 train rows: the large-table regime
    check_fp8_case(W.CONFIGS["C5"], n_sample=32, named_config=True)


def test_fp8_custom_softmax_scale():
    check_fp8_case(W.CONFIGS["C1"].scaled(300, 40), alpha=0.05)


# ---- BF16 comparison path -----------------------------------------------------------

def test_bf16_c1_full():
    check_bf16_case(W.CONFIGS["C1"])


@pytest.mark.parametrize("n,m", [(1, 0), (129, 77), (500, 300)])
def test_bf16_ragged_shapes(n, m):
    check_bf16_case(W.CONFIGS["C1"].scaled(n, m))


def test_bf16_d128_small():
    check_bf16_case(W.CONFIGS["C3"].scaled(700, 130))


def test_bf16_c2_sampled():
    check_bf16_case(W.CONFIGS["C2"], n_sample=64)


def test_bf16_c3_full_size_sampled():
    check_bf16_case(W.CONFIGS["C3"], n_sample=128)


def test_bf16_c4_full_size_sampled():
    # d = 64 at a size that takes the three-tile kernel
    check_bf16_case(W.CONFIGS["C4"], n_sample=32)


# ---- structure of the ICL layer -------------------------------------------------------

def test_test_rows_are_batch_invariant_and_share_kv_with_train_rows():
    w = W.CONFIGS["C1"].scaled(384, 200)
    g = W.generate(w)
    z = oracle_quantized(g)
    _, full = gpu_fp8_forward(z, w)
    # a single test row alone gives the bit-identical output row
    z1 = dict(z); z1["t8"] = np.ascontiguousarray(z["t8"][:, :, 131:132])
    _, single = gpu_fp8_forward(z1, w.scaled(384, 1))
    assert torch.equal(single[:, :, 0], full[:, :, 131])
    # permuting the test batch permutes the outputs and nothing else
    perm = np.random.default_rng(0).permutation(w.n_test)
    z2 = dict(z); z2["t8"] = np.ascontiguousarray(z["t8"][:, :, perm])
    tr2, shuffled = gpu_fp8_forward(z2, w)
    assert torch.equal(shuffled, full[:, :, torch.from_numpy(perm).cuda()])
    # a test query identical to a train query produces the train row's output
    z3 = dict(z); t8 = z["t8"].copy(); t8[:, :, 5] = z["q8"][:, :, 300]; z3["t8"] = t8
    tr3, te3 = gpu_fp8_forward(z3, w)
    assert torch.equal(te3[:, :, 5], tr3[:, :, 300])
    # train outputs never depend on the test queries
    assert torch.equal(tr2, tr3)


def test_runs_are_deterministic():
    w = W.CONFIGS["C2"].scaled(1024, 256)
    z = oracle_quantized(W.generate(w))
    a = gpu_fp8_forward(z, w)
    b = gpu_fp8_forward(z, w)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_forward_argument_errors():
    lib = api.load()
    ws = api.new_workspace(1, 1)
    q = torch.zeros((1, 1, 8, 64), dtype=torch.uint8, device="cuda")
    o = torch.zeros((1, 1, 8, 64), dtype=torch.bfloat16, device="cuda")
    s = torch.ones((1, 1), dtype=torch.float32, device="cuda")
    p = lambda t: t.data_ptr()
    f = lib.fp8attn_icl_forward
    args = lambda **kw: [kw.get("q", p(q)), None, p(q), p(q), p(s), p(s), kw.get("sv", p(s)), 1, 1,
                         kw.get("n", 8), kw.get("m", 0), kw.get("d", 64), 0.0, p(o), None, p(ws),
                         kw.get("wsb", ws.numel()), None]
    assert f(*args(d=32)) == api.ERR_UNSUPPORTED
    assert f(*args(n=0)) == api.ERR_INVALID_ARG
    assert f(*args(m=4)) == api.ERR_INVALID_ARG          # test rows without test tensors
    assert f(*args(sv=None)) == api.ERR_INVALID_ARG
    assert f(*args(q=None)) == api.ERR_INVALID_ARG
    assert f(*args(wsb=16)) == api.ERR_WORKSPACE
    assert f(*args()) == api.OK
    assert api.last_device_status(ws) == (0, 0)


# ---- degenerate inputs ------------------------------------------------------------------

def test_fp8_degenerate_heads_zero_queries_zero_keys_and_saturated_test_queries():
    """Head 0: all-zero queries (uniform weights -> mean of the value rows); head 1: all-zero
    keys (same); test queries far outside the train range saturate at +-448 and still match."""
    w = W.CONFIGS["C1"].scaled(333, 50)
    g = W.generate(w)
    g["q_train"][:, 0] = 0
    g["q_test"][:, 0] = 0
    g["k"][:, 1] = 0
    big = W.bf16_bits_to_f32(g["q_test"][:, 1]) * np.float32(50.0)      # beyond the train-query absmax
    g["q_test"][:, 1] = f32_to_bf16_bits(big)
    z = oracle_quantized(g)
    assert np.all(z["sq"][:, 0] == 1.0) and np.all(z["sk"][:, 1] == 1.0)
    assert (z["t8"][:, 1] & 0x7F).max() == 0x7E
    o_tr, o_te = gpu_fp8_forward(z, w)
    tab = oracle.e4m3_decode_table()
    vhat = tab[z["v8"]] * z["sv"][:, :, None, None].astype(np.float64)
    for out in (o_tr, o_te):
        got = out_to_f64(out)
        for h in (0, 1):
            mean_v = vhat[0, h].mean(axis=0)
            assert np.max(np.abs(got[0, h] - mean_v)) < 2e-2 * max(1.0, np.abs(mean_v).max()) + 5e-3
    for name, out, q8, nq in (("train", o_tr, z["q8"], w.n_train), ("test", o_te, z["t8"], w.n_test)):
        A, Abs, Bnd = oracle.icl_attention_rows(q8, z["k8"], z["v8"], np.arange(nq), sq=z["sq"], sk=z["sk"],
                                                sv=z["sv"])
        check_fp8_attention(out_to_f64(out), A, Abs, Bnd, diffuse=False, label=name, named_config=False)


@pytest.mark.parametrize("d,fp8", [(128, True), (64, True), (128, False), (64, False)])
def test_repeated_launches_are_bit_identical(d, fp8):
    """Every barrier hand-over in the kernel orders real data: a race would show up as
    run-to-run differences, so the same call must give the same bits every time."""
    torch.manual_seed(d + fp8)
    B, H, N, M = 1, 4, 12000, 3000
    ws = api.new_workspace(B, H)
    if fp8:
        mk = lambda r: torch.randint(0, 256, (B, H, r, d), dtype=torch.uint8, device="cuda")
        clean = lambda t: torch.where((t & 0x7F) == 0x7F, t & 0xFE, t)       # no NaN codes
        q, t, k, v = (clean(mk(r)) for r in (N, M, N, N))
        s = torch.full((B, H), 0.003, dtype=torch.float32, device="cuda")
        run = lambda: api.icl_forward_fp8(q, t, k, v, s, s, s, ws)
    else:
        mk = lambda r: torch.randn((B, H, r, d), dtype=torch.bfloat16, device="cuda")
        q, t, k, v = mk(N), mk(M), mk(N), mk(N)
        run = lambda: api.icl_forward_bf16(q, t, k, v, ws)
    first = [o.clone() for o in run()]
    assert all(torch.isfinite(o.float()).all() for o in first)
    for _ in range(6):
        again = run()
        assert torch.equal(again[0], first[0]) and torch.equal(again[1], first[1])
    assert api.last_device_status(ws) == (0, 0)
