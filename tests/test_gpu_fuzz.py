"""Seeded random shapes and flag combinations against the oracle: sizes around the tile,
step and block boundaries (96 / 128 / 256), both head sizes, every forward flag."""
import numpy as np
import pytest
import torch

import oracle
from helpers import Guarded, bf16_bits_to_f64, check_bf16_attention, check_fp8_attention
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu

EDGES = [1, 2, 31, 95, 96, 97, 127, 128, 129, 191, 192, 193, 255, 256, 257, 383, 384, 385, 511, 513, 700]


def cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(count):
        cfg = ["C1", "C2", "C3", "C4", "C5"][rng.integers(0, 5)]
        n = int(EDGES[rng.integers(0, len(EDGES))] + (rng.integers(0, 3) * 256 if rng.random() < 0.3 else 0))
        m = int(EDGES[rng.integers(0, len(EDGES))]) if rng.random() < 0.8 else 0
        out.append((i, cfg, n, m, bool(rng.integers(0, 2)), bool(rng.integers(0, 2)), bool(rng.integers(0, 2)),
                    bool(rng.integers(0, 2))))
    return out


def head0(x):
    return np.ascontiguousarray(np.broadcast_to(x[:, :1], x.shape))


@pytest.mark.parametrize("i,cfg,n,m,fp8,half,gqa,test_only", cases(96, 2609))
def test_random_shapes_and_flags(i, cfg, n, m, fp8, half, gqa, test_only):
    base = W.CONFIGS[cfg]
    w = base.scaled(n, m)
    g = W.generate(w)
    if half:
        g = {k: np.ascontiguousarray(bf16_bits_to_f64(v).astype(np.float16)).view(np.uint16) for k, v in g.items()}
    dtype16 = "fp16" if half else "bf16"
    tdt = torch.float16 if half else torch.bfloat16
    dev16 = lambda b: torch.from_numpy(b.view(np.int16)).cuda().view(tdt)
    test_only = test_only and m > 0
    flags = (api.TEST_ROWS_USE_KV_HEAD0 if gqa else 0) | (api.TEST_ROWS_ONLY if test_only else 0)
    ws = api.new_workspace(w.B, w.H)
    x = {k: dev16(v) for k, v in g.items()}
    q_test = x["q_test"] if m else None
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    # every output buffer sits between canary bytes
    guards = {"o_tr": Guarded((w.B, w.H, n, w.d), tdt), "o_te": Guarded((w.B, w.H, m, w.d), tdt)}
    if fp8:
        for name, rows in (("q8", n), ("k8", n), ("v8", n), ("t8", m)):
            guards[name] = Guarded((w.B, w.H, rows, w.d), torch.uint8)
        for name in ("sq", "sk", "sv"):
            guards[name] = Guarded((w.B, w.H), torch.float32)
        o = api.quantize_qkv(x["q_train"], x["k"], x["v"], q_test, ws,
                             out={k: guards[k].t for k in ("q8", "k8", "v8", "t8", "sq", "sk", "sv")})
        q8, sq = oracle.quantize(g["q_train"], dtype16=dtype16)
        k8, sk = oracle.quantize(g["k"], dtype16=dtype16)
        v8, sv = oracle.quantize(g["v"], dtype16=dtype16)
        assert np.array_equal(o["q8"].cpu().numpy(), q8) and np.array_equal(o["k8"].cpu().numpy(), k8)
        assert np.array_equal(o["v8"].cpu().numpy(), v8) and np.array_equal(o["sq"].cpu().numpy(), sq)
        t8 = None
        if m:
            t8, _ = oracle.quantize(g["q_test"], scale_in=sq, dtype16=dtype16)
            assert np.array_equal(o["t8"].cpu().numpy(), t8)
        o_tr, o_te = api.icl_forward_fp8(None if test_only else o["q8"], o["t8"] if m else None, o["k8"], o["v8"],
                                         o["sq"], o["sk"], o["sv"], ws, flags=flags,
                                         out_train=None if test_only else guards["o_tr"].t,
                                         out_test=guards["o_te"].t if m else None)
    else:
        o_tr, o_te = api.icl_forward_bf16(None if test_only else x["q_train"], q_test, x["k"], x["v"], ws, flags=flags,
                                          out_train=None if test_only else guards["o_tr"].t,
                                          out_test=guards["o_te"].t if m else None)
    assert api.last_device_status(ws) == (0, 0)
    for name, gd in guards.items():
        gd.check(f"fuzz{i} {name}")
    label = f"fuzz{i}/{cfg}/{n}+{m}/fp8={fp8}/half={half}/gqa={gqa}/test_only={test_only}"
    for name, out, nq in (("train", o_tr, n), ("test", o_te, m)):
        if nq == 0 or (name == "train" and test_only):
            assert out is None
            continue
        assert out.dtype == tdt
        kv0 = gqa and name == "test"
        rows = np.arange(nq)
        if fp8:
            kk, vv, ssk, ssv = (head0(k8), head0(v8), head0(sk), head0(sv)) if kv0 else (k8, v8, sk, sv)
            A, Abs, Bnd = oracle.icl_attention_rows(q8 if name == "train" else t8, kk, vv, rows, sq=sq, sk=ssk, sv=ssv)
            check_fp8_attention(f64(out), A, Abs, Bnd, diffuse=False, label=f"{label}/{name}", named_config=False)
        else:
            kk, vv = (head0(g["k"]), head0(g["v"])) if kv0 else (g["k"], g["v"])
            A, Abs, _ = oracle.icl_attention_rows(g["q_train"] if name == "train" else g["q_test"], kk, vv, rows,
                                                  dtype16=dtype16)
            check_bf16_attention(f64(out), A, Abs, label=f"{label}/{name}",
                                 rounding=2.0 ** -12 if half else 2.0 ** -9)
