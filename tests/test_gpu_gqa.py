"""Grouped-query test->train attention (test rows read K/V head 0 of their table, as
in TabPFN-v3 per the paper's appendix) against the oracle, FP8 and BF16 paths."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_bf16_attention, check_fp8_attention
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def to_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def head0(x):
    """[B,H,...] -> every head replaced by head 0 of its table."""
    return np.ascontiguousarray(np.broadcast_to(x[:, :1], x.shape))


@pytest.mark.parametrize("cfg,n,m", [("C4", 1000, 300), ("C3", 700, 130)])
def test_fp8_test_rows_attend_to_kv_head0(cfg, n, m):
    w = W.CONFIGS[cfg].scaled(n, m)          # C4: B=4 tables x H=4 heads
    g = W.generate(w)
    q8, sq = oracle.quantize(g["q_train"])
    k8, sk = oracle.quantize(g["k"])
    v8, sv = oracle.quantize(g["v"])
    t8, _ = oracle.quantize(g["q_test"], scale_in=sq)
    dev = lambda a: torch.from_numpy(a).cuda()
    ws = api.new_workspace(w.B, w.H)
    o_tr, o_te = api.icl_forward_fp8(dev(q8), dev(t8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), ws,
                                     flags=api.TEST_ROWS_USE_KV_HEAD0)
    plain_tr, plain_te = api.icl_forward_fp8(dev(q8), dev(t8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), ws)
    assert api.last_device_status(ws) == (0, 0)
    # train rows are the plain call's, bit for bit; head 0's test rows too
    assert torch.equal(o_tr, plain_tr)
    assert torch.equal(o_te[:, 0], plain_te[:, 0])
    # test rows: oracle over head 0's quantized K/V and scales, own (train-query) scale for Q
    rows = np.arange(w.n_test)
    A, Abs, Bnd = oracle.icl_attention_rows(t8, head0(k8), head0(v8), rows, sq=sq, sk=head0(sk), sv=head0(sv))
    check_fp8_attention(o_te.float().cpu().numpy().astype(np.float64), A, Abs, Bnd, diffuse=False,
                        label=f"{w.name}/gqa-test", named_config=False)
    # and they differ from the plain call for heads other than 0
    assert not torch.equal(o_te[:, 1:], plain_te[:, 1:])


def test_bf16_test_rows_attend_to_kv_head0():
    w = W.CONFIGS["C4"].scaled(600, 200)
    g = W.generate(w)
    ws = api.new_workspace(w.B, w.H)
    o_tr, o_te = api.icl_forward_bf16(to_dev(g["q_train"]), to_dev(g["q_test"]), to_dev(g["k"]),
                                      to_dev(g["v"]), ws, flags=api.TEST_ROWS_USE_KV_HEAD0)
    assert api.last_device_status(ws) == (0, 0)
    A, Abs, _ = oracle.icl_attention_rows(g["q_test"], head0(g["k"]), head0(g["v"]), np.arange(w.n_test))
    check_bf16_attention(o_te.float().cpu().numpy().astype(np.float64), A, Abs, label="gqa-bf16-test")
    A, Abs, _ = oracle.icl_attention_rows(g["q_train"], g["k"], g["v"], np.arange(w.n_train))
    check_bf16_attention(o_tr.float().cpu().numpy().astype(np.float64), A, Abs, label="gqa-bf16-train")


def test_unknown_flag_is_rejected():
    lib = api.load()
    ws = api.new_workspace(1, 1)
    q = torch.zeros((1, 1, 8, 64), dtype=torch.uint8, device="cuda")
    o = torch.zeros((1, 1, 8, 64), dtype=torch.bfloat16, device="cuda")
    s = torch.ones((1, 1), dtype=torch.float32, device="cuda")
    p = lambda t: t.data_ptr()
    rc = lib.fp8attn_icl_forward_ex(p(q), None, p(q), p(q), p(s), p(s), p(s), 1, 1, 8, 0, 64, 0.0, 0x80,
                                    p(o), None, p(ws), ws.numel(), None)
    assert rc == api.ERR_INVALID_ARG
