"""FP8ATTN_SPLIT_TAIL: the query blocks left over after the last full round of CTAs are run
by several CTAs over disjoint key ranges and combined.  Checked against the oracle like the
plain path; rows outside the split blocks must be untouched by it, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from helpers import check_bf16_attention, check_fp8_attention, sample_rows
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu



def sm_count():
    return torch.cuda.get_device_properties(0).multi_processor_count


def bf16_dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def quantized(g):
    q8, sq = oracle.quantize(g["q_train"])
    k8, sk = oracle.quantize(g["k"])
    v8, sv = oracle.quantize(g["v"])
    t8, _ = oracle.quantize(g["q_test"], scale_in=sq)
    return q8, t8, k8, v8, sq, sk, sv


def split_rows_mask(w, test_only=False):
    """Which (head, call, row) take the split path: the blocks past the last full round."""
    bt = 0 if test_only else (w.n_train + 255) // 256
    be = (w.n_test + 255) // 256
    per_head = bt + be
    grid = w.B * w.H * per_head
    full = (grid // sm_count()) * sm_count()
    tr = np.zeros((w.B * w.H, w.n_train), dtype=bool)
    te = np.zeros((w.B * w.H, w.n_test), dtype=bool)
    for blk in range(full, grid):
        bh, b = divmod(blk, per_head)
        if b < bt:
            tr[bh, b * 256:(b + 1) * 256] = True
        else:
            te[bh, (b - bt) * 256:(b - bt + 1) * 256] = True
    return tr.reshape(w.B, w.H, -1), te.reshape(w.B, w.H, -1)


@pytest.mark.parametrize("cfg,n,m", [("C2", 8192, 2048), ("C3", 4500, 700), ("C4", 2600, 300)])
def test_fp8_split_tail_against_oracle(cfg, n, m):
    w = W.CONFIGS[cfg].scaled(n, m)
    g = W.generate(w)
    ref = quantized(g)
    dev = lambda a: torch.from_numpy(a).cuda()
    args = [dev(a) for a in ref]
    ws = api.new_workspace(w.B, w.H, n_train=n, n_test=m, d=w.d)
    p_tr, p_te = api.icl_forward_fp8(*args, ws)
    before = api.launch_count()
    s_tr, s_te = api.icl_forward_fp8(*args, ws, flags=api.SPLIT_TAIL)
    assert api.launch_count() - before == 3                 # full rounds, split blocks, combine
    assert api.last_device_status(ws) == (0, 0)
    m_tr, m_te = split_rows_mask(w)
    assert m_tr.any() or m_te.any()
    # rows outside the split blocks: the same CTAs did the same work
    for plain, split, mask in ((p_tr, s_tr, m_tr), (p_te, s_te, m_te)):
        keep = torch.from_numpy(~mask).cuda()
        assert torch.equal(plain[keep], split[keep])
    # rows inside: a different but equally valid order of the online softmax
    inside = torch.from_numpy(m_te).cuda()
    assert not torch.equal(p_te[inside], s_te[inside])
    q8, t8, k8, v8, sq, sk, sv = ref
    for name, out, q, nq, mask in (("train", s_tr, q8, n, m_tr), ("test", s_te, t8, m, m_te)):
        rows = np.unique(np.concatenate([sample_rows(nq, 24, 3), np.nonzero(mask.any(axis=(0, 1)))[0][::7]]))
        A, Abs, Bnd = oracle.icl_attention_rows(q, k8, v8, rows, sq=sq, sk=sk, sv=sv)
        check_fp8_attention(f64(out[:, :, torch.from_numpy(rows).cuda()]), A, Abs, Bnd, diffuse=False,
                            label=f"split/{cfg}/{name}", named_config=False)


@pytest.mark.parametrize("d,n,m,flags", [(128, 20011, 300, 0), (64, 33000, 129, 0), (128, 9000, 257, 1)])
def test_fp8_split_of_the_test_call_alone(d, n, m, flags):
    """Few test rows against many train keys: the whole grid is less than one round."""
    base = W.CONFIGS["C3" if d == 128 else "C5"]
    w = base.scaled(n, m)
    g = W.generate(w)
    q8, t8, k8, v8, sq, sk, sv = quantized(g)
    dev = lambda a: torch.from_numpy(a).cuda()
    ws = api.new_workspace(w.B, w.H, n_train=n, n_test=m, d=d)
    fl = api.TEST_ROWS_ONLY | api.SPLIT_TAIL | (api.TEST_ROWS_USE_KV_HEAD0 if flags else 0)
    before = api.launch_count()
    _, out = api.icl_forward_fp8(None, dev(t8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), ws, flags=fl,
                                 out_dtype=torch.float16 if d == 64 else torch.bfloat16)
    assert api.launch_count() - before == 2                 # split blocks, combine
    assert api.last_device_status(ws) == (0, 0)
    if flags:
        h0 = lambda x: np.ascontiguousarray(np.broadcast_to(x[:, :1], x.shape))
        k8, v8, sk, sv = h0(k8), h0(v8), h0(sk), h0(sv)
    A, Abs, Bnd = oracle.icl_attention_rows(t8, k8, v8, np.arange(m), sq=sq, sk=sk, sv=sv)
    check_fp8_attention(f64(out), A, Abs, Bnd, diffuse=False, label=f"split-test-only/{d}/{n}+{m}",
                        named_config=False)


def test_bf16_split_tail_against_oracle():
    w = W.CONFIGS["C2"].scaled(4500, 500)
    g = W.generate(w)
    x = {k: bf16_dev(v) for k, v in g.items()}
    ws = api.new_workspace(w.B, w.H, n_train=w.n_train, n_test=w.n_test, d=w.d)
    before = api.launch_count()
    o_tr, o_te = api.icl_forward_bf16(x["q_train"], x["q_test"], x["k"], x["v"], ws, flags=api.SPLIT_TAIL)
    assert api.launch_count() - before == 3 and api.last_device_status(ws) == (0, 0)
    for out, q, nq in ((o_tr, g["q_train"], w.n_train), (o_te, g["q_test"], w.n_test)):
        rows = np.unique(np.concatenate([sample_rows(nq, 30, 5), np.arange(max(0, nq - 300), nq, 5)]))
        A, Abs, _ = oracle.icl_attention_rows(q, g["k"], g["v"], rows)
        check_bf16_attention(f64(out[:, :, torch.from_numpy(rows).cuda()]), A, Abs, label="split/bf16")


def test_split_tail_leaves_other_launch_shapes_alone_and_checks_its_workspace():
    # many rounds: the flag changes nothing, bit for bit, and adds no launch
    w = W.CONFIGS["C3"].scaled(40000, 3000)
    torch.manual_seed(0)
    mk = lambda r: torch.randint(0, 0x7E, (w.B, w.H, r, w.d), dtype=torch.uint8, device="cuda")
    q, t, k, v = mk(w.n_train), mk(w.n_test), mk(w.n_train), mk(w.n_train)
    s = torch.full((w.B, w.H), 0.004, dtype=torch.float32, device="cuda")
    ws = api.new_workspace(w.B, w.H, n_train=w.n_train, n_test=w.n_test, d=w.d)
    a_tr, a_te = api.icl_forward_fp8(q, t, k, v, s, s, s, ws)
    before = api.launch_count()
    b_tr, b_te = api.icl_forward_fp8(q, t, k, v, s, s, s, ws, flags=api.SPLIT_TAIL)
    assert api.launch_count() - before == 1
    assert torch.equal(a_tr, b_tr) and torch.equal(a_te, b_te)
    # the small workspace has no room for the partial results
    small = api.new_workspace(w.B, w.H)
    with pytest.raises(api.Fp8AttnError) as e:
        api.icl_forward_fp8(q, t, k, v, s, s, s, small, flags=api.SPLIT_TAIL)
    assert e.value.status == api.ERR_WORKSPACE
    assert api.workspace_bytes(1, 8, 4096, 0, 128) > api.workspace_bytes(1, 8) + (1 << 20)
