"""fp8attn_quantize_qkv_ordered / fp8attn_reorder_rows: the keys of largest norm first.
The map is a permutation per head; codes and scales are the oracle's, row for row under the
map; the attention result over the reordered K8, V8 meets the same criteria against the
oracle's attention over the keys in their original order (attention sums over keys)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f64, check_fp8_attention, sample_rows
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu

FIRST = 96        # keys the call brings to the front, at least (it aims at 256, estimated from a sample)


def dev16(bits, dtype=torch.bfloat16):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(dtype)


def check_map(dest, k_values):
    """dest [B,H,N] is a permutation per head, stable within the two groups, and the rows it
    puts first are the large ones: every row behind them lies in a lower bin of the selection
    (exponent and four mantissa bits of the squared norm), hence is smaller than all of them
    (up to the rounding of the fp32 sums)."""
    B, H, N = dest.shape
    norm = (k_values.astype(np.float64) ** 2).sum(-1)
    for b in range(B):
        for h in range(H):
            d = dest[b, h]
            assert np.array_equal(np.sort(d), np.arange(N))
            order = np.argsort(d)                      # order[j] = source row at destination j
            n_first = first_group_size(order)
            assert n_first >= min(FIRST, N)
            front, back = order[:n_first], order[n_first:]
            assert np.all(np.diff(front) > 0) and (back.size == 0 or np.all(np.diff(back) > 0))   # stable
            if back.size:
                assert norm[b, h, front].min() >= norm[b, h, back].max() * (1 - 1e-3)


def first_group_size(order):
    """A stable partition is two increasing runs; the first ends at the first descent (or the
    whole head is one run: nothing was behind the front group, or every row was in it)."""
    descents = np.nonzero(np.diff(order) < 0)[0]
    assert descents.size <= 1
    return int(descents[0]) + 1 if descents.size else order.size


@pytest.mark.parametrize("cfg,B,H,n,m,half", [("C3", 1, 3, 3000, 300, False), ("C2", 2, 2, 1500, 0, False),
                                              ("C3", 1, 2, 200, 17, False), ("C5", 1, 2, 2500, 129, True)])
def test_ordered_quantization_matches_the_oracle_under_the_map(cfg, B, H, n, m, half):
    w = dataclasses.replace(W.CONFIGS[cfg].scaled(n, m), B=B, H=H)
    g = W.generate(w)
    if half:
        g = {k: np.ascontiguousarray(bf16_bits_to_f64(v).astype(np.float16)).view(np.uint16) for k, v in g.items()}
    dtype16 = "fp16" if half else "bf16"
    tdt = torch.float16 if half else torch.bfloat16
    x = {k: dev16(v, tdt) for k, v in g.items()}
    ws = api.new_workspace(w.B, w.H)
    before = api.launch_count()
    o = api.quantize_qkv(x["q_train"], x["k"], x["v"], x["q_test"] if m else None, ws, order_keys=True)
    assert api.launch_count() - before == 3            # maximum (with the key norms), order, conversion
    assert api.last_device_status(ws) == (0, 0)
    dest = o["key_dest"].cpu().numpy().astype(np.int64)
    k_values = x["k"].float().cpu().numpy()
    check_map(dest, k_values)
    q8, sq = oracle.quantize(g["q_train"], dtype16=dtype16)
    k8, sk = oracle.quantize(g["k"], dtype16=dtype16)
    v8, sv = oracle.quantize(g["v"], dtype16=dtype16)
    assert np.array_equal(o["q8"].cpu().numpy(), q8)
    for name, ref, s_ref in (("k8", k8, sk), ("v8", v8, sv)):
        got = o[name].cpu().numpy()
        moved = np.empty_like(ref)
        np.put_along_axis(moved, dest[..., None].repeat(w.d, -1), ref, axis=2)      # moved[dest[r]] = ref[r]
        assert np.array_equal(got, moved), name
        assert np.array_equal(o["s" + name[0]].cpu().numpy(), s_ref)
    t8 = None
    if m:
        t8, _ = oracle.quantize(g["q_test"], scale_in=sq, dtype16=dtype16)
        assert np.array_equal(o["t8"].cpu().numpy(), t8)
    # attention over the reordered keys against the oracle over the original ones
    o_tr, o_te = api.icl_forward_fp8(o["q8"], o["t8"] if m else None, o["k8"], o["v8"], o["sq"], o["sk"], o["sv"], ws,
                                     out_dtype=tdt)
    assert api.last_device_status(ws) == (0, 0)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    for name, out, q, nq in (("train", o_tr, q8, n), ("test", o_te, t8, m)):
        if nq == 0:
            continue
        rows = sample_rows(nq, 24, w.seed)
        A, Abs, Bnd = oracle.icl_attention_rows(q, k8, v8, rows, sq=sq, sk=sk, sv=sv)
        check_fp8_attention(f64(out[:, :, torch.from_numpy(rows).cuda()]), A, Abs, Bnd, diffuse=False,
                            label=f"ordered keys {cfg}/{name}", named_config=False)
    # the same map applied to the 16-bit tensors
    k_moved = api.reorder_rows(x["k"], o["key_dest"])
    ref = np.empty_like(g["k"])
    np.put_along_axis(ref, dest[..., None].repeat(w.d, -1), g["k"], axis=2)
    assert np.array_equal(k_moved.view(torch.int16).cpu().numpy().view(np.uint16), ref)


def test_equal_norms_leave_the_order_alone_and_large_rows_come_first():
    B, H, N, d = 1, 2, 1000, 64
    torch.manual_seed(3)
    k = torch.ones((B, H, N, d), dtype=torch.bfloat16, device="cuda")
    k[0, 1] = torch.randn((N, d), device="cuda").to(torch.bfloat16) * 0.01
    big = torch.tensor([7, 500, 999], device="cuda")
    k[0, 1, big] *= 100.0
    q = torch.randn((B, H, N, d), device="cuda").to(torch.bfloat16)
    ws = api.new_workspace(B, H)
    o = api.quantize_qkv(q, k, q, None, ws, order_keys=True)
    dest = o["key_dest"].cpu().numpy()
    assert np.array_equal(dest[0, 0], np.arange(N))                       # one bin: everything "first", in place
    check_map(dest.astype(np.int64), k.float().cpu().numpy())
    # the three large rows are in the group that leads (in their old order)
    n_first = first_group_size(np.argsort(dest[0, 1]))
    assert FIRST <= n_first < N and all(dest[0, 1, r] < n_first for r in (7, 500, 999))
    assert dest[0, 1, 7] < dest[0, 1, 500] < dest[0, 1, 999]


def test_argument_errors():
    B, H, N, d = 1, 2, 300, 64
    x = torch.zeros((B, H, N, d), dtype=torch.bfloat16, device="cuda")
    ws = api.new_workspace(B, H)
    c8 = torch.empty((B, H, N, d), dtype=torch.uint8, device="cuda")
    s = torch.empty((B, H), dtype=torch.float32, device="cuda")
    lib = api.load()
    import ctypes
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = lib.fp8attn_quantize_qkv_ordered(p(x), p(x), p(x), None, B, H, N, 0, d, p(c8), p(c8), p(c8), None, p(s), p(s),
                                          p(s), None, 0, p(ws), ws.numel(), None)
    assert rc == api.ERR_INVALID_ARG                                      # no map to write to
    dest = torch.zeros((B, H, N), dtype=torch.int32, device="cuda")
    rc = lib.fp8attn_reorder_rows(p(x), B, H, N, d, p(dest), p(x), None)
    assert rc == api.ERR_INVALID_ARG                                      # in place
    torch.cuda.synchronize()
