"""The host-to-host step (fp8attn_icl_step_host): copies, quantization and both attention
calls pipelined over chunks of heads.  Checked against the oracle (quantization of the same
host tensors, exact attention on sampled rows) and, bit for bit, against the device-pointer
calls made chunk by chunk."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f64, check_fp8_attention, sample_rows
from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def host16(bits, dtype=torch.bfloat16):
    return torch.from_numpy(bits.view(np.int16)).view(dtype).pin_memory()


def f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def shape_of(w):
    return (w.B, w.H, w.n_train, w.n_test, w.d)


def run_host_step(w, g, flags=0, dtype=torch.bfloat16):
    x = {k: host16(v, dtype) for k, v in g.items()}
    nbytes = api.host_step_scratch_bytes(*shape_of(w), flags | (api.HOST_FP16 if dtype == torch.float16 else 0))
    assert nbytes > 0
    # the scratch starts out dirty: the call must not depend on its contents
    scratch = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device="cuda")
    o_tr, o_te = api.icl_step_host(x["q_train"], x["k"], x["v"], x["q_test"] if w.n_test else None, scratch,
                                   flags=flags)
    assert api.host_step_status(scratch, *shape_of(w), flags | (api.HOST_FP16 if dtype == torch.float16 else 0)) == (0, 0)
    return x, o_tr, o_te


def device_reference(w, x, chunk_heads):
    """The device-pointer calls on each chunk of heads (B = 1, the chunk's heads), as the header
    says the host step computes."""
    BH = w.B * w.H
    flat = {k: v.reshape(1, BH, v.shape[2], w.d) for k, v in x.items()}
    outs_tr, outs_te = [], []
    for h0 in range(0, BH, chunk_heads):
        sl = slice(h0, min(h0 + chunk_heads, BH))
        g = sl.stop - sl.start
        dev = {k: v[:, sl].contiguous().cuda() for k, v in flat.items()}
        ws = api.new_workspace(1, g, n_train=w.n_train, n_test=w.n_test, d=w.d)
        o = api.quantize_qkv(dev["q_train"], dev["k"], dev["v"], dev["q_test"] if w.n_test else None, ws)
        o_tr, o_te = api.icl_forward_fp8(o["q8"], o["t8"] if w.n_test else None, o["k8"], o["v8"], o["sq"], o["sk"],
                                         o["sv"], ws, flags=api.SPLIT_TAIL, out_dtype=dev["k"].dtype)
        assert api.last_device_status(ws) == (0, 0)
        outs_tr.append(o_tr.cpu())
        outs_te.append(None if o_te is None else o_te.cpu())
    tr = torch.cat(outs_tr, dim=1).reshape(w.B, w.H, w.n_train, w.d)
    te = torch.cat(outs_te, dim=1).reshape(w.B, w.H, w.n_test, w.d) if w.n_test else None
    return tr, te


def check_against_oracle(w, g, o_tr, o_te, n_sample, dtype16="bf16"):
    q8, sq = oracle.quantize(g["q_train"], dtype16=dtype16)
    k8, sk = oracle.quantize(g["k"], dtype16=dtype16)
    v8, sv = oracle.quantize(g["v"], dtype16=dtype16)
    for name, out, nq in (("train", o_tr, w.n_train), ("test", o_te, w.n_test)):
        if nq == 0:
            assert out is None
            continue
        src = q8 if name == "train" else oracle.quantize(g["q_test"], scale_in=sq, dtype16=dtype16)[0]
        rows = sample_rows(nq, n_sample, w.seed)
        A, Abs, Bnd = oracle.icl_attention_rows(src, k8, v8, rows, sq=sq, sk=sk, sv=sv)
        check_fp8_attention(f64(out[:, :, torch.from_numpy(rows)]), A, Abs, Bnd, diffuse=False,
                            label=f"host step {w.name}/{name}", named_config=False)


@pytest.mark.parametrize("cfg,B,H,n,m", [("C1", 1, 2, 512, 128), ("C3", 2, 3, 700, 130), ("C4", 1, 4, 1000, 0)])
def test_small_call_one_chunk(cfg, B, H, n, m):
    w = dataclasses.replace(W.CONFIGS[cfg].scaled(n, m), B=B, H=H)
    assert api.host_step_chunks(*shape_of(w)) == 1
    g = W.generate(w)
    x, o_tr, o_te = run_host_step(w, g)
    torch.cuda.synchronize()
    ref_tr, ref_te = device_reference(w, x, w.B * w.H)
    assert torch.equal(o_tr, ref_tr)
    assert (o_te is None and ref_te is None) or torch.equal(o_te, ref_te)
    check_against_oracle(w, g, o_tr, o_te, n_sample=48)


@pytest.mark.parametrize("H,expect_chunks,chunk_heads", [(6, 6, 1), (11, 6, 2)])
def test_pipelined_chunks(H, expect_chunks, chunk_heads):
    # large enough to be cut into chunks; with 11 heads the last chunk holds a single head
    w = dataclasses.replace(W.CONFIGS["C3"].scaled(8192, 1100), B=1, H=H)
    assert api.host_step_chunks(*shape_of(w)) == expect_chunks
    assert api.host_step_chunks(*shape_of(w), api.HOST_ONE_CHUNK) == 1
    g = W.generate(w)
    x, o_tr, o_te = run_host_step(w, g)
    torch.cuda.synchronize()
    ref_tr, ref_te = device_reference(w, x, chunk_heads)
    assert torch.equal(o_tr, ref_tr) and torch.equal(o_te, ref_te)
    check_against_oracle(w, g, o_tr, o_te, n_sample=24)
    # the unpipelined form of the same call: same criteria (the tail split may differ)
    _, p_tr, p_te = run_host_step(w, g, flags=api.HOST_ONE_CHUNK)
    torch.cuda.synchronize()
    check_against_oracle(w, g, p_tr, p_te, n_sample=24)


def test_host_step_with_ordered_keys():
    # FP8ATTN_HOST_ORDER_KEYS: every chunk quantizes with the keys of largest norm first; the
    # result is attention over the same keys, so the oracle criteria are the same
    w = dataclasses.replace(W.CONFIGS["C3"].scaled(8192, 1100), B=1, H=6)
    assert api.host_step_chunks(*shape_of(w), api.HOST_ORDER_KEYS) == 6
    assert api.host_step_scratch_bytes(*shape_of(w), api.HOST_ORDER_KEYS) > api.host_step_scratch_bytes(*shape_of(w))
    g = W.generate(w)
    _, o_tr, o_te = run_host_step(w, g, flags=api.HOST_ORDER_KEYS)
    torch.cuda.synchronize()
    check_against_oracle(w, g, o_tr, o_te, n_sample=24)
    _, p_tr, p_te = run_host_step(w, g)
    torch.cuda.synchronize()
    assert not torch.equal(o_tr, p_tr)          # another order of the online softmax


def test_fp16_tensors():
    w = dataclasses.replace(W.CONFIGS["C2"].scaled(900, 200), B=1, H=3)
    g = {k: np.ascontiguousarray(bf16_bits_to_f64(v).astype(np.float16)).view(np.uint16)
         for k, v in W.generate(w).items()}
    x, o_tr, o_te = run_host_step(w, g, dtype=torch.float16)
    torch.cuda.synchronize()
    assert o_tr.dtype == torch.float16 and o_te.dtype == torch.float16
    ref_tr, ref_te = device_reference(w, x, w.B * w.H)
    assert torch.equal(o_tr, ref_tr) and torch.equal(o_te, ref_te)
    check_against_oracle(w, g, o_tr, o_te, n_sample=32, dtype16="fp16")


def test_calls_in_flight_on_two_streams():
    # two calls, two streams, own scratch each: the copies and kernels of one overlap the other's
    w = dataclasses.replace(W.CONFIGS["C3"].scaled(8192, 1024), B=1, H=6)
    ga, gb = W.generate(w), W.generate(dataclasses.replace(w, seed=w.seed + 100))
    xa = {k: host16(v) for k, v in ga.items()}
    xb = {k: host16(v) for k, v in gb.items()}
    nbytes = api.host_step_scratch_bytes(*shape_of(w))
    sa, sb = torch.empty(nbytes, dtype=torch.uint8, device="cuda"), torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    st_a, st_b = torch.cuda.Stream(), torch.cuda.Stream()
    res = []
    for rep in range(2):        # the second pair is enqueued while the first is still running
        with torch.cuda.stream(st_a):
            res.append((xa, api.icl_step_host(xa["q_train"], xa["k"], xa["v"], xa["q_test"], sa)))
        with torch.cuda.stream(st_b):
            res.append((xb, api.icl_step_host(xb["q_train"], xb["k"], xb["v"], xb["q_test"], sb)))
    torch.cuda.synchronize()
    for scratch in (sa, sb):
        assert api.host_step_status(scratch, *shape_of(w)) == (0, 0)
    refs = {id(xa): device_reference(w, xa, 1), id(xb): device_reference(w, xb, 1)}
    for x, (tr, te) in res:
        assert torch.equal(tr, refs[id(x)][0]) and torch.equal(te, refs[id(x)][1])


def test_argument_errors():
    w = dataclasses.replace(W.CONFIGS["C1"], B=1, H=2)
    g = W.generate(w)
    x = {k: host16(v) for k, v in g.items()}
    nbytes = api.host_step_scratch_bytes(*shape_of(w))
    scratch = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.Fp8AttnError) as e:
        api.icl_step_host(x["q_train"], x["k"], x["v"], x["q_test"], scratch[: nbytes - 256])
    assert e.value.status == api.ERR_WORKSPACE
    with pytest.raises(api.Fp8AttnError) as e:
        api.icl_step_host(x["q_train"], x["k"], x["v"], x["q_test"], scratch, flags=64)
    assert e.value.status == api.ERR_INVALID_ARG
    assert api.host_step_scratch_bytes(1, 2, 512, 128, 96) == 0   # unsupported head size
    assert api.host_step_chunks(1, 2, 0, 128, 64) == 0            # no train rows
    torch.cuda.synchronize()
