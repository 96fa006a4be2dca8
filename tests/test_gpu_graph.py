"""The hot path inside a CUDA graph: every entry point only enqueues work on the
caller's stream (no allocation, no host synchronisation), so a step can be captured
once and replayed on new data in the same buffers."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2609_13031_b200 import api
from paper_2609_13031_b200 import workloads as W

pytestmark = pytest.mark.gpu


def dev16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def test_step_replays_from_a_cuda_graph():
    w = W.CONFIGS["C2"].scaled(1500, 300)
    first = {k: dev16(v) for k, v in W.generate(w).items()}
    second = {k: dev16(v) for k, v in W.generate(dataclasses.replace(w, seed=77)).items()}
    ws = api.new_workspace(w.B, w.H)
    x = {k: torch.empty_like(v) for k, v in first.items()}
    q = api.quantize_qkv(first["q_train"], first["k"], first["v"], first["q_test"], ws)   # buffers + warm-up
    o_tr = torch.empty((w.B, w.H, w.n_train, w.d), dtype=torch.bfloat16, device="cuda")
    o_te = torch.empty((w.B, w.H, w.n_test, w.d), dtype=torch.bfloat16, device="cuda")

    def step():
        api.quantize_qkv(x["q_train"], x["k"], x["v"], x["q_test"], ws, out=q)
        api.icl_forward_fp8(q["q8"], q["t8"], q["k8"], q["v8"], q["sq"], q["sk"], q["sv"], ws,
                            out_train=o_tr, out_test=o_te)

    # eager reference results for both data sets
    want = []
    for data in (first, second):
        for k in x:
            x[k].copy_(data[k])
        step()
        want.append((o_tr.clone(), o_te.clone(), q["sq"].clone()))
    torch.cuda.synchronize()

    launches = api.launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    per_step = api.launch_count() - launches
    assert per_step == 2                                   # one-launch quantizer, attention

    for data, (w_tr, w_te, w_sq) in zip((first, second), want):
        for k in x:
            x[k].copy_(data[k])
        o_tr.zero_()
        o_te.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(o_tr, w_tr) and torch.equal(o_te, w_te) and torch.equal(q["sq"], w_sq)
    assert not torch.equal(want[0][0], want[1][0])
    assert api.last_device_status(ws) == (0, 0)


def test_split_tail_step_replays_from_a_cuda_graph():
    """The key-split launch sequence (split blocks, main grid released early, combine) is
    capturable as well and replays bit-identically."""
    w = W.CONFIGS["C2"].scaled(4500, 500)
    x = {k: dev16(v) for k, v in W.generate(w).items()}
    ws = api.new_workspace(w.B, w.H, n_train=w.n_train, n_test=w.n_test, d=w.d)
    q = api.quantize_qkv(x["q_train"], x["k"], x["v"], x["q_test"], ws)
    o_tr = torch.empty((w.B, w.H, w.n_train, w.d), dtype=torch.bfloat16, device="cuda")
    o_te = torch.empty((w.B, w.H, w.n_test, w.d), dtype=torch.bfloat16, device="cuda")

    def step():
        api.icl_forward_fp8(q["q8"], q["t8"], q["k8"], q["v8"], q["sq"], q["sk"], q["sv"], ws,
                            out_train=o_tr, out_test=o_te, flags=api.SPLIT_TAIL)

    step()
    torch.cuda.synchronize()
    want = (o_tr.clone(), o_te.clone())
    launches = api.launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    assert api.launch_count() - launches == 3
    for _ in range(3):
        o_tr.zero_()
        o_te.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(o_tr, want[0]) and torch.equal(o_te, want[1])
    assert api.last_device_status(ws) == (0, 0)
