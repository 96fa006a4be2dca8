"""The C-ABI library builds, loads on a machine without a GPU, and exports every
function that include/fp8attn.h declares (no compute calls here)."""
import ctypes
import os
import re

from paper_2609_13031_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b([a-z0-9_]+attn_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_loads_and_exports_header_symbols():
    build.build_cuda()
    lib = ctypes.CDLL(api.LIB_PATH)
    names = declared_functions()
    assert set(api.EXPORTS) <= set(names)
    assert len(names) >= 7
    for n in names:
        assert hasattr(lib, n), n


def test_host_only_entry_points():
    api.load()
    assert api.status_string(0) == "ok"
    assert "timed out" in api.status_string(api.ERR_TIMEOUT)
    assert api.workspace_bytes(1, 8) >= 256 + 32
    assert api.workspace_bytes(4, 4) % 256 == 0
    assert api.workspace_bytes(0, 4) == 0


def test_host_step_plan_is_host_only_arithmetic():
    """Chunking of the host-to-host step: whole heads, at most 8 chunks, one chunk for small
    calls or on request; two buffer sets when pipelined, so the scratch shrinks with chunking."""
    api.load()
    c3 = (1, 8, 65536, 16384, 128)
    assert api.host_step_chunks(*c3) == 8 and api.host_step_chunks(*c3, api.HOST_ONE_CHUNK) == 1
    assert api.host_step_chunks(1, 2, 512, 128, 64) == 1                  # small: nothing to overlap
    assert api.host_step_chunks(4, 4, 262144, 65536, 64) == 8             # 16 heads, two per chunk
    assert api.host_step_chunks(1, 11, 8192, 1100, 128) == 6              # ragged last chunk
    assert api.host_step_chunks(1, 1, 1 << 20, 0, 64) == 1                # one head cannot be cut
    one = api.host_step_scratch_bytes(*c3, api.HOST_ONE_CHUNK)
    piped = api.host_step_scratch_bytes(*c3)
    per_head = (3 * 65536 + 16384) * 128 * (2 + 1) + (65536 + 16384) * 128 * 2   # inputs, codes, outputs
    assert one >= 8 * per_head and 2 * per_head <= piped < one / 2
    assert one % 256 == 0 and piped % 256 == 0
    assert api.host_step_scratch_bytes(1, 8, 0, 16, 64) == 0 and api.host_step_scratch_bytes(1, 8, 64, 16, 96) == 0


def test_dispatch_gate_matches_the_paper_constant():
    import os
    from helpers import read_golden_table
    gold = dict(read_golden_table(os.path.join(ROOT, "tests", "golden", "paper_constants.txt")))
    gate = int(float(gold["fp8_gate_train_rows"]))          # Method section: N > 8192
    assert api.GATE_TRAIN_ROWS == gate
    assert not api.gate_use_fp8(gate) and api.gate_use_fp8(gate + 1)
    assert not api.gate_use_fp8(1) and api.gate_use_fp8(1 << 20)


def test_argument_checks_run_on_the_host_before_anything_touches_a_gpu():
    """Every entry point validates its arguments first, so the error codes can be checked on
    a machine without a GPU.  Pointers here are fake, suitably aligned addresses: a call that
    fails validation must not dereference or launch anything."""
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("fake pointers are only ever passed where no GPU could be reached")
    lib = api.load()
    P, WS = 0x10000, 0x20000                      # 16- and 256-byte aligned fake device addresses
    ws_bytes = api.workspace_bytes(1, 2)
    q = lambda *a: lib.fp8attn_quantize(*a)
    # shape and pointer checks of the quantizer
    assert q(P, 0, 2, 8, 64, None, P, P, WS, ws_bytes, None) == api.ERR_INVALID_ARG      # B = 0
    assert q(P, 1, 2, 8, 96, None, P, P, WS, ws_bytes, None) == api.ERR_UNSUPPORTED      # d = 96
    assert q(P, 1, 2, -1, 64, None, P, P, WS, ws_bytes, None) == api.ERR_INVALID_ARG     # rows < 0
    assert q(None, 1, 2, 8, 64, None, P, P, WS, ws_bytes, None) == api.ERR_INVALID_ARG   # no input
    assert q(P + 2, 1, 2, 8, 64, None, P, P, WS, ws_bytes, None) == api.ERR_INVALID_ARG  # misaligned
    assert q(P, 1, 2, 8, 64, None, P, None, WS, ws_bytes, None) == api.ERR_INVALID_ARG   # no scale at all
    assert q(P, 1, 2, 8, 64, None, P, P, None, ws_bytes, None) == api.ERR_WORKSPACE
    assert q(P, 1, 2, 8, 64, None, P, P, WS + 16, ws_bytes, None) == api.ERR_WORKSPACE   # misaligned
    assert q(P, 1, 2, 8, 64, None, P, P, WS, ws_bytes - 1, None) == api.ERR_WORKSPACE    # too small
    assert lib.fp8attn_quantize_ex(P, 1, 2, 8, 64, None, P, P, 0x40, WS, ws_bytes, None) == api.ERR_INVALID_ARG
    # the fused forward
    f = lambda *a: lib.fp8attn_icl_forward(*a)
    ok = [P, P, P, P, P, P, P, 1, 2, 8, 4, 64, 0.0, P, P, WS, ws_bytes, None]
    def bad(i, v):
        a = list(ok)
        a[i] = v
        return f(*a)
    assert bad(0, None) == api.ERR_INVALID_ARG         # train queries missing
    assert bad(1, None) == api.ERR_INVALID_ARG         # test queries missing although n_test > 0
    assert bad(4, None) == api.ERR_INVALID_ARG         # a scale missing
    assert bad(9, 0) == api.ERR_INVALID_ARG            # n_train = 0
    assert bad(10, -1) == api.ERR_INVALID_ARG          # n_test < 0
    assert bad(11, 256) == api.ERR_UNSUPPORTED         # head dimension
    assert bad(12, float("nan")) == api.ERR_INVALID_ARG
    assert bad(14, None) == api.ERR_INVALID_ARG        # test output missing
    assert bad(16, 0) == api.ERR_WORKSPACE
    # allocation-free quantizer: its own size limit
    assert lib.fp8attn_quantize_noalloc(P, 1, api.NOALLOC_MAX_HEADS + 1, 8, 64, None, P, P, None) == api.ERR_TOO_LARGE
    # arguments in order, but no GPU: the call reports it; nothing falls back to the CPU
    assert f(*ok) in (api.ERR_CUDA, api.ERR_UNSUPPORTED)
    assert q(P, 1, 2, 8, 64, None, P, P, WS, ws_bytes, None) in (api.ERR_CUDA, api.ERR_UNSUPPORTED)
