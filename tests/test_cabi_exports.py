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


def test_dispatch_gate_matches_the_paper_constant():
    import os
    from helpers import read_golden_table
    gold = dict(read_golden_table(os.path.join(ROOT, "tests", "golden", "paper_constants.txt")))
    gate = int(float(gold["fp8_gate_train_rows"]))          # Method section: N > 8192
    assert api.GATE_TRAIN_ROWS == gate
    assert not api.gate_use_fp8(gate) and api.gate_use_fp8(gate + 1)
    assert not api.gate_use_fp8(1) and api.gate_use_fp8(1 << 20)
