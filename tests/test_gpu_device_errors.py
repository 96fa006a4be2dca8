"""The device-side error path: a bounded wait that runs out is reported through the
workspace status words, the kernel returns normally, the error is sticky until it
has been read, and the context stays usable.  The wait is made to expire on a
barrier that nothing signals (no fault, trap or hang is involved)."""
import pytest
import torch

from paper_2609_13031_b200 import api

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_is_sticky_and_clears():
    ws = api.new_workspace(1, 2)
    assert api.last_device_status(ws) == (0, 0)
    api.selftest_wait_timeout(ws, limit_us=500)
    torch.cuda.synchronize()                                   # the kernel came back by itself
    # while the error is pending, an attention launch on this workspace does nothing
    q = torch.randint(0, 100, (1, 2, 256, 64), dtype=torch.uint8, device="cuda")
    s = torch.ones((1, 2), dtype=torch.float32, device="cuda")
    out = torch.full((1, 2, 256, 64), 7.0, dtype=torch.bfloat16, device="cuda")
    api.icl_forward_fp8(q, None, q, q, s, s, s, ws, out_train=out)
    torch.cuda.synchronize()
    assert torch.all(out == 7.0)
    status, detail = api.last_device_status(ws)
    assert status == api.ERR_TIMEOUT
    assert detail >> 24 == 11                                   # the self-test's wait id
    assert "timed out" in api.status_string(status)
    # read once -> cleared; the same workspace and context work again
    assert api.last_device_status(ws) == (0, 0)
    api.icl_forward_fp8(q, None, q, q, s, s, s, ws, out_train=out)
    assert api.last_device_status(ws) == (0, 0)
    assert not torch.all(out == 7.0) and torch.isfinite(out.float()).all()


def test_selftest_argument_checks():
    lib = api.load()
    ws = api.new_workspace(1, 1)
    assert lib.fp8attn_selftest_wait_timeout(ws.data_ptr(), ws.numel(), 0, None) == api.ERR_INVALID_ARG
    assert lib.fp8attn_selftest_wait_timeout(None, ws.numel(), 10, None) == api.ERR_WORKSPACE
