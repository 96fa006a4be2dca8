"""Python binding of libfp8attn.so (declared in ``include/fp8attn.h``).

Argument marshalling only: every function hands device pointers, sizes and the
current CUDA stream to the C-ABI entry point of the same name.  torch is used
for device memory and streams.  There is no fallback: if the CUDA library has
not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfp8attn.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = range(7)
NOALLOC_MAX_HEADS = 4096

EXPORTS = (
    "fp8attn_quantize", "fp8attn_icl_forward", "bf16attn_icl_forward",
    "fp8attn_workspace_bytes", "fp8attn_last_device_status", "fp8attn_status_string",
    "fp8attn_launch_count", "fp8attn_quantize_noalloc",
    "fp8attn_icl_forward_ex", "bf16attn_icl_forward_ex", "fp8attn_gate_use_fp8",
    "fp8attn_quantize_qkv", "fp8attn_quantize_qkv_ex", "fp8attn_perturb",
    "fp8attn_selftest_wait_timeout", "fp8attn_quantize_ex",
    "fp8attn_icl_step_host", "fp8attn_host_step_scratch_bytes", "fp8attn_host_step_chunks",
    "fp8attn_host_step_status", "fp8attn_attention_rows_per_cta",
    "fp8attn_quantize_qkv_ordered", "fp8attn_reorder_rows",
)
# flags of fp8attn_quantize_ex / fp8attn_quantize_qkv_ex
QUERY_SCALE_FROM_ALL_ROWS = 1
INPUT_FP16 = 2
SCALES_GIVEN = 4
QKV_TWO_LAUNCHES = 8
# flags of fp8attn_icl_forward_ex / bf16attn_icl_forward_ex
TEST_ROWS_USE_KV_HEAD0 = 1
TEST_ROWS_ONLY = 2
IO_FP16 = 4
SPLIT_TAIL = 8
GATE_TRAIN_ROWS = 8192
# flags of fp8attn_icl_step_host
HOST_ONE_CHUNK = 1
HOST_FP16 = 2
HOST_ORDER_KEYS = 4

_lib = None


class Fp8AttnError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status_string(status)} (status {status})")


def load() -> ctypes.CDLL:
    """Load the CUDA library; raises if it is missing (build it with
    ``python -m paper_2609_13031_b200.build`` or ``__graft_entry__.build()``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: the CUDA extension has not been built and there is no "
            "CPU fallback.  Run `python -m paper_2609_13031_b200.build`.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float,
                             ctypes.c_size_t)
    lib.fp8attn_quantize.restype = i32
    lib.fp8attn_quantize.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp, vp, sz, vp]
    lib.fp8attn_quantize_ex.restype = i32
    lib.fp8attn_quantize_ex.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp, ctypes.c_uint32, vp, sz, vp]
    lib.fp8attn_quantize_noalloc.restype = i32
    lib.fp8attn_quantize_noalloc.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp, vp]
    lib.fp8attn_icl_forward.restype = i32
    lib.fp8attn_icl_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i64, i32, f32,
                                        vp, vp, vp, sz, vp]
    u32 = ctypes.c_uint32
    lib.fp8attn_icl_forward_ex.restype = i32
    lib.fp8attn_icl_forward_ex.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i64, i64, i32, f32, u32,
                                           vp, vp, vp, sz, vp]
    lib.bf16attn_icl_forward_ex.restype = i32
    lib.bf16attn_icl_forward_ex.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, i32, f32, u32, vp, vp,
                                            vp, sz, vp]
    lib.fp8attn_quantize_qkv.restype = i32
    lib.fp8attn_quantize_qkv.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, i32, vp, vp, vp, vp,
                                         vp, vp, vp, vp, sz, vp]
    lib.fp8attn_quantize_qkv_ex.restype = i32
    lib.fp8attn_quantize_qkv_ex.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, i32, vp, vp, vp, vp,
                                            vp, vp, vp, u32, vp, sz, vp]
    lib.fp8attn_quantize_qkv_ordered.restype = i32
    lib.fp8attn_quantize_qkv_ordered.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, i32, vp, vp, vp, vp,
                                                 vp, vp, vp, vp, u32, vp, sz, vp]
    lib.fp8attn_reorder_rows.restype = i32
    lib.fp8attn_reorder_rows.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp]
    lib.fp8attn_perturb.restype = i32
    lib.fp8attn_perturb.argtypes = [vp, i32, i32, i64, i32, f32, ctypes.c_uint64, u32, vp, vp, vp, sz, vp]
    lib.fp8attn_selftest_wait_timeout.restype = i32
    lib.fp8attn_selftest_wait_timeout.argtypes = [vp, sz, u32, vp]
    lib.fp8attn_gate_use_fp8.restype = i32
    lib.fp8attn_gate_use_fp8.argtypes = [i64]
    lib.bf16attn_icl_forward.restype = i32
    lib.bf16attn_icl_forward.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, i32, f32, vp, vp, vp,
                                         sz, vp]
    lib.fp8attn_workspace_bytes.restype = sz
    lib.fp8attn_workspace_bytes.argtypes = [i32, i32, i64, i64, i32]
    lib.fp8attn_last_device_status.restype = i32
    lib.fp8attn_last_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.fp8attn_status_string.restype = ctypes.c_char_p
    lib.fp8attn_status_string.argtypes = [i32]
    lib.fp8attn_launch_count.restype = ctypes.c_uint64
    lib.fp8attn_launch_count.argtypes = []
    lib.fp8attn_attention_rows_per_cta.restype = i32
    lib.fp8attn_attention_rows_per_cta.argtypes = [i32, i32, i64, i64, i32, u32]
    lib.fp8attn_host_step_scratch_bytes.restype = sz
    lib.fp8attn_host_step_scratch_bytes.argtypes = [i32, i32, i64, i64, i32, u32]
    lib.fp8attn_host_step_chunks.restype = i32
    lib.fp8attn_host_step_chunks.argtypes = [i32, i32, i64, i64, i32, u32]
    lib.fp8attn_icl_step_host.restype = i32
    lib.fp8attn_icl_step_host.argtypes = [vp, vp, vp, vp, i32, i32, i64, i64, i32, f32, u32, vp, vp, vp, sz, vp]
    lib.fp8attn_host_step_status.restype = i32
    lib.fp8attn_host_step_status.argtypes = [vp, i32, i32, i64, i64, i32, u32, vp, ctypes.POINTER(ctypes.c_uint32)]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().fp8attn_status_string(int(status)).decode()


def launch_count() -> int:
    return int(load().fp8attn_launch_count())


def _ptr(t: torch.Tensor | None):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(fn: str, rc: int):
    if rc != OK:
        raise Fp8AttnError(fn, rc)


def workspace_bytes(B: int, H: int, n_train: int = 0, n_test: int = 0, d: int = 64) -> int:
    return int(load().fp8attn_workspace_bytes(B, H, n_train, n_test, d))


def new_workspace(B: int, H: int, device="cuda", n_train: int = 0, n_test: int = 0,
                  d: int = 64) -> torch.Tensor:
    """A zero-filled workspace tensor for tensors with B*H heads.  Given the sizes of an
    attention call (n_train > 0) it also holds the scratch that SPLIT_TAIL needs."""
    return torch.zeros(workspace_bytes(B, H, n_train, n_test, d), dtype=torch.uint8, device=device)


def _dims(x: torch.Tensor):
    assert x.dim() == 4 and x.is_cuda and x.is_contiguous(), "expected contiguous CUDA [B,H,rows,d]"
    return x.shape


def _is16(t: torch.Tensor) -> bool:
    return t.dtype in (torch.bfloat16, torch.float16)


def quantize(x: torch.Tensor, workspace: torch.Tensor, scale_in: torch.Tensor | None = None,
             out: torch.Tensor | None = None, scale_out: torch.Tensor | None = None):
    """fp8attn_quantize (bf16 input) / fp8attn_quantize_ex with FP8ATTN_INPUT_FP16 (fp16 input):
    [B,H,rows,d] -> (e4m3 codes as uint8 [B,H,rows,d], fp32 scale [B,H])."""
    B, H, rows, d = _dims(x)
    assert _is16(x)
    if out is None:
        out = torch.empty((B, H, rows, d), dtype=torch.uint8, device=x.device)
    if scale_out is None:
        scale_out = torch.empty((B, H), dtype=torch.float32, device=x.device)
    if scale_in is not None:
        assert scale_in.dtype == torch.float32 and scale_in.is_contiguous() and scale_in.numel() == B * H
    if x.dtype == torch.float16:
        rc = load().fp8attn_quantize_ex(_ptr(x), B, H, rows, d, _ptr(scale_in), _ptr(out),
                                        _ptr(scale_out), INPUT_FP16, _ptr(workspace),
                                        workspace.numel(), _stream())
        _check("fp8attn_quantize_ex", rc)
        return out, scale_out
    rc = load().fp8attn_quantize(_ptr(x), B, H, rows, d, _ptr(scale_in), _ptr(out), _ptr(scale_out),
                                 _ptr(workspace), workspace.numel(), _stream())
    _check("fp8attn_quantize", rc)
    return out, scale_out


def quantize_noalloc(x: torch.Tensor, out: torch.Tensor, scale_out: torch.Tensor,
                     scale_in: torch.Tensor | None = None):
    """fp8attn_quantize_noalloc: like ``quantize`` but with no workspace; the
    scratch it needs is built into the library.  For hosts that may not allocate
    device memory, the caller passes every buffer (``out``: uint8 like ``x``,
    ``scale_out``: fp32 [B,H]) and this wrapper allocates nothing either.  At
    most ``NOALLOC_MAX_HEADS`` heads; calls on one device must not overlap."""
    B, H, rows, d = _dims(x)
    assert x.dtype == torch.bfloat16 and out.dtype == torch.uint8 and out.shape == x.shape
    assert scale_out.dtype == torch.float32 and scale_out.numel() == B * H
    rc = load().fp8attn_quantize_noalloc(_ptr(x), B, H, rows, d, _ptr(scale_in), _ptr(out),
                                         _ptr(scale_out), _stream())
    _check("fp8attn_quantize_noalloc", rc)
    return out, scale_out


def quantize_qkv(q_train, k, v, q_test, workspace, out=None, flags: int = 0, order_keys: bool = False):
    """fp8attn_quantize_qkv: all four quantizations of one attention call in two
    launches.  Returns dict(q8, k8, v8, t8, sq, sk, sv); ``out`` may supply those
    tensors preallocated.  With SCALES_GIVEN, ``out`` must hold sq, sk, sv and they
    are read instead of written (one launch).  ``order_keys``:
    fp8attn_quantize_qkv_ordered, K8 and V8 come out with the keys of largest norm first and
    the dict also holds ``key_dest`` (int32 [B,H,n_train], the row each key moved to)."""
    if flags & SCALES_GIVEN:
        assert out is not None and all(n in out for n in ("sq", "sk", "sv"))
    B, H, n_train, d = _dims(k)
    n_test = 0 if q_test is None else q_test.shape[2]
    dev = k.device
    for t in (q_train, k, v) + (() if q_test is None else (q_test,)):
        assert t.dtype == k.dtype and _is16(t)
    if k.dtype == torch.float16:
        flags |= INPUT_FP16
    o = dict(out or {})
    for name, rows in (("q8", n_train), ("k8", n_train), ("v8", n_train), ("t8", n_test)):
        if name not in o:
            o[name] = torch.empty((B, H, rows, d), dtype=torch.uint8, device=dev)
    for name in ("sq", "sk", "sv"):
        if name not in o:
            o[name] = torch.empty((B, H), dtype=torch.float32, device=dev)
    args = (_ptr(q_train), _ptr(k), _ptr(v), _ptr(q_test) if n_test else None, B, H, n_train, n_test, d,
            _ptr(o["q8"]), _ptr(o["k8"]), _ptr(o["v8"]), _ptr(o["t8"]) if n_test else None,
            _ptr(o["sq"]), _ptr(o["sk"]), _ptr(o["sv"]))
    if order_keys:
        if "key_dest" not in o:
            o["key_dest"] = torch.empty((B, H, n_train), dtype=torch.int32, device=dev)
        rc = load().fp8attn_quantize_qkv_ordered(*args, _ptr(o["key_dest"]), int(flags), _ptr(workspace),
                                                 workspace.numel(), _stream())
        _check("fp8attn_quantize_qkv_ordered", rc)
    elif flags:
        rc = load().fp8attn_quantize_qkv_ex(*args, int(flags), _ptr(workspace), workspace.numel(), _stream())
        _check("fp8attn_quantize_qkv_ex", rc)
    else:
        rc = load().fp8attn_quantize_qkv(*args, _ptr(workspace), workspace.numel(), _stream())
        _check("fp8attn_quantize_qkv", rc)
    return o


def reorder_rows(x: torch.Tensor, dest: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """fp8attn_reorder_rows: out[b,h,dest[b,h,r],:] = x[b,h,r,:] for a 16-bit tensor."""
    B, H, rows, d = _dims(x)
    assert _is16(x) and dest.dtype == torch.int32 and dest.is_cuda and dest.is_contiguous() and dest.numel() == B * H * rows
    if out is None:
        out = torch.empty_like(x)
    rc = load().fp8attn_reorder_rows(_ptr(x), B, H, rows, d, _ptr(dest), _ptr(out), _stream())
    _check("fp8attn_reorder_rows", rc)
    return out


def perturb(x: torch.Tensor, epsilon: float, seed: int, stream_id: int, workspace: torch.Tensor,
            out: torch.Tensor | None = None, rho_out: torch.Tensor | None = None):
    """fp8attn_perturb: x + epsilon * rho[b,h] * N(0,1) per head (paper Eq. 3); returns (out, rho)."""
    B, H, rows, d = _dims(x)
    assert x.dtype == torch.bfloat16
    if out is None:
        out = torch.empty_like(x)
    if rho_out is None:
        rho_out = torch.empty((B, H), dtype=torch.float32, device=x.device)
    rc = load().fp8attn_perturb(_ptr(x), B, H, rows, d, float(epsilon), int(seed), int(stream_id),
                                _ptr(out), _ptr(rho_out), _ptr(workspace), workspace.numel(), _stream())
    _check("fp8attn_perturb", rc)
    return out, rho_out


def selftest_wait_timeout(workspace: torch.Tensor, limit_us: int = 1000) -> None:
    """fp8attn_selftest_wait_timeout: make one bounded device wait expire on purpose."""
    rc = load().fp8attn_selftest_wait_timeout(_ptr(workspace), workspace.numel(), int(limit_us), _stream())
    _check("fp8attn_selftest_wait_timeout", rc)


def attention_rows_per_cta(B: int, H: int, n_train: int, n_test: int, d: int, flags: int = 0) -> int:
    """fp8attn_attention_rows_per_cta: 256 or 384 query rows per CTA for a call of these sizes."""
    return int(load().fp8attn_attention_rows_per_cta(B, H, n_train, n_test, d, int(flags)))


def gate_use_fp8(n_train: int) -> bool:
    """fp8attn_gate_use_fp8: the paper's N > 8192 dispatch rule."""
    return bool(load().fp8attn_gate_use_fp8(int(n_train)))


def icl_forward_fp8(q_train, q_test, k, v, scale_q, scale_k, scale_v, workspace,
                    softmax_scale: float = 0.0, out_train=None, out_test=None, flags: int = 0,
                    out_dtype=torch.bfloat16):
    """fp8attn_icl_forward (flags == 0) / fp8attn_icl_forward_ex on uint8 e4m3
    tensors; returns (out_train, out_test) in ``out_dtype`` (bf16, or fp16 =
    FP8ATTN_IO_FP16).  With TEST_ROWS_ONLY ``q_train`` may be None and out_train
    is None."""
    B, H, n_train, d = _dims(k)
    n_test = 0 if q_test is None else q_test.shape[2]
    test_only = bool(flags & TEST_ROWS_ONLY)
    for t in (k, v) + (() if test_only else (q_train,)):
        assert t.dtype == torch.uint8
    for t in (out_train, out_test):
        if t is not None:
            out_dtype = t.dtype
    assert out_dtype in (torch.bfloat16, torch.float16)
    if out_dtype == torch.float16:
        flags |= IO_FP16
    if out_train is None and not test_only:
        out_train = torch.empty((B, H, n_train, d), dtype=out_dtype, device=k.device)
    if out_test is None and n_test > 0:
        out_test = torch.empty((B, H, n_test, d), dtype=out_dtype, device=k.device)
    if test_only:
        q_train, out_train = None, None
    if flags:
        rc = load().fp8attn_icl_forward_ex(
            _ptr(q_train), _ptr(q_test) if n_test else None, _ptr(k), _ptr(v),
            _ptr(scale_q), _ptr(scale_k), _ptr(scale_v), B, H, n_train, n_test, d,
            float(softmax_scale), int(flags), _ptr(out_train), _ptr(out_test) if n_test else None,
            _ptr(workspace), workspace.numel(), _stream())
        _check("fp8attn_icl_forward_ex", rc)
        return out_train, out_test
    rc = load().fp8attn_icl_forward(
        _ptr(q_train), _ptr(q_test) if n_test else None, _ptr(k), _ptr(v),
        _ptr(scale_q), _ptr(scale_k), _ptr(scale_v), B, H, n_train, n_test, d,
        float(softmax_scale), _ptr(out_train), _ptr(out_test) if n_test else None,
        _ptr(workspace), workspace.numel(), _stream())
    _check("fp8attn_icl_forward", rc)
    return out_train, out_test


def icl_forward_bf16(q_train, q_test, k, v, workspace, softmax_scale: float = 0.0,
                     out_train=None, out_test=None, flags: int = 0):
    """bf16attn_icl_forward on bf16 tensors (or, with fp16 tensors, its
    FP8ATTN_IO_FP16 form); returns (out_train, out_test) in the input dtype.
    With TEST_ROWS_ONLY ``q_train`` may be None and out_train is None."""
    B, H, n_train, d = _dims(k)
    n_test = 0 if q_test is None else q_test.shape[2]
    test_only = bool(flags & TEST_ROWS_ONLY)
    assert _is16(k)
    for t in (v,) + (() if test_only else (q_train,)) + (() if q_test is None else (q_test,)):
        assert t.dtype == k.dtype
    if k.dtype == torch.float16:
        flags |= IO_FP16
    if out_train is None and not test_only:
        out_train = torch.empty((B, H, n_train, d), dtype=k.dtype, device=k.device)
    if out_test is None and n_test > 0:
        out_test = torch.empty((B, H, n_test, d), dtype=k.dtype, device=k.device)
    for t in (out_train, out_test):
        assert t is None or t.dtype == k.dtype
    if test_only:
        q_train, out_train = None, None
    if flags:
        rc = load().bf16attn_icl_forward_ex(
            _ptr(q_train), _ptr(q_test) if n_test else None, _ptr(k), _ptr(v), B, H, n_train, n_test,
            d, float(softmax_scale), int(flags), _ptr(out_train), _ptr(out_test) if n_test else None,
            _ptr(workspace), workspace.numel(), _stream())
        _check("bf16attn_icl_forward_ex", rc)
        return out_train, out_test
    rc = load().bf16attn_icl_forward(
        _ptr(q_train), _ptr(q_test) if n_test else None, _ptr(k), _ptr(v), B, H, n_train, n_test, d,
        float(softmax_scale), _ptr(out_train), _ptr(out_test) if n_test else None,
        _ptr(workspace), workspace.numel(), _stream())
    _check("bf16attn_icl_forward", rc)
    return out_train, out_test


def last_device_status(workspace: torch.Tensor):
    """Synchronise the current stream; returns (status, detail) recorded by the kernels."""
    detail = ctypes.c_uint32(0)
    rc = load().fp8attn_last_device_status(_ptr(workspace), _stream(), ctypes.byref(detail))
    return int(rc), int(detail.value)


def _host_dims(q_train, k, v, q_test):
    assert k.dim() == 4 and not k.is_cuda and k.is_contiguous() and _is16(k), "expected contiguous host [B,H,rows,d]"
    for t in (q_train, v):
        assert t.shape == k.shape and t.dtype == k.dtype and not t.is_cuda and t.is_contiguous()
    B, H, n_train, d = k.shape
    n_test = 0
    if q_test is not None:
        assert q_test.dtype == k.dtype and not q_test.is_cuda and q_test.is_contiguous()
        assert q_test.shape[:2] == k.shape[:2] and q_test.shape[3] == d
        n_test = q_test.shape[2]
    return B, H, n_train, n_test, d


def host_step_scratch_bytes(B: int, H: int, n_train: int, n_test: int, d: int, flags: int = 0) -> int:
    return int(load().fp8attn_host_step_scratch_bytes(B, H, n_train, n_test, d, int(flags)))


def host_step_chunks(B: int, H: int, n_train: int, n_test: int, d: int, flags: int = 0) -> int:
    return int(load().fp8attn_host_step_chunks(B, H, n_train, n_test, d, int(flags)))


def icl_step_host(q_train, k, v, q_test, scratch: torch.Tensor, softmax_scale: float = 0.0, flags: int = 0,
                  out_train=None, out_test=None):
    """fp8attn_icl_step_host: quantize + both attention calls from HOST tensors (page-locked
    for overlap) to HOST results, pipelined over chunks of heads.  ``scratch``: uint8 CUDA
    tensor of at least ``host_step_scratch_bytes`` bytes.  Enqueues on the current stream and
    returns (out_train, out_test) host tensors that are complete once that stream has been
    synchronised."""
    B, H, n_train, n_test, d = _host_dims(q_train, k, v, q_test)
    if k.dtype == torch.float16:
        flags |= HOST_FP16
    if out_train is None:
        out_train = torch.empty(k.shape, dtype=k.dtype).pin_memory()
    if out_test is None and n_test > 0:
        out_test = torch.empty(q_test.shape, dtype=k.dtype).pin_memory()
    for t in (out_train, out_test):
        assert t is None or (not t.is_cuda and t.is_contiguous() and t.dtype == k.dtype)
    assert scratch.is_cuda and scratch.dtype == torch.uint8
    rc = load().fp8attn_icl_step_host(_ptr(q_train), _ptr(k), _ptr(v), _ptr(q_test) if n_test else None,
                                      B, H, n_train, n_test, d, float(softmax_scale), int(flags),
                                      _ptr(out_train), _ptr(out_test) if n_test else None,
                                      _ptr(scratch), scratch.numel(), _stream())
    _check("fp8attn_icl_step_host", rc)
    return out_train, out_test


def host_step_status(scratch: torch.Tensor, B: int, H: int, n_train: int, n_test: int, d: int, flags: int = 0):
    """Synchronise the current stream; (status, detail) of the workspaces of a host step."""
    detail = ctypes.c_uint32(0)
    rc = load().fp8attn_host_step_status(_ptr(scratch), B, H, n_train, n_test, d, int(flags), _stream(),
                                         ctypes.byref(detail))
    return int(rc), int(detail.value)


def icl_attention(q_train, q_test, k, v, workspace=None, softmax_scale: float = 0.0, flags: int = 0):
    """The whole hot path on bf16 inputs: quantize Q_train, K, V per head, quantize
    Q_test with the train-query scale, then the fused FP8 attention (``flags``: forward
    flags, e.g. SPLIT_TAIL)."""
    B, H, n_train, d = _dims(k)
    if workspace is None:
        workspace = new_workspace(B, H, k.device, n_train=n_train if flags & SPLIT_TAIL else 0, d=d)
    has_test = q_test is not None and q_test.shape[2] > 0
    o = quantize_qkv(q_train, k, v, q_test if has_test else None, workspace)
    q8, k8, v8, sq, sk, sv = o["q8"], o["k8"], o["v8"], o["sq"], o["sk"], o["sv"]
    t8 = o["t8"] if has_test else None
    return icl_forward_fp8(q8, t8, k8, v8, sq, sk, sv, workspace, softmax_scale, flags=flags,
                           out_dtype=k.dtype)


def icl_attention_arms(q_train, q_test, k, v, fp8_train: bool, fp8_test: bool, workspace=None,
                       softmax_scale: float = 0.0):
    """The arms of the paper's precision ablation: the train->train call and the
    test->train call each run either in FP8 or in 16 bits (n_test = 0 and
    TEST_ROWS_ONLY select one call).  Returns (out_train, out_test)."""
    B, H, _, _ = _dims(k)
    if workspace is None:
        workspace = new_workspace(B, H, k.device)
    assert q_test is not None and q_test.shape[2] > 0
    if fp8_train == fp8_test:
        if fp8_train:
            return icl_attention(q_train, q_test, k, v, workspace, softmax_scale)
        return icl_forward_bf16(q_train, q_test, k, v, workspace, softmax_scale)
    o = quantize_qkv(q_train, k, v, q_test, workspace)
    fp8 = (o["q8"], o["t8"], o["k8"], o["v8"], o["sq"], o["sk"], o["sv"])
    if fp8_train:
        out_train, _ = icl_forward_fp8(fp8[0], None, *fp8[2:], workspace, softmax_scale, out_dtype=k.dtype)
        _, out_test = icl_forward_bf16(None, q_test, k, v, workspace, softmax_scale, flags=TEST_ROWS_ONLY)
    else:
        out_train, _ = icl_forward_bf16(q_train, None, k, v, workspace, softmax_scale)
        _, out_test = icl_forward_fp8(None, fp8[1], *fp8[2:], workspace, softmax_scale,
                                      flags=TEST_ROWS_ONLY, out_dtype=k.dtype)
    return out_train, out_test


def icl_attention_gated(q_train, q_test, k, v, workspace=None, softmax_scale: float = 0.0):
    """The paper's final configuration: FP8 path only above the N > 8192 gate
    (fp8attn_gate_use_fp8), the 16-bit path below it."""
    B, H, n_train, _ = _dims(k)
    if workspace is None:
        workspace = new_workspace(B, H, k.device)
    if gate_use_fp8(n_train):
        return icl_attention(q_train, q_test, k, v, workspace, softmax_scale)
    has_test = q_test is not None and q_test.shape[2] > 0
    return icl_forward_bf16(q_train, q_test if has_test else None, k, v, workspace, softmax_scale)
