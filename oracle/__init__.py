"""CPU oracle for the FP8 ICL-attention path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes access to ``fp8attn_oracle.cpp`` (plain C++17, fp64, no BLAS).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product never does.  It shares no code with the CUDA path
and imports nothing from it.

Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns and FP8
tensors as ``uint8`` codes, both shaped ``[B, H, rows, d]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fp8attn_oracle.cpp")
_LIB = os.path.join(_HERE, "libfp8attn_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (seconds).  Returns the library path."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
           "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _AttnArgs(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("is_fp8", ctypes.c_int),
        ("sq", ctypes.c_void_p), ("sk", ctypes.c_void_p), ("sv", ctypes.c_void_p),
        ("B", ctypes.c_int), ("H", ctypes.c_int),
        ("nq", ctypes.c_int64), ("n_train", ctypes.c_int64), ("d", ctypes.c_int),
        ("alpha", ctypes.c_double),
        ("rows", ctypes.c_void_p), ("n_rows", ctypes.c_int64),
        ("mode", ctypes.c_int),
        ("A", ctypes.c_void_p), ("Abs", ctypes.c_void_p), ("Bnd", ctypes.c_void_p),
        ("nthreads", ctypes.c_int),
    ]


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.oracle_hardware_threads.restype = ctypes.c_int
            lib.oracle_e4m3_decode.restype = ctypes.c_double
            lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
            lib.oracle_e4m3_encode.restype = ctypes.c_uint8
            lib.oracle_e4m3_encode.argtypes = [ctypes.c_double]
            lib.oracle_e4m3_encode_array.restype = None
            lib.oracle_e4m3_encode_array.argtypes = [
                ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
            lib.oracle_quantize.restype = None
            lib.oracle_quantize.argtypes = [
                ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                ctypes.c_int]
            lib.oracle_quantize_ex.restype = None
            lib.oracle_quantize_ex.argtypes = [
                ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                ctypes.c_int]
            lib.oracle_half_to_float.restype = ctypes.c_float
            lib.oracle_half_to_float.argtypes = [ctypes.c_uint16]
            lib.oracle_icl_attention_rows.restype = None
            lib.oracle_icl_attention_rows.argtypes = [ctypes.POINTER(_AttnArgs)]
            lib.oracle_perturb.restype = None
            lib.oracle_perturb.argtypes = [
                ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                ctypes.c_double, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p,
                ctypes.c_int]
            row_args = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                        ctypes.c_float, ctypes.c_float, ctypes.c_int64,
                        ctypes.c_int64, ctypes.c_int, ctypes.c_double,
                        ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p]
            lib.oracle_softmax_row.restype = None
            lib.oracle_softmax_row.argtypes = row_args
            lib.oracle_lifted_p8_row.restype = None
            lib.oracle_lifted_p8_row.argtypes = row_args
            _lib = lib
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


# ---- codec -----------------------------------------------------------------

def e4m3_decode(code: int) -> float:
    return float(_load().oracle_e4m3_decode(int(code) & 0xFF))


def e4m3_encode(y: float) -> int:
    return int(_load().oracle_e4m3_encode(float(y)))


def e4m3_encode_array(y: np.ndarray) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.float32)
    out = np.empty(y.shape, dtype=np.uint8)
    _load().oracle_e4m3_encode_array(_ptr(y), y.size, _ptr(out))
    return out


def e4m3_decode_table() -> np.ndarray:
    """fp64 value of each of the 256 codes (NaN for 0x7F / 0xFF)."""
    return np.array([e4m3_decode(c) for c in range(256)], dtype=np.float64)


# ---- quantize (Eq. 2) --------------------------------------------------------

_DTYPE16 = {"bf16": 0, "fp16": 1}


def rounding_envelope(x: float) -> float:
    """The oracle's worst-case e4m3 rounding error at magnitude x (the envelope behind Bnd)."""
    lib = _load()
    lib.oracle_rounding_envelope.restype = ctypes.c_double
    lib.oracle_rounding_envelope.argtypes = [ctypes.c_double]
    return float(lib.oracle_rounding_envelope(float(x)))


def round_to_bf16(x: float) -> float:
    """The oracle's fp32 -> nearest bf16 (as a float), used for the e4m3-P mode's output."""
    lib = _load()
    lib.oracle_round_to_bf16.restype = ctypes.c_float
    lib.oracle_round_to_bf16.argtypes = [ctypes.c_float]
    return float(lib.oracle_round_to_bf16(float(x)))


def double_to_bf16_bits(v: float) -> int:
    """The oracle's fp64 -> nearest bf16 bit pattern, used by the perturbation."""
    lib = _load()
    lib.oracle_double_to_bf16_bits.restype = ctypes.c_uint16
    lib.oracle_double_to_bf16_bits.argtypes = [ctypes.c_double]
    return int(lib.oracle_double_to_bf16_bits(float(v)))


def half_to_float(bits: int) -> float:
    """Value of one IEEE fp16 bit pattern, by the format's definition."""
    return float(_load().oracle_half_to_float(int(bits) & 0xFFFF))


def quantize(x_bf16_bits: np.ndarray, scale_in: np.ndarray | None = None,
             nthreads: int | None = None, dtype16: str = "bf16"):
    """16-bit patterns [B,H,R,d] (bf16, or IEEE fp16 with dtype16="fp16")
    -> (codes uint8 [B,H,R,d], scale fp32 [B,H])."""
    x = np.ascontiguousarray(x_bf16_bits, dtype=np.uint16)
    B, H, R, d = x.shape
    codes = np.empty(x.shape, dtype=np.uint8)
    scale = np.empty((B, H), dtype=np.float32)
    s_in = None
    if scale_in is not None:
        s_in = np.ascontiguousarray(scale_in, dtype=np.float32).reshape(B, H)
    nt = nthreads or hardware_threads()
    _load().oracle_quantize_ex(_ptr(x), _DTYPE16[dtype16], B, H, R, d, _ptr(s_in), _ptr(codes),
                               _ptr(scale), nt)
    return codes, scale


# ---- attention (Eq. 1 over the dequantized operands) -------------------------

def icl_attention_rows(q, k, v, rows, *, sq=None, sk=None, sv=None,
                       alpha: float | None = None, mode: str = "exact",
                       nthreads: int | None = None, dtype16: str = "bf16"):
    """Attention outputs of selected query rows against ALL train keys.

    q: [B,H,nq,d], k/v: [B,H,N,d]; uint8 = FP8 codes (scales [B,H] required),
    uint16 = bf16 bits, or IEEE fp16 bits with dtype16="fp16" (no scales).
    ``rows``: 1-D int array of query rows,
    evaluated for every (b,h).  mode "exact": returns (A, Abs, Bnd) fp64
    [B,H,len(rows),d]; mode "p8": returns the two-pass e4m3-P result (A only,
    bf16-rounded values held in fp64).
    """
    q = np.ascontiguousarray(q)
    k = np.ascontiguousarray(k)
    v = np.ascontiguousarray(v)
    is_fp8 = q.dtype == np.uint8
    assert q.dtype == k.dtype == v.dtype and q.dtype in (np.uint8, np.uint16)
    B, H, nq, d = q.shape
    N = k.shape[2]
    assert k.shape == (B, H, N, d) and v.shape == (B, H, N, d)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    assert rows.ndim == 1 and (rows.size == 0 or (rows.min() >= 0 and rows.max() < nq))
    if alpha is None:
        alpha = 1.0 / np.sqrt(d)
    scales = []
    for s in (sq, sk, sv):
        if is_fp8:
            assert s is not None
            scales.append(np.ascontiguousarray(s, dtype=np.float32).reshape(B * H))
        else:
            assert s is None
            scales.append(None)
    shape = (B, H, rows.size, d)
    A = np.zeros(shape, dtype=np.float64)
    Abs = np.zeros(shape, dtype=np.float64)
    Bnd = np.zeros(shape, dtype=np.float64)
    args = _AttnArgs(
        q=_ptr(q), k=_ptr(k), v=_ptr(v),
        is_fp8=1 if is_fp8 else (2 if _DTYPE16[dtype16] else 0),
        sq=_ptr(scales[0]), sk=_ptr(scales[1]), sv=_ptr(scales[2]),
        B=B, H=H, nq=nq, n_train=N, d=d, alpha=float(alpha),
        rows=_ptr(rows), n_rows=rows.size, mode={"exact": 0, "p8": 1}[mode],
        A=_ptr(A), Abs=_ptr(Abs), Bnd=_ptr(Bnd),
        nthreads=nthreads or hardware_threads())
    if rows.size:
        _load().oracle_icl_attention_rows(ctypes.byref(args))
    if mode == "exact":
        return A, Abs, Bnd
    return A


def _row_call(fn, q, k, sq, sk, alpha, bh, row, out):
    q = np.ascontiguousarray(q)
    k = np.ascontiguousarray(k)
    B, H, nq, d = q.shape
    N = k.shape[2]
    if alpha is None:
        alpha = 1.0 / np.sqrt(d)
    fn(_ptr(q), _ptr(k), int(q.dtype == np.uint8), float(sq), float(sk),
       nq, N, d, float(alpha), int(bh), int(row), _ptr(out))
    return out


def softmax_row(q, k, bh: int, row: int, sq: float = 1.0, sk: float = 1.0,
                alpha: float | None = None) -> np.ndarray:
    """Softmax weights p_j / l of one query row over the train keys."""
    out = np.empty(k.shape[2], dtype=np.float64)
    return _row_call(_load().oracle_softmax_row, q, k, sq, sk, alpha, bh, row, out)


def lifted_p8_row(q, k, bh: int, row: int, sq: float = 1.0, sk: float = 1.0,
                  alpha: float | None = None) -> np.ndarray:
    """e4m3 codes of 2^8 * exp(t_j - max t) for one query row."""
    out = np.empty(k.shape[2], dtype=np.uint8)
    return _row_call(_load().oracle_lifted_p8_row, q, k, sq, sk, alpha, bh, row, out)


# ---- Gaussian perturbation (Eq. 3) ---------------------------------------------

def perturb(x_bf16_bits: np.ndarray, epsilon: float, seed: int, stream_id: int,
            nthreads: int | None = None):
    """bf16 bits [B,H,R,d] -> (perturbed bf16 bits, rho fp64 [B,H]):
    x + epsilon * rho[b,h] * N(0,1), rho = per-head RMS."""
    x = np.ascontiguousarray(x_bf16_bits, dtype=np.uint16)
    B, H, R, d = x.shape
    out = np.empty_like(x)
    rho = np.zeros((B, H), dtype=np.float64)
    _load().oracle_perturb(_ptr(x), B, H, R, d, float(epsilon), int(seed), int(stream_id),
                           _ptr(out), _ptr(rho), nthreads or hardware_threads())
    return out, rho
