"""Seeded synthetic inputs shaped like the paper's kernel benchmark.

The five configurations stand in for one ICL-attention layer call of a tabular
foundation model (H heads, head dim 64 or 128, N train rows, M test rows; the
paper's latency tables use B=1, H=8, d=64/128, N up to 512k and its suites reach
1M train rows).  No dataset, weight or activation of the paper is used: values
are N(0,1) with the structure each configuration names.

This module only draws numbers (see ``gen.c``); it contains none of the
method's arithmetic and is the one piece shared by the CUDA tests and the CPU
oracle's tests.  Tensors are numpy ``uint16`` arrays of bf16 bit patterns,
shaped ``[B, H, rows, d]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libworkloads.so")
_lock = threading.Lock()
_lib = None

Q_TRAIN, K, V, Q_TEST = 0, 1, 2, 3


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    d: int
    n_train: int
    n_test: int
    seed: int
    n_outlier: int = 0          # outlier channels per head, scaled by outlier_gain
    outlier_gain: float = 1.0
    row_sigma: float = 0.0      # per-row gain exp(row_sigma * N(0,1))
    k_shift: float = 0.0        # constant added to every entry of K

    @property
    def flops(self) -> float:
        """Tensor-core FLOPs of both attention calls: 4*B*H*d*N*(N+M)."""
        return 4.0 * self.B * self.H * self.d * self.n_train * (self.n_train + self.n_test)

    @property
    def quantize_elems(self) -> int:
        return self.B * self.H * self.d * (3 * self.n_train + self.n_test)

    def scaled(self, n_train: int, n_test: int, name: str | None = None) -> "Workload":
        return replace(self, n_train=n_train, n_test=n_test,
                       name=name or f"{self.name}@{n_train}+{n_test}")


CONFIGS = {
    "C1": Workload("C1", B=1, H=2, d=64, n_train=512, n_test=128, seed=0),
    "C2": Workload("C2", B=1, H=8, d=64, n_train=8192, n_test=2048, seed=1,
                   n_outlier=4, outlier_gain=20.0),
    "C3": Workload("C3", B=1, H=8, d=128, n_train=65536, n_test=16384, seed=2,
                   row_sigma=0.5),
    "C4": Workload("C4", B=4, H=4, d=64, n_train=262144, n_test=65536, seed=3,
                   k_shift=3.0),
    "C5": Workload("C5", B=1, H=8, d=64, n_train=1048576, n_test=131072, seed=4,
                   n_outlier=2, outlier_gain=20.0),
}


def build(force: bool = False) -> str:
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.run(["gcc", "-O2", "-shared", "-fPIC", "-pthread", "-o", tmp, _SRC, "-lm"],
                   check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.workload_fill.restype = ctypes.c_int
            lib.workload_fill.argtypes = [
                ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int, ctypes.c_int,
                ctypes.c_int, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int]
            lib.workload_outlier_mask.restype = None
            lib.workload_outlier_mask.argtypes = [
                ctypes.c_uint64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                ctypes.c_void_p]
            _lib = lib
    return _lib


def fill(out: np.ndarray, w: Workload, tensor_id: int, nthreads: int | None = None) -> np.ndarray:
    """Fill ``out`` (uint16 [B,H,rows,d], C-contiguous, may be pinned memory)."""
    assert out.dtype == np.uint16 and out.flags.c_contiguous
    B, H, R, d = out.shape
    assert (B, H, d) == (w.B, w.H, w.d)
    if out.size == 0:
        return out
    nt = nthreads or (os.cpu_count() or 1)
    _load().workload_fill(out.ctypes.data_as(ctypes.c_void_p), w.seed, tensor_id,
                          B, H, R, d, w.n_outlier, w.outlier_gain, w.row_sigma,
                          w.k_shift if tensor_id == K else 0.0, nt)
    return out


def generate(w: Workload, nthreads: int | None = None) -> dict:
    """All four bf16 tensors of a workload as uint16 bit patterns."""
    res = {}
    for name, tid, rows in (("q_train", Q_TRAIN, w.n_train), ("k", K, w.n_train),
                            ("v", V, w.n_train), ("q_test", Q_TEST, w.n_test)):
        res[name] = fill(np.empty((w.B, w.H, rows, w.d), dtype=np.uint16), w, tid, nthreads)
    return res


def outlier_mask(w: Workload, bh: int) -> np.ndarray:
    m = np.zeros(w.d, dtype=np.uint8)
    _load().workload_outlier_mask(w.seed, bh, w.d, w.n_outlier, m.ctypes.data_as(ctypes.c_void_p))
    return m.astype(bool)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)
