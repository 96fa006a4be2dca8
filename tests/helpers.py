"""Shared test helpers: numpy-side conversions and the parity criteria."""
import numpy as np


def read_golden_table(path):
    rows = []
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            rows.append(line.split())
    return rows


def bf16_bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_bits(x):
    """Round-to-nearest-even fp32 -> bf16 bit patterns (numpy, test side)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> 16) & 1
    return ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)


def numpy_attention_f64(q, k, v, alpha):
    """Plain fp64 softmax attention: q [nq,d], k/v [N,d] real-valued."""
    t = alpha * (q @ k.T)
    t = t - t.max(axis=1, keepdims=True)
    p = np.exp(t)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v, p
