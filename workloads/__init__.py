"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module only *generates numbers*: weight tensors with the shapes and value
distributions of LLM decoder layers, and activation vectors.  It contains none
of the compression method's arithmetic (no field split, no Huffman code, no
bitstream), so both the CUDA library and the CPU oracle may be fed from it
without sharing any code of the method itself.

Real checkpoints are not available offline; the paper's compression table
(Section 5.1) is matched in bits/parameter by Gaussian weights with a per-row
scale, which is what every generator here produces unless stated otherwise.

All tensors are returned as ``numpy.uint16`` arrays holding raw bf16 (or fp16)
bit patterns, row-major ``[rows=out_features][cols=in_features]``.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "f32_to_bf16_bits",
    "bf16_bits_to_f32",
    "gaussian_weights",
    "student_t_weights",
    "uniform_exponent_weights",
    "all_patterns_weights",
    "skewed_exponent_weights",
    "activations",
    "LAYER_LLAMA7B",
    "LAYER_8B",
    "FFN_70B",
    "layer_tensors",
]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rnd = ((u >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
    return ((u + rnd) >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _row_scale(rng: np.random.Generator, rows: int) -> np.ndarray:
    return rng.uniform(0.5, 2.0, size=(rows, 1)).astype(np.float32)


def gaussian_weights(rows: int, cols: int, std: float, seed: int, dtype: str = "bf16") -> np.ndarray:
    """N(0, std^2) entries, each output row multiplied by a scale drawn U(0.5, 2)."""
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)
    w *= _row_scale(rng, rows)
    if dtype == "bf16":
        return f32_to_bf16_bits(w)
    if dtype == "fp16":
        return w.astype(np.float16).view(np.uint16)
    if dtype == "fp16_from_bf16":  # bf16-trained weights later stored as fp16
        return bf16_bits_to_f32(f32_to_bf16_bits(w)).astype(np.float16).view(np.uint16)
    raise ValueError(dtype)


def student_t_weights(rows: int, cols: int, seed: int, scale: float = 0.02, nu: float = 3.0,
                      outlier_frac: float = 0.01, outlier_gain: float = 50.0) -> np.ndarray:
    """Heavy-tailed stress case: Student-t(nu) entries, row scaled, 1 % of rows amplified."""
    rng = np.random.default_rng(seed)
    w = rng.standard_t(nu, size=(rows, cols)).astype(np.float32) * np.float32(scale)
    w *= _row_scale(rng, rows)
    n_out = max(1, int(round(rows * outlier_frac)))
    w[rng.choice(rows, n_out, replace=False)] *= np.float32(outlier_gain)
    return f32_to_bf16_bits(w)


def uniform_exponent_weights(rows: int, cols: int, seed: int, e_lo: int = 111, e_hi: int = 143) -> np.ndarray:
    """Worst case for the coder: bf16 exponent uniform on [e_lo, e_hi), sign and mantissa uniform.
    Values stay finite and moderate so a matrix-vector product is still meaningful."""
    rng = np.random.default_rng(seed)
    e = rng.integers(e_lo, e_hi, size=(rows, cols), dtype=np.uint16)
    m = rng.integers(0, 128, size=(rows, cols), dtype=np.uint16)
    s = rng.integers(0, 2, size=(rows, cols), dtype=np.uint16)
    return ((s << 15) | (e << 7) | m).astype(np.uint16)


def all_patterns_weights(rows: int, cols: int, seed: int) -> np.ndarray:
    """Every 16-bit pattern (NaN, Inf, denormals, both zeros included), repeated and shuffled.
    For lossless-decode checks only."""
    rng = np.random.default_rng(seed)
    n = rows * cols
    reps = -(-n // 65536)
    v = np.tile(np.arange(65536, dtype=np.uint32), reps)[:n].astype(np.uint16)
    if n < 65536:
        v = rng.integers(0, 65536, size=n, dtype=np.uint32).astype(np.uint16)
    rng.shuffle(v)
    return v.reshape(rows, cols)


def skewed_exponent_weights(rows: int, cols: int, seed: int, e_top: int = 130, span: int = 28, dtype: str = "bf16") -> np.ndarray:
    """Exponents with a geometric law: exponent e_top - j has probability proportional to 2^-j (j < span), sign and
    mantissa uniform.  Such a field has Huffman codewords of every length up to about `span` bits, so every
    length limit from 8 to 12 bites and long codewords do occur: the stress case for the longer decode tables.
    Values stay finite and moderate.  dtype "fp16": the same law on the 5-bit exponent (e_top and span are clipped)."""
    rng = np.random.default_rng(seed)
    j = np.minimum(rng.geometric(0.5, size=(rows, cols)) - 1, span - 1).astype(np.int64)
    s = rng.integers(0, 2, size=(rows, cols), dtype=np.uint16)
    if dtype == "bf16":
        e = (e_top - j).astype(np.uint16)
        m = rng.integers(0, 128, size=(rows, cols), dtype=np.uint16)
        return ((s << 15) | (e << 7) | m).astype(np.uint16)
    e = np.clip(min(e_top, 17) - j, 1, 30).astype(np.uint16)
    # the mantissa halves follow the same kind of law, so that their codes grow long too
    mh = np.minimum(rng.geometric(0.5, size=(rows, cols)) - 1, 31).astype(np.uint16)
    ml = np.minimum(rng.geometric(0.5, size=(rows, cols)) - 1, 31).astype(np.uint16)
    return ((s << 15) | (e << 10) | (mh << 5) | ml).astype(np.uint16)


def activations(batch: int, cols: int, seed: int, dtype: str = "bf16") -> np.ndarray:
    """x ~ N(0, 1) rounded to the weight dtype, shape [batch][cols]."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((batch, cols), dtype=np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    return x.astype(np.float16).view(np.uint16)


# (name, rows, cols) per decoder layer; std of the Gaussian is given beside each table.
LAYER_LLAMA7B = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
LAYER_8B = [("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
            ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336)]
FFN_70B = [("up", 28672, 8192), ("down", 8192, 28672)]


def layer_tensors(table, std: float, seed: int, dtype: str = "bf16"):
    """Yield (name, weights) for every matrix of a layer table; tensor i uses seed + i."""
    for i, (name, rows, cols) in enumerate(table):
        yield name, gaussian_weights(rows, cols, std, seed + i, dtype)
