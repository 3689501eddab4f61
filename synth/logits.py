"""Seeded logits and Gumbel noise.

Every row of every tensor is drawn from its own counter-keyed stream
``(seed, pool_entry, row)``, so a checker can regenerate any single row of a
full-size batch without materialising the whole tensor, and so the values do
not depend on the batch size or on which rows are generated.
"""

from __future__ import annotations

import numpy as np


def _row_rng(seed: int, entry: int, row: int, stream: int):
    return np.random.Generator(np.random.Philox(key=[seed * 4 + stream, (entry << 32) | row]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round-to-nearest-even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = (rounded >> np.uint32(16)).astype(np.uint16)
    nan = (u & np.uint32(0x7FFFFFFF)) > np.uint32(0x7F800000)
    if nan.any():
        out = np.where(nan, ((u >> np.uint32(16)) | np.uint32(0x0040)).astype(np.uint16), out)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_logits(seed: int, entry: int, rows, vocab_size: int, ld: int | None = None,
                  sigma: float = 1.0, dtype: str = "f32", out: np.ndarray | None = None):
    """Logits ~ N(0, sigma^2) for the given row indices of pool entry ``entry``.

    Returns ``[len(rows)][ld]`` float32 (``dtype='f32'``) or uint16 bfloat16 bit
    patterns (``dtype='bf16'``); columns ``vocab_size..ld`` are zero padding.
    """
    rows = list(rows)
    ld = vocab_size if ld is None else ld
    np_dtype = np.float32 if dtype == "f32" else np.uint16
    if out is None:
        out = np.zeros((len(rows), ld), dtype=np_dtype)
    for i, r in enumerate(rows):
        x = _row_rng(seed, entry, r, 0).standard_normal(vocab_size, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        out[i, :vocab_size] = x if dtype == "f32" else f32_to_bf16_bits(x)
    return out


def gumbel_noise(seed: int, entry: int, rows, vocab_size: int, ld: int | None = None,
                 out: np.ndarray | None = None):
    """Standard Gumbel noise g = -log(-log u), u uniform in (0, 1), as float32
    ``[len(rows)][ld]`` (zero padding past ``vocab_size``)."""
    rows = list(rows)
    ld = vocab_size if ld is None else ld
    if out is None:
        out = np.zeros((len(rows), ld), dtype=np.float32)
    tiny = np.finfo(np.float64).tiny
    for i, r in enumerate(rows):
        u = _row_rng(seed, entry, r, 1).random(vocab_size)
        u = np.clip(u, tiny, 1.0 - 2.0 ** -53)
        out[i, :vocab_size] = (-np.log(-np.log(u))).astype(np.float32)
    return out
