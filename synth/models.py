"""Stand-ins for language models: deterministic logits as a function of the
token prefix, so that a decoding loop can be replayed exactly.

``target`` and ``draft`` agree often but not always (the draft is the target
plus seeded noise), which is the situation speculative decoding is made for."""

from __future__ import annotations

import numpy as np

from .logits import normal_logits


def prefix_key(prefix) -> int:
    """Order-sensitive 31-bit hash of a token-id sequence."""
    h = 1469598103
    for t in prefix:
        h = (h * 1099511 + int(t) + 1) % 2147483629
    return h


def target_logits(seed: int, row: int, prefix, vocab_size: int) -> np.ndarray:
    return normal_logits(seed, prefix_key(prefix), [row], vocab_size)[0]


def draft_logits(seed: int, row: int, prefix, vocab_size: int, disagreement: float = 0.6) -> np.ndarray:
    base = target_logits(seed, row, prefix, vocab_size)
    noise = normal_logits(seed + 7919, prefix_key(prefix), [row], vocab_size)[0]
    return (base + np.float32(disagreement) * noise).astype(np.float32)
