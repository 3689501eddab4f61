"""Synthetic token vocabularies.

A vocabulary is stored the way the C ABI takes it: all token byte strings
concatenated in one ``uint8`` array plus ``V + 1`` non-decreasing ``int64``
offsets, token ``v`` being ``bytes[offsets[v]:offsets[v + 1]]`` (the
detokenization d(v) of the paper's App. B.1).

The generators stand in for a real LM vocabulary (the paper measures with a
~256k-entry one, Section 5.1): ids 0..255 are the 256 single-byte tokens
(id == byte value), so every byte string can be tokenized, and the rest are
random strings with a sub-word-like length mix.
"""

from __future__ import annotations

import numpy as np

_LOWER = np.frombuffer(b"abcdefghijklmnopqrstuvwxyz", dtype=np.uint8)
_API_SYMBOLS = np.frombuffer(b'abcdefghijklmnopqrstuvwxyz0123456789_(),=" ', dtype=np.uint8)
# printable ASCII 0x21..0x7E minus lowercase letters: 94 - 26 = 68 symbols
_OTHER_PRINTABLE = np.array(
    [c for c in range(0x21, 0x7F) if not (0x61 <= c <= 0x7A)], dtype=np.uint8
)
assert _API_SYMBOLS.size == 43 and _OTHER_PRINTABLE.size == 68


def vocab_from_strings(tokens):
    """Pack an explicit list of ``bytes``/``str`` tokens into (bytes, offsets)."""
    toks = [t.encode("latin-1") if isinstance(t, str) else bytes(t) for t in tokens]
    offsets = np.zeros(len(toks) + 1, dtype=np.int64)
    for i, t in enumerate(toks):
        offsets[i + 1] = offsets[i] + len(t)
    data = np.frombuffer(b"".join(toks), dtype=np.uint8).copy()
    return data, offsets


def _pack(lengths: np.ndarray, chars: np.ndarray):
    """Prefix the 256 single-byte tokens to random strings given as lengths + flat chars."""
    all_len = np.concatenate([np.ones(256, dtype=np.int64), lengths.astype(np.int64)])
    offsets = np.zeros(all_len.size + 1, dtype=np.int64)
    np.cumsum(all_len, out=offsets[1:])
    data = np.concatenate([np.arange(256, dtype=np.uint8), chars.astype(np.uint8)])
    assert data.size == offsets[-1]
    return data, offsets


def make_vocab_api(seed: int = 0, n_random: int = 768):
    """256 byte tokens + ``n_random`` strings, length uniform 2..6, characters
    uniform over the 43 symbols ``a-z 0-9 _ ( ) , = " space``."""
    rng = np.random.Generator(np.random.PCG64(seed))
    lengths = rng.integers(2, 7, size=n_random)
    chars = _API_SYMBOLS[rng.integers(0, _API_SYMBOLS.size, size=int(lengths.sum()))]
    return _pack(lengths, chars)


def make_vocab_geometric(vocab_size: int, seed: int = 0, p: float = 0.3, cap: int = 16):
    """256 byte tokens + ``vocab_size - 256`` strings of length min(G, cap),
    G ~ Geometric(p) on {1, 2, ...}; each character independently 60 % a
    uniform lowercase letter, 15 % a space, 25 % uniform over the other 68
    printable ASCII symbols."""
    if vocab_size < 256:
        raise ValueError("vocab_size must be at least 256")
    n = vocab_size - 256
    rng = np.random.Generator(np.random.PCG64(seed))
    lengths = np.minimum(rng.geometric(p, size=n), cap)
    total = int(lengths.sum())
    kind = rng.random(total)
    lower = _LOWER[rng.integers(0, 26, size=total)]
    other = _OTHER_PRINTABLE[rng.integers(0, _OTHER_PRINTABLE.size, size=total)]
    chars = np.where(kind < 0.60, lower, np.where(kind < 0.75, np.uint8(0x20), other))
    return _pack(lengths, chars)


# Multi-character structural tokens of the kind real LM vocabularies hold for
# JSON-like text: they cross terminal boundaries and open or close several
# nesting levels at once.
_JSON_TOKENS = [
    b"]]", b"]]]", b"]]]]", b"}}", b"}}}", b"}]", b"]}", b"}]}", b"]}]", b'"]', b'"}', b'"]]',
    b'"}]', b'":', b'": ', b'":[', b'":{', b'": [', b'": {', b", ", b',"', b', "', b"[[", b"[[[",
    b"[{", b'[{"', b'{"', b'[]', b"{}", b"[],", b"{},", b"[]]", b"{}]", b"{}}", b"[]}", b"],",
    b"], ", b"},", b"}, ", b'},{"', b"],[", b"], [", b"true", b"false", b"null", b"true,",
    b"false]", b"null}", b"tru", b"fal", b"nul", b"1]", b"1}", b"12", b"-1", b"0]", b"0}", b"0,",
    b"10", b"100", b"01", b'""', b'"a"', b'"a":', b'a"]', b'a"}', b'\\"', b'\\\\', b"] ,", b"",
]


def make_vocab_json(vocab_size: int, seed: int = 0):
    """``make_vocab_geometric`` with its first random strings replaced by a fixed
    list of structural JSON tokens (brackets, quotes, literals and their
    combinations); ids 0..255 stay the single bytes."""
    base_bytes, base_off = make_vocab_geometric(vocab_size, seed=seed)
    n = min(len(_JSON_TOKENS), vocab_size - 256)
    toks = [bytes(base_bytes[base_off[v]:base_off[v + 1]]) for v in range(256 + n, vocab_size)]
    return vocab_from_strings([bytes([c]) for c in range(256)] + _JSON_TOKENS[:n] + toks)
