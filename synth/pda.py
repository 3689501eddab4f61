"""Byte-level push-down automata used as constraint inputs (Section 3).

A PDA is stored the way the C ABI takes it, as flat edge arrays: edge ``j``
goes from ``src[j]`` to ``tgt[j]`` reading byte ``inp[j]``; before it the
stack must end with ``pops[pop_off[j]:pop_off[j+1]]`` (last entry = top),
which it removes, and it appends ``pushes[push_off[j]:push_off[j+1]]``.
``accept`` flags the final states.  Only inputs are built here: nothing in
this module walks tokens, composes automata or decodes.
"""

from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Pda:
    n_states: int
    n_symbols: int
    start: int
    src: np.ndarray
    inp: np.ndarray
    tgt: np.ndarray
    pop_off: np.ndarray
    pops: np.ndarray
    push_off: np.ndarray
    pushes: np.ndarray
    accept: np.ndarray
    state_names: tuple = ()
    symbol_names: tuple = ()

    @property
    def n_edges(self) -> int:
        return int(self.src.size)


class PdaBuilder:
    """Collects named states / stack symbols and edges, then packs them."""

    def __init__(self):
        self.states: list[str] = []
        self.symbols: list[str] = []
        self.edges: list[tuple] = []
        self.final: set[str] = set()

    def state(self, name: str) -> str:
        if name not in self.states:
            self.states.append(name)
        return name

    def symbol(self, name: str) -> str:
        if name not in self.symbols:
            self.symbols.append(name)
        return name

    def edge(self, src, byte_set, tgt, pops=(), pushes=()):
        """One edge per byte of ``byte_set`` (an int, bytes, str or iterable of ints)."""
        if isinstance(byte_set, int):
            byte_set = [byte_set]
        elif isinstance(byte_set, str):
            byte_set = byte_set.encode("latin-1")
        self.state(src)
        self.state(tgt)
        for p in tuple(pops) + tuple(pushes):
            self.symbol(p)
        for b in byte_set:
            self.edges.append((src, int(b), tgt, tuple(pops), tuple(pushes)))

    def build(self, start: str) -> Pda:
        sid = {n: i for i, n in enumerate(self.states)}
        yid = {n: i for i, n in enumerate(self.symbols)}
        n = len(self.edges)
        src = np.zeros(n, dtype=np.int32)
        inp = np.zeros(n, dtype=np.int32)
        tgt = np.zeros(n, dtype=np.int32)
        pop_off = np.zeros(n + 1, dtype=np.int32)
        push_off = np.zeros(n + 1, dtype=np.int32)
        pops, pushes = [], []
        for j, (s, b, t, po, pu) in enumerate(self.edges):
            src[j], inp[j], tgt[j] = sid[s], b, sid[t]
            pops += [yid[x] for x in po]
            pushes += [yid[x] for x in pu]
            pop_off[j + 1] = len(pops)
            push_off[j + 1] = len(pushes)
        accept = np.array([1 if s in self.final else 0 for s in self.states], dtype=np.uint8)
        return Pda(len(self.states), len(self.symbols), sid[start], src, inp, tgt, pop_off,
                   np.array(pops, dtype=np.int32), push_off, np.array(pushes, dtype=np.int32),
                   accept, tuple(self.states), tuple(self.symbols))


def anbn_pda() -> Pda:
    """The language a^n b^n, n >= 1 (the grammar S -> ab | a S b of Figure 6).

    The first ``a`` pushes a bottom marker, every later ``a`` a counter symbol;
    a ``b`` pops one symbol, and the one that pops the marker reaches the final
    state, which has no outgoing edge."""
    b = PdaBuilder()
    b.edge("start", "a", "as", pushes=("Z",))
    b.edge("as", "a", "as", pushes=("A",))
    for s in ("as", "bs"):
        b.edge(s, "b", "bs", pops=("A",))
        b.edge(s, "b", "done", pops=("Z",))
    b.final.add("done")
    return b.build("start")


def dyck_pda(pairs=(b"()", b"[]", b"{}"), fillers: bytes = b"") -> Pda:
    """Non-empty balanced bracket strings over the given (open, close) pairs,
    with optional filler bytes allowed anywhere inside the outermost pair.
    The outermost bracket of type k pushes a marker ``Zk`` whose close leads to
    the final state ``done``, from which a new outermost bracket may start."""
    b = PdaBuilder()
    for k, (o, c) in enumerate(pairs):
        for s in ("start", "done"):
            b.edge(s, o, "in", pushes=("Z%d" % k,))
        b.edge("in", o, "in", pushes=("B%d" % k,))
        b.edge("in", c, "in", pops=("B%d" % k,))
        b.edge("in", c, "done", pops=("Z%d" % k,))
    if fillers:
        b.edge("in", fillers, "in")
    b.final.add("done")
    return b.build("start")


_DIGITS19 = b"123456789"
_DIGITS = b"0123456789"


def json_pda(space: bool = True) -> Pda:
    """Nested JSON with an object or array at the top: objects, arrays,
    strings (any byte but quote / backslash, or backslash + any byte), integers
    ``-?(0|[1-9][0-9]*)``, ``true`` / ``false`` / ``null``; with ``space`` one
    optional blank after ``:`` and ``,``.  Stack symbols: ARR / OBJ for nested
    containers, ARR0 / OBJ0 for the outermost one (closing it reaches the final
    state)."""
    b = PdaBuilder()
    str_body = [c for c in range(256) if c not in (0x22, 0x5C)]
    anybyte = list(range(256))

    def value_edges(src):
        b.edge(src, "[", "arr_first", pushes=("ARR",))
        b.edge(src, "{", "obj_first", pushes=("OBJ",))
        b.edge(src, '"', "str")
        b.edge(src, "-", "num_minus")
        b.edge(src, "0", "num_zero")
        b.edge(src, _DIGITS19, "num_int")
        for word in ("true", "false", "null"):
            b.edge(src, word[0], "%s_1" % word)

    def after_value_edges(src):
        for sym in ("ARR", "ARR0"):
            b.edge(src, ",", "arr_next", pops=(sym,), pushes=(sym,))
        for sym in ("OBJ", "OBJ0"):
            b.edge(src, ",", "obj_next", pops=(sym,), pushes=(sym,))
        b.edge(src, "]", "after_value", pops=("ARR",))
        b.edge(src, "]", "done", pops=("ARR0",))
        b.edge(src, "}", "after_value", pops=("OBJ",))
        b.edge(src, "}", "done", pops=("OBJ0",))

    b.edge("start", "[", "arr_first", pushes=("ARR0",))
    b.edge("start", "{", "obj_first", pushes=("OBJ0",))

    value_edges("value")
    value_edges("arr_first")
    b.edge("arr_first", "]", "after_value", pops=("ARR",))
    b.edge("arr_first", "]", "done", pops=("ARR0",))
    value_edges("arr_next")
    if space:
        b.edge("arr_next", " ", "value")

    b.edge("obj_first", '"', "key")
    b.edge("obj_first", "}", "after_value", pops=("OBJ",))
    b.edge("obj_first", "}", "done", pops=("OBJ0",))
    b.edge("obj_next", '"', "key")
    if space:
        b.edge("obj_next", " ", "obj_key")
        b.edge("obj_key", '"', "key")
    b.edge("key", str_body, "key")
    b.edge("key", "\\", "key_esc")
    b.edge("key_esc", anybyte, "key")
    b.edge("key", '"', "after_key")
    b.edge("after_key", ":", "colon")
    value_edges("colon")
    if space:
        b.edge("colon", " ", "value")

    b.edge("str", str_body, "str")
    b.edge("str", "\\", "str_esc")
    b.edge("str_esc", anybyte, "str")
    b.edge("str", '"', "after_value")

    b.edge("num_minus", "0", "num_zero")
    b.edge("num_minus", _DIGITS19, "num_int")
    b.edge("num_int", _DIGITS, "num_int")
    after_value_edges("num_zero")
    after_value_edges("num_int")
    after_value_edges("after_value")

    for word in ("true", "false", "null"):
        for i in range(1, len(word)):
            nxt = "after_value" if i == len(word) - 1 else "%s_%d" % (word, i + 1)
            b.edge("%s_%d" % (word, i), word[i], nxt)

    b.state("done")
    b.final.add("done")
    return b.build("start")


def stackless_pda(trans: np.ndarray, accept: np.ndarray, start: int) -> Pda:
    """A byte DFA written as a PDA that never touches its stack."""
    src, inp = np.nonzero(np.asarray(trans) >= 0)
    n = src.size
    zeros = np.zeros(n + 1, dtype=np.int32)
    return Pda(int(trans.shape[0]), 0, int(start), src.astype(np.int32), inp.astype(np.int32),
               np.asarray(trans)[src, inp].astype(np.int32), zeros, np.zeros(0, dtype=np.int32),
               zeros.copy(), np.zeros(0, dtype=np.int32),
               np.ascontiguousarray(accept, dtype=np.uint8))


def random_pda(seed: int, n_states: int = 6, n_symbols: int = 3, alphabet: bytes = b"abcd",
               max_push: int = 3) -> Pda:
    """A random deterministic real-time PDA over a small alphabet: per (state,
    byte) either no edge, one edge that pops nothing, or edges popping pairwise
    different symbols; every edge pushes 0..max_push random symbols (an edge
    may push back the symbol it popped).  About a third of the states accept."""
    rng = np.random.Generator(np.random.PCG64(seed))
    b = PdaBuilder()
    states = ["q%d" % i for i in range(n_states)]
    syms = ["s%d" % i for i in range(n_symbols)]
    for q in states:
        b.state(q)
    for y in syms:
        b.symbol(y)

    def pushes():
        return tuple(syms[int(k)] for k in rng.integers(0, n_symbols, size=int(rng.integers(0, max_push + 1))))

    for q in states:
        for byte in alphabet:
            kind = rng.random()
            if kind < 0.25 or n_symbols == 0 and kind < 0.5:
                continue
            if kind < 0.6 or n_symbols == 0:
                b.edge(q, byte, states[int(rng.integers(n_states))], pushes=pushes() if n_symbols else ())
            else:
                for y in syms:
                    if rng.random() < 0.7:
                        b.edge(q, byte, states[int(rng.integers(n_states))], pops=(y,), pushes=pushes())
    for q in states:
        if rng.random() < 0.35:
            b.final.add(q)
    return b.build(states[0])
