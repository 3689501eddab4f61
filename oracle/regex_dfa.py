"""ORACLE (test infrastructure, not product code): regex -> NFA -> DFA.

Follows the paper's pipeline for the character-level automaton A_R
(Algorithm 2, automaton construction; Section 2.1): a regular expression is turned into a
non-deterministic FSA with epsilon edges by Thompson's construction
(BuildRegexFSA), and that FSA is determinized by the subset construction
(Section 2.1 recalls that every FSA has an equivalent deterministic one;
Figure 2 shows it for a+|ab).  The alphabet is the 256 byte
values.  Matching is whole-string (the FSA accepts w iff a path from I to F
spells w, Section 2.1).

After determinization, states from which no accepting state can be reached
are removed (edges into them become "no edge", -1), so that a token is allowed
only if acceptance stays reachable; states are numbered in breadth-first
order from the start state, bytes ascending.

Slow and plain on purpose.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may import this package.
"""

from __future__ import annotations

import numpy as np

EPS = None  # edge label for "no input"


# --------------------------------------------------------------------------
# parsing into a small AST:  ("set", frozenset_of_bytes) | ("cat", [..]) |
# ("alt", [..]) | ("repeat", node, lo, hi_or_None)
# --------------------------------------------------------------------------

_CLASS_ESCAPES = {
    "d": frozenset(range(48, 58)),
    "s": frozenset(b" \t\n\r\f\v"),
    "w": frozenset(range(48, 58)) | frozenset(range(65, 91)) | frozenset(range(97, 123)) | {95},
}
_CHAR_ESCAPES = {"n": 10, "t": 9, "r": 13, "f": 12, "v": 11, "0": 0}
_EVERY = frozenset(range(256))


def parse(pattern: str, terminals=()):
    """``terminals``: names of terminal labels; the empty named group
    ``(?P<NAME>)`` stands for one edge labelled with symbol 256 + index of NAME
    (Section 2.5.1: a terminal label is an input symbol outside the byte
    alphabet, later matched by any token of a pre-computed set)."""
    pos = 0
    n = len(pattern)
    terminals = list(terminals)

    def fail(msg):
        raise ValueError("bad regex %r at %d: %s" % (pattern, pos, msg))

    def read_escape():
        nonlocal pos
        if pos >= n:
            fail("trailing backslash")
        ch = pattern[pos]
        pos += 1
        if ch in _CLASS_ESCAPES:
            return _CLASS_ESCAPES[ch]
        if ch.lower() in _CLASS_ESCAPES and ch.isupper():
            return _EVERY - _CLASS_ESCAPES[ch.lower()]
        if ch in _CHAR_ESCAPES:
            return frozenset([_CHAR_ESCAPES[ch]])
        if ch == "x":
            value = int(pattern[pos:pos + 2], 16)
            pos += 2
            return frozenset([value])
        return frozenset([ord(ch)])

    def read_class():
        nonlocal pos
        negate = pos < n and pattern[pos] == "^"
        if negate:
            pos += 1
        members = set()
        at_start = True
        while True:
            if pos >= n:
                fail("unterminated class")
            ch = pattern[pos]
            if ch == "]" and not at_start:
                pos += 1
                break
            at_start = False
            pos += 1
            item = read_escape() if ch == "\\" else frozenset([ord(ch)])
            if (len(item) == 1 and pos + 1 < n and pattern[pos] == "-"
                    and pattern[pos + 1] != "]"):
                pos += 1
                ch2 = pattern[pos]
                pos += 1
                hi_item = read_escape() if ch2 == "\\" else frozenset([ord(ch2)])
                lo_b, hi_b = min(item), min(hi_item)
                if len(hi_item) != 1 or hi_b < lo_b:
                    fail("bad range")
                members.update(range(lo_b, hi_b + 1))
            else:
                members.update(item)
        if any(b > 255 for b in members):
            fail("non-byte symbol")
        return frozenset(_EVERY - members) if negate else frozenset(members)

    def read_atom():
        nonlocal pos
        ch = pattern[pos]
        pos += 1
        if ch == "(":
            if pattern.startswith("?P<", pos):
                close = pattern.find(">)", pos)
                name = pattern[pos + 3:close] if close >= 0 else None
                if name is None or name not in terminals:
                    fail("unknown terminal label")
                pos = close + 2
                return ("set", frozenset([256 + terminals.index(name)]))
            if pattern.startswith("?:", pos):
                pos += 2
            elif pos < n and pattern[pos] == "?":
                fail("unsupported group")
            node = read_alternation()
            if pos >= n or pattern[pos] != ")":
                fail("expected )")
            pos += 1
            return node
        if ch == "[":
            return ("set", read_class())
        if ch == ".":
            return ("set", _EVERY)
        if ch == "\\":
            return ("set", read_escape())
        if ch in "*+?{":
            fail("nothing to repeat")
        if ord(ch) > 255:
            fail("non-byte symbol")
        return ("set", frozenset([ord(ch)]))

    def read_repeat():
        nonlocal pos
        node = read_atom()
        while pos < n:
            ch = pattern[pos]
            if ch == "*":
                pos += 1
                node = ("repeat", node, 0, None)
            elif ch == "+":
                pos += 1
                node = ("repeat", node, 1, None)
            elif ch == "?":
                pos += 1
                node = ("repeat", node, 0, 1)
            elif ch == "{":
                close = pattern.find("}", pos)
                if close < 0:
                    fail("unterminated {")
                spec = pattern[pos + 1:close]
                pos = close + 1
                if "," in spec:
                    lo_s, hi_s = spec.split(",", 1)
                    lo = int(lo_s) if lo_s.strip() else 0
                    hi = int(hi_s) if hi_s.strip() else None
                else:
                    lo = hi = int(spec)
                if hi is not None and hi < lo:
                    fail("bad bounds")
                node = ("repeat", node, lo, hi)
            else:
                break
        return node

    def read_concat():
        items = []
        while pos < n and pattern[pos] not in "|)":
            items.append(read_repeat())
        return ("cat", items)

    def read_alternation():
        nonlocal pos
        options = [read_concat()]
        while pos < n and pattern[pos] == "|":
            pos += 1
            options.append(read_concat())
        return options[0] if len(options) == 1 else ("alt", options)

    tree = read_alternation()
    if pos != n:
        fail("unexpected )")
    return tree


# --------------------------------------------------------------------------
# Thompson construction: an FSA (Sigma, Q, I, F, E) with epsilon edges
# --------------------------------------------------------------------------

class NFA:
    """edges[q] = list of (label, target); label is a frozenset of bytes or EPS."""

    def __init__(self):
        self.edges = []
        self.start = None
        self.final = None

    def new_state(self):
        self.edges.append([])
        return len(self.edges) - 1

    def add(self, src, label, dst):
        self.edges[src].append((label, dst))


def thompson(tree) -> NFA:
    """Each sub-expression becomes a fragment with one entry and one exit state."""
    nfa = NFA()

    def build(node):
        kind = node[0]
        if kind == "set":
            s, t = nfa.new_state(), nfa.new_state()
            if node[1]:
                nfa.add(s, node[1], t)
            return s, t
        if kind == "cat":
            s = nfa.new_state()
            cur = s
            for child in node[1]:
                cs, ct = build(child)
                nfa.add(cur, EPS, cs)
                cur = ct
            return s, cur
        if kind == "alt":
            s, t = nfa.new_state(), nfa.new_state()
            for child in node[1]:
                cs, ct = build(child)
                nfa.add(s, EPS, cs)
                nfa.add(ct, EPS, t)
            return s, t
        if kind == "repeat":
            _, child, lo, hi = node
            s = nfa.new_state()
            cur = s
            for _ in range(lo):                      # mandatory copies
                cs, ct = build(child)
                nfa.add(cur, EPS, cs)
                cur = ct
            t = nfa.new_state()
            if hi is None:                           # then any number more
                cs, ct = build(child)
                nfa.add(cur, EPS, cs)
                nfa.add(ct, EPS, cur)
                nfa.add(cur, EPS, t)
            else:                                    # then up to hi - lo optional copies
                for _ in range(hi - lo):
                    nfa.add(cur, EPS, t)
                    cs, ct = build(child)
                    nfa.add(cur, EPS, cs)
                    cur = ct
                nfa.add(cur, EPS, t)
            return s, t
        raise AssertionError(kind)

    # the recursion depth follows the nesting of the pattern, not its length
    nfa.start, nfa.final = build(tree)
    return nfa


def nfa_accepts(nfa: NFA, data: bytes) -> bool:
    """Direct simulation of the NFA (used to cross-check determinization)."""
    cur = _closure(nfa, {nfa.start})
    for b in data:
        nxt = set()
        for q in cur:
            for label, dst in nfa.edges[q]:
                if label is not EPS and b in label:
                    nxt.add(dst)
        cur = _closure(nfa, nxt)
        if not cur:
            return False
    return nfa.final in cur


def _closure(nfa: NFA, states):
    seen = set(states)
    stack = list(states)
    while stack:
        q = stack.pop()
        for label, dst in nfa.edges[q]:
            if label is EPS and dst not in seen:
                seen.add(dst)
                stack.append(dst)
    return frozenset(seen)


# --------------------------------------------------------------------------
# subset construction
# --------------------------------------------------------------------------

def determinize(nfa: NFA, n_symbols: int = 256):
    """Returns (trans int32 [S][n_symbols] with -1 for "no edge", accept uint8 [S], start=0).
    Symbols 256.. are terminal labels.

    DFA states are epsilon-closed sets of NFA states, discovered breadth-first
    with bytes ascending.  Bytes that no edge label tells apart behave alike, so
    each group of such bytes is expanded once and the result copied.
    """
    labels = sorted({label for es in nfa.edges for label, _ in es if label is not EPS},
                    key=lambda s: sorted(s))
    signature = {}
    group_of = []
    group_first = []
    for b in range(n_symbols):
        sig = tuple(b in label for label in labels)
        if sig not in signature:
            signature[sig] = len(group_first)
            group_first.append(b)
        group_of.append(signature[sig])

    start = _closure(nfa, {nfa.start})
    ids = {start: 0}
    order = [start]
    rows = []
    head = 0
    while head < len(order):
        cur = order[head]
        head += 1
        row_by_group = []
        for b in group_first:
            moved = set()
            for q in cur:
                for label, dst in nfa.edges[q]:
                    if label is not EPS and b in label:
                        moved.add(dst)
            if not moved:
                row_by_group.append(-1)
                continue
            target = _closure(nfa, moved)
            if target not in ids:
                ids[target] = len(order)
                order.append(target)
            row_by_group.append(ids[target])
        rows.append([row_by_group[group_of[b]] for b in range(n_symbols)])
    trans = np.array(rows, dtype=np.int32).reshape(len(order), n_symbols)
    accept = np.array([nfa.final in s for s in order], dtype=np.uint8)
    return trans, accept, 0


def trim(trans: np.ndarray, accept: np.ndarray, start: int):
    """Remove states that cannot reach an accepting state; renumber breadth-first."""
    S, A = trans.shape
    # backward reachability from the accepting states over reversed edges
    preds = [set() for _ in range(S)]
    for q in range(S):
        for t in set(int(t) for t in trans[q] if t >= 0):
            preds[t].add(q)
    useful = accept.astype(bool).copy()
    stack = [q for q in range(S) if useful[q]]
    while stack:
        t = stack.pop()
        for q in preds[t]:
            if not useful[q]:
                useful[q] = True
                stack.append(q)
    if not useful[start]:
        return np.full((1, A), -1, dtype=np.int32), np.zeros(1, dtype=np.uint8), 0
    new_id = {start: 0}
    order = [start]
    head = 0
    while head < len(order):
        q = order[head]
        head += 1
        for b in range(A):
            t = int(trans[q, b])
            if t >= 0 and useful[t] and t not in new_id:
                new_id[t] = len(order)
                order.append(t)
    out = np.full((len(order), A), -1, dtype=np.int32)
    for i, q in enumerate(order):
        for b in range(A):
            t = int(trans[q, b])
            if t >= 0 and useful[t]:
                out[i, b] = new_id[t]
    return out, accept[order].astype(np.uint8), 0


def compile_regex(pattern: str, terminals=()):
    """regex -> Thompson NFA -> subset construction -> trim.  With terminal
    labels the table has 256 + len(terminals) columns (split_terminals)."""
    return trim(*determinize(thompson(parse(pattern, terminals)), 256 + len(terminals)))


def split_terminals(trans):
    """(byte transitions [S][256], terminal transitions [S][T])."""
    trans = np.asarray(trans)
    return np.ascontiguousarray(trans[:, :256]), np.ascontiguousarray(trans[:, 256:])


def dfa_accepts(trans, accept, start, data: bytes) -> bool:
    q = start
    for b in data:
        q = int(trans[q, b])
        if q < 0:
            return False
    return bool(accept[q])


def dfa_equivalent(a, b) -> bool:
    """Language equality of two DFAs by walking the product automaton."""
    (ta, aa, sa), (tb, ab, sb) = a, b
    seen = {(sa, sb)}
    stack = [(sa, sb)]
    while stack:
        p, q = stack.pop()
        pa = bool(aa[p]) if p >= 0 else False
        qa = bool(ab[q]) if q >= 0 else False
        if pa != qa:
            return False
        for byte in range(ta.shape[1]):
            np_ = int(ta[p, byte]) if p >= 0 else -1
            nq = int(tb[q, byte]) if q >= 0 else -1
            if np_ < 0 and nq < 0:
                continue
            if (np_, nq) not in seen:
                seen.add((np_, nq))
                stack.append((np_, nq))
    return True
