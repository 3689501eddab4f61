"""Regex -> byte-level DFA front-end used to make the *inputs* of the library.

The library itself starts from a byte DFA; this module only prepares that
input for the regex-shaped workloads.  It compiles with Brzozowski
derivatives over hash-consed regex terms (counted repetition ``x{m,n}`` stays
symbolic, so ``x{0,4096}`` costs one state per count, not a copied
sub-automaton), removes states that cannot reach acceptance, merges
equivalent states by partition refinement and numbers states in breadth-first
order from the start state with bytes ascending, so the table for a given
regex is reproducible.

Dialect: the mathematical regular expressions the paper uses (Section 2.1) in
common notation, over the alphabet of all 256 byte values, whole-string match:
literals, ``\\`` escapes (``\\d \\s \\w \\n \\t \\r \\xHH``, any other escaped
byte stands for itself), ``.`` (any byte), classes ``[a-z0-9_]`` and negated
classes ``[^"\\\\]`` (complement within all 256 bytes), groups ``( )`` and
``(?: )``, alternation ``|``, ``* + ?`` and ``{m} {m,} {m,n}``.
"""

from __future__ import annotations

import numpy as np

ALL = (1 << 256) - 1


def _mask(bs) -> int:
    m = 0
    for b in bs:
        m |= 1 << b
    return m


_DIGIT = _mask(range(0x30, 0x3A))
_SPACE = _mask(b" \t\n\r\f\v")
_WORD = _DIGIT | _mask(range(0x41, 0x5B)) | _mask(range(0x61, 0x7B)) | (1 << 0x5F)
_ESC_SETS = {"d": _DIGIT, "D": ALL & ~_DIGIT, "s": _SPACE, "S": ALL & ~_SPACE,
             "w": _WORD, "W": ALL & ~_WORD}
_ESC_CHARS = {"n": 0x0A, "t": 0x09, "r": 0x0D, "f": 0x0C, "v": 0x0B, "0": 0x00}


class _Terms:
    """Hash-consed regex terms with normalising constructors.

    A term is an int id; ``self.t[id]`` is its tuple, ``self.nul[id]`` whether
    it matches the empty string.
    """

    def __init__(self):
        self.t = []
        self.nul = []
        self.ids = {}
        self.dcache = {}
        self.EMPTY = self._mk(("empty",), False)   # matches nothing
        self.EPS = self._mk(("eps",), True)        # matches only ""

    def _mk(self, key, nullable):
        i = self.ids.get(key)
        if i is None:
            i = len(self.t)
            self.ids[key] = i
            self.t.append(key)
            self.nul.append(nullable)
        return i

    def set(self, m):
        return self.EMPTY if m == 0 else self._mk(("set", m), False)

    def cat(self, a, b):
        if a == self.EMPTY or b == self.EMPTY:
            return self.EMPTY
        if a == self.EPS:
            return b
        if b == self.EPS:
            return a
        if self.t[a][0] == "cat":           # keep concatenations right-nested
            parts = []
            while self.t[a][0] == "cat":
                parts.append(self.t[a][1])
                a = self.t[a][2]
            parts.append(a)
            for p in reversed(parts):
                b = self._mk(("cat", p, b), self.nul[p] and self.nul[b])
            return b
        return self._mk(("cat", a, b), self.nul[a] and self.nul[b])

    def alt(self, items):
        flat = set()
        for x in items:
            if self.t[x][0] == "alt":
                flat.update(self.t[x][1])
            elif x != self.EMPTY:
                flat.add(x)
        # merge plain byte sets into one
        sets = [x for x in flat if self.t[x][0] == "set"]
        if len(sets) > 1:
            m = 0
            for x in sets:
                m |= self.t[x][1]
                flat.discard(x)
            flat.add(self.set(m))
        if not flat:
            return self.EMPTY
        if len(flat) == 1:
            return next(iter(flat))
        key = tuple(sorted(flat))
        return self._mk(("alt", key), any(self.nul[x] for x in key))

    def rep(self, a, lo, hi):
        """a{lo,hi}; hi None = unbounded."""
        if hi is not None and (hi < lo or hi == 0):
            return self.EPS if lo == 0 and hi == 0 else self.EMPTY
        if a == self.EMPTY:
            return self.EPS if lo == 0 else self.EMPTY
        if a == self.EPS:
            return self.EPS
        if self.nul[a]:
            lo = 0
        if lo == 1 and hi == 1:
            return a
        if hi is None and self.t[a][0] == "rep" and self.t[a][3] is None and self.t[a][2] <= 1:
            if lo <= 1:                      # (x*)* = x*, (x+)* = x*, (x+)+ = x+, (x*)+ = x*
                return self.rep(self.t[a][1], min(lo, self.t[a][2]), None)
        return self._mk(("rep", a, lo, hi), lo == 0)

    def deriv(self, x, c):
        """Brzozowski derivative of term ``x`` by byte ``c``."""
        key = (x, c)
        r = self.dcache.get(key)
        if r is not None:
            return r
        node = self.t[x]
        kind = node[0]
        if kind == "empty" or kind == "eps":
            r = self.EMPTY
        elif kind == "set":
            r = self.EPS if (node[1] >> c) & 1 else self.EMPTY
        elif kind == "cat":
            a, b = node[1], node[2]
            r = self.cat(self.deriv(a, c), b)
            if self.nul[a]:
                r = self.alt([r, self.deriv(b, c)])
        elif kind == "alt":
            r = self.alt([self.deriv(y, c) for y in node[1]])
        else:  # rep
            a, lo, hi = node[1], node[2], node[3]
            rest = self.rep(a, max(lo - 1, 0), None if hi is None else hi - 1)
            r = self.cat(self.deriv(a, c), rest)
        self.dcache[key] = r
        return r


class _Parser:
    def __init__(self, pattern: str, terms: _Terms, terminals=()):
        self.p = pattern
        self.i = 0
        self.T = terms
        self.terminals = list(terminals)

    def error(self, msg):
        raise ValueError("regex error at %d in %r: %s" % (self.i, self.p, msg))

    def peek(self):
        return self.p[self.i] if self.i < len(self.p) else None

    def parse(self):
        r = self.alternation()
        if self.i != len(self.p):
            self.error("unbalanced ')'")
        return r

    def alternation(self):
        alts = [self.concatenation()]
        while self.peek() == "|":
            self.i += 1
            alts.append(self.concatenation())
        return self.T.alt(alts) if len(alts) > 1 else alts[0]

    def concatenation(self):
        items = []
        while self.peek() is not None and self.peek() not in "|)":
            items.append(self.repetition())
        r = self.T.EPS
        for x in reversed(items):
            r = self.T.cat(x, r)
        return r

    def repetition(self):
        a = self.atom()
        while True:
            ch = self.peek()
            if ch == "*":
                self.i += 1
                a = self.T.rep(a, 0, None)
            elif ch == "+":
                self.i += 1
                a = self.T.rep(a, 1, None)
            elif ch == "?":
                self.i += 1
                a = self.T.rep(a, 0, 1)
            elif ch == "{":
                j = self.p.find("}", self.i)
                if j < 0:
                    self.error("unterminated {")
                body = self.p[self.i + 1:j]
                self.i = j + 1
                if "," in body:
                    lo_s, hi_s = body.split(",", 1)
                    lo = int(lo_s) if lo_s.strip() else 0
                    hi = int(hi_s) if hi_s.strip() else None
                else:
                    lo = hi = int(body)
                a = self.T.rep(a, lo, hi)
            else:
                return a

    def escape(self):
        """After a backslash: returns a byte-set mask."""
        ch = self.peek()
        if ch is None:
            self.error("dangling backslash")
        self.i += 1
        if ch in _ESC_SETS:
            return _ESC_SETS[ch]
        if ch in _ESC_CHARS:
            return 1 << _ESC_CHARS[ch]
        if ch == "x":
            v = int(self.p[self.i:self.i + 2], 16)
            self.i += 2
            return 1 << v
        return 1 << self.byte_of(ch)

    def byte_of(self, ch):
        o = ord(ch)
        if o > 255:
            self.error("non-byte character; encode the pattern first")
        return o

    def char_class(self):
        neg = False
        if self.peek() == "^":
            neg = True
            self.i += 1
        m = 0
        first = True
        while True:
            ch = self.peek()
            if ch is None:
                self.error("unterminated [")
            if ch == "]" and not first:
                self.i += 1
                break
            first = False
            self.i += 1
            if ch == "\\":
                lo_m = self.escape()
            else:
                lo_m = 1 << self.byte_of(ch)
            single = lo_m & (lo_m - 1) == 0
            if single and self.peek() == "-" and self.i + 1 < len(self.p) and self.p[self.i + 1] != "]":
                self.i += 1
                ch2 = self.peek()
                self.i += 1
                hi_m = self.escape() if ch2 == "\\" else 1 << self.byte_of(ch2)
                lo_b, hi_b = lo_m.bit_length() - 1, hi_m.bit_length() - 1
                if hi_m & (hi_m - 1) or hi_b < lo_b:
                    self.error("bad range")
                m |= _mask(range(lo_b, hi_b + 1))
            else:
                m |= lo_m
        return (ALL & ~m) if neg else m

    def atom(self):
        ch = self.peek()
        self.i += 1
        if ch == "(":
            if self.p.startswith("?P<", self.i):
                # empty named group = one edge carrying a terminal label (symbol 256 + index)
                j = self.p.find(">)", self.i)
                name = self.p[self.i + 3:j] if j >= 0 else None
                if name is None or name not in self.terminals:
                    self.error("unknown terminal label")
                self.i = j + 2
                return self.T.set(1 << (256 + self.terminals.index(name)))
            if self.p.startswith("?:", self.i):
                self.i += 2
            elif self.peek() == "?":
                self.error("unsupported group syntax")
            r = self.alternation()
            if self.peek() != ")":
                self.error("missing ')'")
            self.i += 1
            return r
        if ch == "[":
            return self.T.set(self.char_class())
        if ch == ".":
            return self.T.set(ALL)
        if ch == "\\":
            return self.T.set(self.escape())
        if ch in "*+?{":
            self.error("nothing to repeat")
        return self.T.set(1 << self.byte_of(ch))


def _byte_classes(terms: _Terms, n_symbols: int = 256):
    """Partition the symbols into classes no symbol set of the regex tells apart."""
    sets = sorted({node[1] for node in terms.t if node[0] == "set"})
    sig = {}
    cls = np.zeros(n_symbols, dtype=np.int32)
    reps = []
    for b in range(n_symbols):
        s = tuple((m >> b) & 1 for m in sets)
        if s not in sig:
            sig[s] = len(reps)
            reps.append(b)
        cls[b] = sig[s]
    return cls, reps


def _trim_merge_renumber(tc: np.ndarray, acc: np.ndarray, start: int):
    """tc: [S][C] class-level table (-1 = no edge).  Drop states that cannot
    reach acceptance, merge equivalent states, renumber breadth-first."""
    S, C = tc.shape
    # co-accessibility by backward fixpoint
    live = acc.astype(bool).copy()
    while True:
        tgt_live = np.where(tc >= 0, live[np.maximum(tc, 0)], False)
        new = live | tgt_live.any(axis=1)
        if (new == live).all():
            break
        live = new
    if not live[start]:
        # empty language: a single non-accepting state with no edges
        return np.full((1, C), -1, dtype=np.int32), np.zeros(1, dtype=np.uint8), 0
    tc = np.where((tc >= 0) & live[np.maximum(tc, 0)], tc, -1)
    # merge equivalent states: Hopcroft partition refinement over the live
    # states plus one explicit dead sink (index S) that every missing edge enters
    sink = S
    tgt = np.where(tc >= 0, tc, sink)
    tgt = np.concatenate([tgt, np.full((1, C), sink, dtype=tgt.dtype)], axis=0)
    states = [int(q) for q in np.nonzero(live)[0]] + [sink]
    inv = [dict() for _ in range(C)]           # inv[c][t] = states entering t on class c
    for q in states:
        row = tgt[q]
        for c in range(C):
            inv[c].setdefault(int(row[c]), []).append(q)
    blocks = {}
    block_of = {}
    for q in states:
        key = 2 if q == sink else int(acc[q])
        blocks.setdefault(key, set()).add(q)
        block_of[q] = key
    next_id = 3
    work = {(b_, c) for b_ in blocks for c in range(C)}
    while work:
        a_id, c = work.pop()
        x = set()
        inv_c = inv[c]
        for t in blocks[a_id]:
            x.update(inv_c.get(t, ()))
        touched = {}
        for q in x:
            touched.setdefault(block_of[q], []).append(q)
        for y_id, hit in touched.items():
            y = blocks[y_id]
            if len(hit) == len(y):
                continue
            hit_set = set(hit)
            y -= hit_set
            new_id = next_id
            next_id += 1
            blocks[new_id] = hit_set
            for q in hit_set:
                block_of[q] = new_id
            for c2 in range(C):
                if (y_id, c2) in work:
                    work.add((new_id, c2))
                else:
                    work.add((new_id, c2) if len(hit_set) <= len(y) else (y_id, c2))
    block = np.full(S, -1, dtype=np.int64)
    for q in states[:-1]:
        block[q] = block_of[q]
    # breadth-first renumbering over blocks, classes (= min byte) ascending
    rep_state = {}
    for q in range(S):
        if live[q] and block[q] not in rep_state:
            rep_state[int(block[q])] = q
    order = {int(block[start]): 0}
    queue = [int(block[start])]
    rows = []
    head = 0
    while head < len(queue):
        b = queue[head]
        head += 1
        q = rep_state[b]
        row = np.full(C, -1, dtype=np.int32)
        for c in range(C):
            t = tc[q, c]
            if t >= 0:
                tb_ = int(block[t])
                if tb_ not in order:
                    order[tb_] = len(queue)
                    queue.append(tb_)
                row[c] = order[tb_]
        rows.append(row)
    out_acc = np.array([acc[rep_state[b]] for b in queue], dtype=np.uint8)
    return np.stack(rows), out_acc, 0


def regex_to_dfa(pattern: str, terminals=()):
    """Compile ``pattern`` to ``(trans int32 [S][256 + len(terminals)], accept uint8 [S], start)``.

    ``terminals`` names the terminal labels the pattern may use as empty named
    groups ``(?P<NAME>)`` (the paper's wildcard extension, Section 2.5.1); label
    ``i`` is symbol ``256 + i``, its column holds the terminal edges."""
    T = _Terms()
    root = _Parser(pattern, T, terminals).parse()
    cls, reps = _byte_classes(T, 256 + len(list(terminals)))
    # classes are numbered by their smallest byte, so class order == byte order
    index = {root: 0}
    queue = [root]
    rows = []
    head = 0
    while head < len(queue):
        x = queue[head]
        head += 1
        row = []
        for c in reps:
            d = T.deriv(x, c)
            if d == T.EMPTY:
                row.append(-1)
                continue
            j = index.get(d)
            if j is None:
                j = len(queue)
                index[d] = j
                queue.append(d)
            row.append(j)
        rows.append(row)
    tc = np.array(rows, dtype=np.int32).reshape(len(queue), len(reps))
    acc = np.array([T.nul[x] for x in queue], dtype=np.uint8)
    tc, acc, start = _trim_merge_renumber(tc, acc, 0)
    trans = np.ascontiguousarray(tc[:, cls], dtype=np.int32)
    return trans, acc, start
