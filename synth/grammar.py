"""Grammar -> byte-level PDA front-end for bracketed grammars (an input
generator; the counterpart of the BuildGrammarPDA step that Algorithm 3 takes
from the literature).

A grammar is a start expression plus named rules of two kinds:

* macros     ``name: expression``.  Plain abbreviations, expanded in place;
             they must not be recursive.
* brackets   ``name: (open byte, expression, close byte)``.  The only place
             where recursion may pass: the body sits between two delimiter
             bytes, e.g. an array between ``[`` and ``]``.

Expressions are regular expressions in the dialect of ``regex_frontend`` in
which ``<name>`` refers to a rule.  Because every recursive call starts and
ends with a byte of its own, the resulting PDA is real-time: the opening byte
pushes the call's return address (one stack symbol per call site, like the
dotted rules of the paper's Figure 6) and jumps to the callee's body, the
closing byte pops it and resumes after the call.  Every edge reads one byte,
pops at most one symbol and pushes at most one.  Grammars that are not
deterministic in this form are rejected.
"""

from __future__ import annotations

import re

import numpy as np

from .pda import Pda, PdaBuilder
from .regex_frontend import regex_to_dfa

_REF = re.compile(r"<([A-Za-z_][A-Za-z_0-9]*)>")


class GrammarError(ValueError):
    pass


def _expand(expr: str, macros: dict, brackets: dict, trail=()):
    """Replace ``<macro>`` by its (parenthesised) expansion and ``<bracket>`` by a
    terminal label of the regex front-end."""
    def sub(m):
        name = m.group(1)
        if name in brackets:
            return "(?P<%s>)" % name
        if name not in macros:
            raise GrammarError("unknown rule <%s>" % name)
        if name in trail:
            raise GrammarError("macro <%s> is recursive; recursion must pass through a bracket rule" % name)
        return "(?:" + _expand(macros[name], macros, brackets, trail + (name,)) + ")"
    return _REF.sub(sub, expr)


def grammar_to_pda(start: str, macros: dict | None = None, brackets: dict | None = None) -> Pda:
    """``start``: expression of the whole language.  ``macros``: name -> expression.
    ``brackets``: name -> (open, expression, close) with single-byte delimiters."""
    macros = dict(macros or {})
    brackets = dict(brackets or {})
    names = sorted(brackets)
    opens, closes = {}, {}
    for n in names:
        o, _, c = brackets[n]
        o = o.encode("latin-1") if isinstance(o, str) else bytes(o)
        c = c.encode("latin-1") if isinstance(c, str) else bytes(c)
        if len(o) != 1 or len(c) != 1:
            raise GrammarError("bracket rule <%s> needs single-byte delimiters" % n)
        opens[n], closes[n] = o[0], c[0]

    # one DFA per body, over bytes plus one "call" symbol per bracket rule
    bodies = {"": start}
    bodies.update({n: brackets[n][1] for n in names})
    dfas = {}
    for key, expr in bodies.items():
        dfas[key] = regex_to_dfa(_expand(expr, macros, brackets), names)

    b = PdaBuilder()

    def st(key, q):
        return "%s#%d" % (key or "start", q)

    # PDA state 0 must be the start state of the start expression
    trans0, _, s0 = dfas[""]
    b.state(st("", s0))
    callers = {n: [] for n in names}          # bracket -> return-address symbols of its call sites
    for key, (trans, acc, s) in dfas.items():
        for q in range(trans.shape[0]):
            b.state(st(key, q))
            for byte in range(256):
                t = int(trans[q, byte])
                if t >= 0:
                    b.edge(st(key, q), byte, st(key, t))
            for i, n in enumerate(names):
                r = int(trans[q, 256 + i])
                if r < 0:
                    continue
                if trans[q, opens[n]] >= 0:
                    raise GrammarError("not deterministic: in <%s> both a byte edge and a call of <%s> "
                                       "start with byte %r" % (key or "start", n, chr(opens[n])))
                for j in range(i):
                    if trans[q, 256 + j] >= 0 and opens[names[j]] == opens[n]:
                        raise GrammarError("not deterministic: calls of <%s> and <%s> start with the "
                                           "same byte" % (names[j], n))
                sym = "%s@%s" % (st(key, r), n)            # return address of this call site
                callee = dfas[n]
                b.edge(st(key, q), opens[n], st(n, callee[2]), pushes=(sym,))
                if (sym, st(key, r)) not in callers[n]:      # several call sites may share a return address
                    callers[n].append((sym, st(key, r)))
    for n in names:
        trans, acc, _ = dfas[n]
        for f in np.nonzero(acc)[0]:
            if trans[f, closes[n]] >= 0:
                raise GrammarError("not deterministic: the body of <%s> can read its own closing byte "
                                   "where it may also end" % n)
            for sym, ret in callers[n]:
                b.edge(st(n, int(f)), closes[n], ret, pops=(sym,))
    for q in np.nonzero(dfas[""][1])[0]:
        b.final.add(st("", int(q)))
    pda = b.build(st("", s0))
    if pda.n_symbols > 254:
        raise GrammarError("%d call sites; at most 254 supported" % pda.n_symbols)
    return pda


# Nested JSON as a bracketed grammar (same language as synth.pda.json_pda(space=True)).
JSON_MACROS = {
    "string": r'"([^"\\]|\\.)*"',
    "number": r"-?(0|[1-9][0-9]*)",
    "value": r"<object>|<array>|<string>|<number>|true|false|null",
    "pair": r"<string>: ?<value>",
}
JSON_BRACKETS = {
    "array": ("[", r"(<value>(, ?<value>)*)?", "]"),
    "object": ("{", r"(<pair>(, ?<pair>)*)?", "}"),
}
JSON_START = r"<object>|<array>"


def json_grammar_pda() -> Pda:
    return grammar_to_pda(JSON_START, JSON_MACROS, JSON_BRACKETS)


def anbn_grammar_pda() -> Pda:
    """S -> ab | a S b, written with the recursion between the delimiters a and b."""
    return grammar_to_pda("<S>", {}, {"S": ("a", "<S>?", "b")})
