"""Pins for the oracle's regex -> NFA -> DFA front-end (CPU only)."""
import itertools
import re

import numpy as np
import pytest

from oracle import regex_dfa as rd
from synth import constraints
from synth.regex_frontend import regex_to_dfa
from helpers import column_classes, read_regexes

PAPER = read_regexes()
REGEXES = {
    "api_call": constraints.API_CALL_REGEX,
    "flat_json": constraints.FLAT_JSON_REGEX,
    "string_small": r'"([^"\\]|\\.){0,3}"',
    "counted": r"(ab|c){2,4}d?",
    "classes": r"[^a-c]x*\d+\s?\w",
    **PAPER,
}


def strings_upto(alphabet, n):
    for k in range(n + 1):
        for t in itertools.product(alphabet, repeat=k):
            yield bytes(t)


@pytest.mark.parametrize("name", sorted(REGEXES))
def test_dfa_matches_library_regex_by_brute_force(name):
    # Every string up to length 6 over one byte per DFA byte class (at most 7
    # classes, else length 5 / 4) must be accepted iff Python's own regex
    # engine fully matches it.
    pattern = REGEXES[name]
    trans, accept, start = rd.compile_regex(pattern)
    reps = column_classes(trans)
    rng = np.random.default_rng(0)
    if len(reps) > 12:
        reps = sorted(set(rng.choice(reps, size=12, replace=False).tolist()))
    max_len = 6 if len(reps) <= 7 else (5 if len(reps) <= 10 else 4)
    lib = re.compile(pattern.encode("latin-1"), re.DOTALL)
    n_acc = 0
    for s in strings_upto(reps, max_len):
        want = lib.fullmatch(s) is not None
        got = rd.dfa_accepts(trans, accept, start, s)
        assert got == want, (pattern, s)
        n_acc += want
    # and a few hundred longer strings grown along DFA edges (so that many are accepted)
    for _ in range(300):
        q, s = start, bytearray()
        for _ in range(int(rng.integers(1, 40))):
            outs = np.nonzero(trans[q] >= 0)[0]
            if outs.size == 0:
                break
            b = int(rng.choice(outs))
            s.append(b)
            q = int(trans[q, b])
        if rng.random() < 0.3 and s:
            s[int(rng.integers(len(s)))] = int(rng.integers(256))
        s = bytes(s)
        assert rd.dfa_accepts(trans, accept, start, s) == (lib.fullmatch(s) is not None), (pattern, s)


def test_a_plus_or_ab():
    # Figure 2: /a+|ab/ accepts exactly a^n (n >= 1) and ab.
    d = rd.compile_regex("a+|ab")
    lang = {s for s in strings_upto(b"abc", 6) if rd.dfa_accepts(*d, s)}
    assert lang == {b"a" * n for n in range(1, 7)} | {b"ab"}
    # and the NFA before determinization accepts the same strings
    nfa = rd.thompson(rd.parse("a+|ab"))
    assert {s for s in strings_upto(b"abc", 6) if rd.nfa_accepts(nfa, s)} == lang
    # determinized: no epsilon edges by construction, at most one edge per (state, byte)
    assert d[0].shape[1] == 256


def test_ab_only():
    # Figure 1 (left): the FSA that accepts ab and nothing else.
    d = rd.compile_regex("ab")
    assert {s for s in strings_upto(b"abx", 5) if rd.dfa_accepts(*d, s)} == {b"ab"}


@pytest.mark.parametrize("name", sorted(REGEXES))
def test_nfa_and_dfa_agree(name):
    pattern = REGEXES[name]
    nfa = rd.thompson(rd.parse(pattern))
    d = rd.compile_regex(pattern)
    reps = column_classes(d[0])[:5]
    for s in strings_upto(reps, 4):
        assert rd.nfa_accepts(nfa, s) == rd.dfa_accepts(*d, s)


def test_trim_leaves_only_useful_states():
    for pattern in REGEXES.values():
        trans, accept, start = rd.compile_regex(pattern)
        S = trans.shape[0]
        # every state reaches an accepting state
        ok = accept.astype(bool).copy()
        for _ in range(S):
            ok |= np.array([ok[row[row >= 0]].any() for row in trans])
        assert ok.all()
        # every state is reachable from the start, numbered in discovery order
        seen, order = {start}, [start]
        for q in order:
            for b in range(256):
                t = int(trans[q, b])
                if t >= 0 and t not in seen:
                    seen.add(t)
                    order.append(t)
        assert order == list(range(S))


def test_empty_language_and_empty_string():
    t, a, s = rd.compile_regex("[^\\x00-\\xff]")
    assert t.shape == (1, 256) and (t < 0).all() and not a.any()
    t, a, s = rd.compile_regex("")
    assert a[s] and (t < 0).all()


@pytest.mark.parametrize("name", sorted(REGEXES) + ["schema40", "string_4096"])
def test_input_frontend_is_equivalent_to_oracle(name):
    # The byte DFAs fed to both the library and the oracle come from the input
    # generator's own regex front-end; it must define the same language as the
    # oracle's Thompson + subset construction.
    if name == "schema40":
        pattern = constraints.schema40_regex(0)
    elif name == "string_4096":
        pattern = constraints.STRING_LITERAL_REGEX
    else:
        pattern = REGEXES[name]
    a = rd.compile_regex(pattern)
    b = regex_to_dfa(pattern)
    assert rd.dfa_equivalent(a, b)
    assert b[0].shape[0] <= a[0].shape[0]


def test_dfa_equivalent_detects_difference():
    a = rd.compile_regex("ab*c")
    assert rd.dfa_equivalent(a, regex_to_dfa("ab*c"))
    assert not rd.dfa_equivalent(a, regex_to_dfa("ab*c?"))
    assert not rd.dfa_equivalent(a, regex_to_dfa("ab+c"))


def test_string_literal_state_count():
    # start + 4097 "k items read" + 4096 "after a backslash" + accept
    trans, accept, start = regex_to_dfa(constraints.STRING_LITERAL_REGEX)
    assert trans.shape[0] == 1 + 4097 + 4096 + 1
    assert int(accept.sum()) == 1
