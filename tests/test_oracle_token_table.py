"""Pins for the oracle's token table T[q][v] = delta*(q, bytes(v)) (CPU only)."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import regex_dfa as rd
from synth import constraints, vocab_from_strings
from synth.configs import config_dfas, config_vocab
from synth.regex_frontend import regex_to_dfa
from helpers import read_records, split_tokens

RECORDS = [r for r in read_records("paper_examples.txt") if "tokens" in r and "regex" in r]


def bits(mask_row, V):
    return [(int(mask_row[v >> 5]) >> (v & 31)) & 1 for v in range(V)]


def run_tokens(nxt, mask, start, ids):
    """Accept a token-id sequence with the token automaton (tables only)."""
    q = start
    for v in ids:
        if not (int(mask[q, v >> 5]) >> (v & 31)) & 1:
            return -1
        q = int(nxt[q, v])
        assert q >= 0
    return q


def example_setup(rec):
    if rec["regex"].startswith("config:"):
        name = rec["regex"].split(":", 1)[1]
        dfa = config_dfas(name)[0]
        vb, vo = config_vocab(name)
        toks = [bytes(vb[vo[i]:vo[i + 1]]) for i in range(vo.size - 1)]
        extra = [t for t in split_tokens(rec["tokens"]) if t not in toks]
        toks = toks + extra        # the example's own tokens join the vocabulary
    else:
        dfa = rd.compile_regex(rec["regex"])
        toks = split_tokens(rec["vocab"]) if "vocab" in rec else sorted(set(split_tokens(rec["tokens"])))
    return dfa, toks


@pytest.mark.parametrize("rec", RECORDS, ids=[r["id"] for r in RECORDS])
def test_paper_worked_examples(rec):
    dfa, toks = example_setup(rec)
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
    seq = split_tokens(rec["tokens"])
    assert b"".join(seq) == rec["text"].encode("latin-1")
    ids = [toks.index(t) for t in seq]
    q = run_tokens(nxt, mask, dfa[2], ids)
    accepted = q >= 0 and bool(dfa[1][q])
    assert accepted == (rec["accepted"] == "yes")


def test_foo_plus_d_edges():
    # Figure 4 vocabulary against /(foo)+d/ (Figure 5): derived edge sets.
    toks = [b"f", b"oo", b"foo", b"for", b"food"]
    dfa = rd.compile_regex("(foo)+d")
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
    allowed = lambda q: {toks[v] for v in range(5) if bits(mask[q], 5)[v]}
    s0 = dfa[2]
    assert allowed(s0) == {b"f", b"foo", b"food"}
    after_f = int(nxt[s0, 0])
    assert allowed(after_f) == {b"oo"}
    after_foo = int(nxt[s0, 2])
    assert int(nxt[after_f, 1]) == after_foo          # f|oo and foo meet
    assert allowed(after_foo) == {b"f", b"foo", b"food"} - set() and b"for" not in allowed(after_foo)
    for q in range(dfa[0].shape[0]):
        assert b"for" not in allowed(q)
    end = int(nxt[s0, 4])
    assert dfa[1][end] and allowed(end) == set()


def test_hex_vs_digits():
    # Section 2.4: A accepts hexadecimal numbers but V only has the digits 0-9:
    # letters a-f are simply never reachable in token form.
    dfa = rd.compile_regex("[0-9a-f]+")
    toks = [bytes([c]) for c in b"0123456789"] + [b"12", b"999"]
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
    for seq in itertools.product(range(len(toks)), repeat=3):
        q = run_tokens(nxt, mask, dfa[2], seq)
        assert q >= 0 and dfa[1][q]
        text = b"".join(toks[i] for i in seq)
        assert rd.dfa_accepts(*dfa, text) and not any(c in text for c in b"abcdef")


TINY = [
    ("(ab|c)*d", [b"a", b"b", b"ab", b"c", b"cd", b"abc"]),
    ("a+|ab", [b"a", b"aa", b"ab", b"b", b"ba"]),
    ('"([^"\\\\]|\\\\.){0,3}"', [b'"', b"x", b"\\", b'\\"', b'x"', b'"x']),
    ("(foo|bar)\\((123|456)\\)", [b"fo", b"o(1", b"2", b"3)", b"foo", b"("]),
    ("x*", [b"x", b"xx", b"", b"y"]),
]


@pytest.mark.parametrize("pattern,toks", TINY)
def test_theorem2_exhaustive(pattern, toks):
    # Theorem 2: a token sequence is accepted by the token automaton iff its
    # detokenization matches the regex.  All sequences up to length 5.
    dfa = rd.compile_regex(pattern)
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
    n = len(toks)
    nonempty = [i for i in range(n) if toks[i]]
    for k in range(6):
        for seq in itertools.product(range(n), repeat=k):
            q = run_tokens(nxt, mask, dfa[2], seq)
            got = q >= 0 and bool(dfa[1][q])
            if any(not toks[i] for i in seq):
                assert q < 0          # the empty token never has an edge
                continue
            text = b"".join(toks[i] for i in seq)
            assert got == rd.dfa_accepts(*dfa, text), (pattern, seq)
            # prefix-liveness: the walk survives iff the DFA does not die on the text
            alive = dfa[2]
            for b in text:
                alive = int(dfa[0][alive, b]) if alive >= 0 else -1
            assert (q >= 0) == (alive >= 0)
            if q >= 0:
                assert q == alive


@pytest.mark.parametrize("name", ["api_1k", "json_32k"])
def test_closed_forms(name):
    dfa = config_dfas(name)[0]
    vb, vo = config_vocab(name)
    V = vo.size - 1
    trans, accept, start = dfa
    S = trans.shape[0]
    nxt, mask = oracle.token_table(trans, accept, vb, vo, threads=4)
    # (i) the 256 single-byte tokens reproduce the DFA itself
    assert (nxt[:, :256] == trans).all()
    # (iii) mask bit <=> next != DEAD, padding bits zero, popcount = count
    bit = ((mask[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(S, -1)
    assert (bit[:, :V] == (nxt >= 0)).all() and not bit[:, V:].any()
    # independent recomputation with numpy, one byte position at a time
    lens = (vo[1:] - vo[:-1]).astype(np.int64)
    cur = np.repeat(np.arange(S, dtype=np.int64)[:, None], V, axis=1)
    for k in range(int(lens.max())):
        has = lens > k
        byte = np.where(has, vb[np.minimum(vo[:-1] + k, vb.size - 1)], 0).astype(np.int64)
        step = np.where(cur >= 0, trans[np.maximum(cur, 0), byte[None, :]], -1)
        cur = np.where(has[None, :], step, cur)
    assert (cur == nxt).all()


def test_homomorphism():
    # next[q][uv] = next[next[q][u]][v] whenever u, v and uv are all tokens
    dfa = config_dfas("api_1k")[0]
    base = [b"foo", b"(", b"x", b'="', b"ba", b"r", b'")', b", ", b"n=", b"12", b")"]
    toks = list(base) + [u + v for u in base for v in base]
    vb, vo = vocab_from_strings(toks)
    nxt, _ = oracle.token_table(dfa[0], dfa[1], vb, vo)
    nb = len(base)
    for q in range(dfa[0].shape[0]):
        for i in range(nb):
            for j in range(nb):
                mid = int(nxt[q, i])
                want = int(nxt[mid, j]) if mid >= 0 else -1
                assert int(nxt[q, nb + i * nb + j]) == want


def test_eos_rule_and_slices():
    dfa = rd.compile_regex("ab?")
    toks = [b"a", b"b", b"<eos>", b"ab"]
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(dfa[0], dfa[1], vb, vo, eos_id=2)
    for q in range(dfa[0].shape[0]):
        assert bits(mask[q], 4)[2] == int(dfa[1][q]) and nxt[q, 2] == -1
    # a slice of states equals the same rows of the full table
    full_n, full_m = oracle.token_table(dfa[0], dfa[1], vb, vo)
    part_n, part_m = oracle.token_table(dfa[0], dfa[1], vb, vo, q_lo=1, q_hi=3)
    assert (part_n == full_n[1:3]).all() and (part_m == full_m[1:3]).all()
    # threads do not change the result
    t_n, t_m = oracle.token_table(dfa[0], dfa[1], vb, vo, threads=3)
    assert (t_n == full_n).all() and (t_m == full_m).all()


def test_duplicate_tokens_get_equal_columns():
    dfa = rd.compile_regex("(ab)+")
    vb, vo = vocab_from_strings([b"ab", b"a", b"ab", b"b"])
    nxt, mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
    assert (nxt[:, 0] == nxt[:, 2]).all()
