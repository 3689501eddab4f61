"""Pins for terminal labels (wildcard edges matched by pre-computed token sets,
Section 2.5.1) in the oracle: regex front-end, token table and step (CPU only)."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import regex_dfa as rd
from synth import vocab_from_strings
from helpers import read_records


def sets_word(tokens, predicates):
    """uint32 per token: bit t set iff predicates[t](token)."""
    return np.array([sum(1 << t for t, p in enumerate(predicates) if tok and p(tok)) for tok in tokens],
                    dtype=np.uint32)


def reference_edge(trans, term, sets, q, tok_bytes, v):
    """Definition, written independently of the C code: ordinary edge if the byte
    walk survives, else the first terminal edge (label order) whose set holds v."""
    if len(tok_bytes) == 0:
        return -1
    s = q
    for b in tok_bytes:
        s = int(trans[s, b])
        if s < 0:
            break
    if s >= 0:
        return s
    for t in range(term.shape[1]):
        if term[q, t] >= 0 and (int(sets[v]) >> t) & 1:
            return int(term[q, t])
    return -1


def run(nxt, mask, start, ids):
    q = start
    for v in ids:
        if not (int(mask[q, v >> 5]) >> (v & 31)) & 1:
            return -1
        q = int(nxt[q, v])
    return q


def test_summary_bullets_example():
    rec = [r for r in read_records("paper_examples.txt") if r["id"] == "summary_bullets"][0]
    names = rec["terminals"].split(",")
    full = rd.compile_regex(rec["regex"], names)
    trans, term = rd.split_terminals(full[0])
    accept, start = full[1], full[2]
    toks = [b"Summary:", b"\n", b"* ", b"\n* ", b"alpha", b"beta gamma", b"two\nlines", b":", b"Sum", b"mary:"]
    sets = sets_word(toks, [lambda t: b"\n" not in t])          # newline-free tokens
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(trans, accept, vb, vo, term_trans=term, token_sets=sets)
    T = {t: i for i, t in enumerate(toks)}

    def accepted(seq):
        q = run(nxt, mask, start, [T[t] for t in seq])
        return q >= 0 and bool(accept[q])

    bullet = [b"\n", b"* ", b"alpha"]
    head = [b"Summary:"]
    assert not accepted(head + bullet * 2)
    for k in (3, 4, 5):
        assert accepted(head + bullet * k)
    assert not accepted(head + bullet * 6)
    assert accepted([b"Sum", b"mary:"] + [b"\n* ", b"beta gamma", b"alpha"] * 3)   # several tokens per bullet
    assert not accepted(head + bullet * 2 + [b"\n", b"* ", b"two\nlines"])         # newline inside a bullet
    assert not accepted(head + bullet * 3 + [b":"] + [b"\n"])                      # dangling newline
    assert accepted(head + bullet * 3 + [b":"])                                    # ":" is a paragraph token
    # inside a bullet the wildcard set is allowed en masse, next to the ordinary "\n"
    q = run(nxt, mask, start, [T[t] for t in head + bullet])
    allowed = {toks[v] for v in range(len(toks)) if (int(mask[q, 0]) >> v) & 1}
    assert allowed == {b"\n", b"\n* ", b"* ", b"alpha", b"beta gamma", b":", b"Summary:", b"Sum", b"mary:"}


def test_precedence_normal_edge_then_label_order():
    trans = np.full((4, 256), -1, dtype=np.int32)
    trans[0, ord("a")] = 1
    term = np.full((4, 2), -1, dtype=np.int32)
    term[0, 0], term[0, 1] = 2, 3
    accept = np.array([0, 1, 1, 1], dtype=np.uint8)
    toks = [b"a", b"b", b"c", b"d", b""]
    sets = np.array([0b11, 0b11, 0b10, 0b00, 0b11], dtype=np.uint32)
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(trans, accept, vb, vo, term_trans=term, token_sets=sets)
    assert nxt[0].tolist() == [1, 2, 3, -1, -1]         # ordinary edge, lower label, only label, none, empty
    assert int(mask[0, 0]) == 0b00111
    assert (nxt[1:] == -1).all() and not mask[1:].any()
    # the step follows the same edges
    logits = np.array([[0, 0, 9, 0, 99]], dtype=np.float32)
    res = oracle.step([(trans, accept)], vb, vo, logits, [0], term_trans=[term], token_sets=sets)
    assert res["tokens"][0] == 2 and res["states"][0] == 3 and res["accept"][0] == 1
    assert res["masked"][0].tolist()[:3] == [0, 0, 9] and np.isneginf(res["masked"][0, 3:]).all()


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_against_the_definition(seed):
    rng = np.random.default_rng(seed)
    S, T, V = int(rng.integers(1, 9)), int(rng.integers(0, 4)), 40
    trans = rng.integers(0, S, size=(S, 256)).astype(np.int32)
    trans[rng.random((S, 256)) < 0.7] = -1
    term = rng.integers(0, S, size=(S, T)).astype(np.int32)
    term[rng.random((S, T)) < 0.5] = -1
    accept = (rng.random(S) < 0.4).astype(np.uint8)
    toks = [bytes(rng.integers(97, 101, size=int(rng.integers(0, 4))).astype(np.uint8)) for _ in range(V)]
    sets = rng.integers(0, 1 << T, size=V).astype(np.uint32) if T else np.zeros(V, dtype=np.uint32)
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(trans, accept, vb, vo, term_trans=term, token_sets=sets, threads=2)
    for q in range(S):
        for v in range(V):
            want = reference_edge(trans, term, sets, q, toks[v], v)
            assert nxt[q, v] == want
            assert ((int(mask[q, v >> 5]) >> (v & 31)) & 1) == int(want >= 0)
    # en masse: mask = ordinary mask OR the sets of the labels that have an edge
    plain_next, plain_mask = oracle.token_table(trans, accept, vb, vo)
    nonempty = np.array([len(t) > 0 for t in toks])
    for q in range(S):
        union = np.zeros(V, dtype=bool)
        for t in range(T):
            if term[q, t] >= 0:
                union |= ((sets >> t) & 1).astype(bool)
        bits = ((mask[q][:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[:V].astype(bool)
        assert np.array_equal(bits, (plain_next[q] >= 0) | (union & nonempty))


def test_without_labels_nothing_changes():
    d = rd.compile_regex("(ab|c)*d")
    toks = [b"a", b"b", b"ab", b"c", b"cd", b"abc", b"d"]
    vb, vo = vocab_from_strings(toks)
    a = oracle.token_table(d[0], d[1], vb, vo)
    b = oracle.token_table(d[0], d[1], vb, vo, term_trans=np.zeros((d[0].shape[0], 0), dtype=np.int32),
                           token_sets=np.zeros(len(toks), dtype=np.uint32))
    c = oracle.token_table(d[0], d[1], vb, vo, term_trans=np.full((d[0].shape[0], 3), -1, dtype=np.int32),
                           token_sets=np.full(len(toks), 7, dtype=np.uint32))
    for x in (b, c):
        assert np.array_equal(a[0], x[0]) and np.array_equal(a[1], x[1])


def test_terminal_only_language():
    # (?P<W>)* accepts exactly the sequences of tokens of the set W
    full = rd.compile_regex("(?P<W>)*", ["W"])
    trans, term = rd.split_terminals(full[0])
    toks = [b"x", b"yy", b"z", b"w"]
    sets = np.array([1, 0, 1, 1], dtype=np.uint32)
    vb, vo = vocab_from_strings(toks)
    nxt, mask = oracle.token_table(trans, full[1], vb, vo, term_trans=term, token_sets=sets)
    for k in range(4):
        for seq in itertools.product(range(4), repeat=k):
            q = run(nxt, mask, full[2], seq)
            assert (q >= 0 and bool(full[1][q])) == all(sets[v] for v in seq)
