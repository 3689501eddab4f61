"""Pins for the push-down oracle (Section 3 of the paper; CPU only).

The oracle's PDA acceptance, its token-level edges (composition with the
detokenizer) and its Algorithm 3 step are checked against things fixed outside
it: closed forms of the languages, Python's ``json`` parser, brute force on tiny
vocabularies (Theorem 3), the finite-state oracle for automata that never touch
their stack, and numpy for the selection.
"""
import itertools
import json

import numpy as np
import pytest

import oracle
from oracle import pda as op
from helpers import read_records, split_tokens
from synth import (anbn_pda, dyck_pda, gumbel_noise, json_pda, normal_logits, stackless_pda,
                   vocab_from_strings)
from synth.configs import config_dfas, config_vocab

NEG_INF_BITS = np.uint32(0xFF800000)


def all_words(alphabet: bytes, max_len: int):
    for n in range(max_len + 1):
        for t in itertools.product(alphabet, repeat=n):
            yield bytes(t)


def is_anbn(w: bytes) -> bool:
    n = len(w) // 2
    return n >= 1 and w == b"a" * n + b"b" * n


def is_dyck(w: bytes, pairs, fillers: bytes) -> bool:
    """Concatenation of one or more balanced groups; fillers only inside a group."""
    closing = {p[1]: p[0] for p in pairs}
    opening = {p[0] for p in pairs}
    stack = []
    groups = 0
    for c in w:
        if c in opening:
            stack.append(c)
        elif c in closing:
            if not stack or stack[-1] != closing[c]:
                return False
            stack.pop()
            if not stack:
                groups += 1
        elif c in fillers:
            if not stack:
                return False
        else:
            return False
    return not stack and groups >= 1


# ----------------------------------------------------------------- acceptance

def test_anbn_language_by_brute_force():
    rec = [r for r in read_records("paper_examples.txt") if r["id"] == "anbn_grammar"][0]
    assert rec["language"].startswith("a^n b^n")
    P = anbn_pda()
    words = list(all_words(b"abc", 9))
    got = op.accepts(P, words, threads=4)
    want = np.array([is_anbn(w) for w in words], dtype=np.uint8)
    assert np.array_equal(got, want)
    assert got.sum() == 4


def test_dyck_language_by_brute_force():
    pairs = (b"()", b"[]")
    P = dyck_pda(pairs, fillers=b"x")
    words = list(all_words(b"()[]x", 7))
    got = op.accepts(P, words, threads=4)
    want = np.array([is_dyck(w, pairs, b"x") for w in words], dtype=np.uint8)
    assert np.array_equal(got, want)
    assert want.sum() > 50


def test_json_pda_against_the_json_module():
    # Without blanks, and over an alphabet that cannot spell fractions, exponents or
    # escapes, the PDA's language is JSON with an array or object at the top.
    P = json_pda(space=False)
    alphabet = b'[]{}"a:,1'
    words = list(all_words(alphabet, 7)) + [w for w in all_words(b'[]-01,', 6)]
    got = op.accepts(P, words, threads=8)

    def valid(w):
        if not w or w[:1] not in (b"[", b"{") or w[-1:] not in (b"]", b"}"):
            return False
        try:
            json.loads(w.decode("ascii"))
            return True
        except ValueError:
            return False

    want = np.array([valid(w) for w in words], dtype=np.uint8)
    assert np.array_equal(got, want)
    assert want.sum() > 200
    deep = [b'{"k": [1, -20, {"x": null, "y": [true, false]}], "s": "a\\"b"}',
            b'[[[[[[]]]]], {}]', b'[1, 2', b'[1 ,2]', b'{"a" :1}', b'[tru]', b'{"a":1,}']
    assert list(op.accepts(json_pda(space=True), deep)) == [1, 1, 0, 0, 0, 0, 0]


def test_initial_stack_and_nondeterminism():
    P = anbn_pda()
    Z, A = P.symbol_names.index("Z"), P.symbol_names.index("A")
    bs = P.state_names.index("bs")
    # start in the middle: state "bs" with Z A A on the stack accepts exactly bbb
    start_bs = type(P)(**{**P.__dict__, "start": bs})
    words = list(all_words(b"ab", 4))
    got = op.accepts(start_bs, words, init_stack=[Z, A, A])
    assert [w for w, g in zip(words, got) if g] == [b"bbb"]
    # a non-deterministic PDA (palindromes over {a, b} with a middle guess is not
    # needed: two edges on the same byte suffice): a* a  ==  a+
    from synth import PdaBuilder
    b = PdaBuilder()
    b.edge("s", "a", "s")
    b.edge("s", "a", "f")
    b.final.add("f")
    N = b.build("s")
    assert list(op.accepts(N, [b"", b"a", b"aaa", b"ab"])) == [0, 1, 1, 0]


# ------------------------------------------------ token-level edges (composition)

def run_tokens(P, tokens, stack=()):
    """Accept a token sequence with the token-level PDA's edges: from (q, s) take
    the edge of the next token whose pops the stack ends with."""
    q, s = P.start, list(stack)
    for t in tokens:
        hit = None
        for tgt, pops, pushes in op.token_edges(P, q, t):
            if len(pops) <= len(s) and tuple(s[len(s) - len(pops):]) == pops:
                assert hit is None, "two edges match: not deterministic"
                hit = (tgt, pops, pushes)
        if hit is None:
            return False
        q = hit[0]
        s = s[:len(s) - len(hit[1])] + list(hit[2])
    return bool(P.accept[q])


def test_figure5_vocabulary_edges():
    rec = [r for r in read_records("paper_examples.txt") if r["id"] == "anbn_vocabulary"][0]
    toks = split_tokens(rec["tokens"])
    assert toks == [b"a", b"b", b"bb", b"aaab"]
    P = anbn_pda()
    st = {n: i for i, n in enumerate(P.state_names)}
    Z, A = P.symbol_names.index("Z"), P.symbol_names.index("A")
    # aaab crosses the a / b boundary: three pushes, one of them popped again
    assert op.token_edges(P, st["start"], b"aaab") == [(st["bs"], (), (Z, A))]
    assert op.token_edges(P, st["as"], b"aaab") == [(st["bs"], (), (A, A))]
    # bb pops two symbols; which two decides where it ends
    assert sorted(op.token_edges(P, st["bs"], b"bb")) == sorted(
        [(st["bs"], (A, A), ()), (st["done"], (Z, A), ())])
    assert op.token_edges(P, st["start"], b"b") == []
    assert op.token_edges(P, st["done"], b"a") == []
    assert op.token_edges(P, st["start"], b"") == []


@pytest.mark.parametrize("case", ["anbn", "dyck", "json"])
def test_theorem3_on_tiny_vocabularies(case):
    # A token sequence is accepted by the token-level PDA iff its detokenization
    # is in the byte language - all token sequences up to a length bound.
    if case == "anbn":
        P, toks, max_len, member = anbn_pda(), [b"a", b"b", b"bb", b"aaab"], 6, is_anbn
    elif case == "dyck":
        pairs = (b"()", b"[]")
        P = dyck_pda(pairs, fillers=b"x")
        toks, max_len = [b"(", b")", b"[", b"]]", b"x)", b"([", b")]"], 5
        member = lambda w: is_dyck(w, pairs, b"x")  # noqa: E731
    else:
        P = json_pda(space=False)
        toks, max_len = [b"[", b"]", b"]]", b"1,", b"[[", b'{"a":', b"}]", b"}", b"0"], 5

        def member(w):
            try:
                json.loads(w.decode("ascii"))
                return w[:1] in (b"[", b"{")
            except ValueError:
                return False
    n_yes = 0
    for n in range(max_len + 1):
        for seq in itertools.product(toks, repeat=n):
            want = member(b"".join(seq))
            assert run_tokens(P, seq) == want, seq
            n_yes += want
    assert n_yes >= 3


# -------------------------------------------------------- allowed set and the step

def py_walk(P, edges, q, stack, data):
    """Run bytes through a deterministic byte PDA directly: (state, stack) or None."""
    s, cur = list(stack), q
    for byte in data:
        nxt = None
        for j in edges.get((cur, int(byte)), []):
            pops = list(P.pops[P.pop_off[j]:P.pop_off[j + 1]])
            if len(pops) <= len(s) and s[len(s) - len(pops):] == pops:
                nxt = j
                break
        if nxt is None:
            return None
        npop = P.pop_off[nxt + 1] - P.pop_off[nxt]
        s = s[:len(s) - npop] + [int(x) for x in P.pushes[P.push_off[nxt]:P.push_off[nxt + 1]]]
        cur = int(P.tgt[nxt])
    return cur, s


def edge_index(P):
    edges = {}
    for j in range(P.n_edges):
        edges.setdefault((int(P.src[j]), int(P.inp[j])), []).append(j)
    return edges


def py_allowed(P, vb, vo, q, stack):
    """Validity by running the bytes of each token through the byte PDA directly
    (deterministic automata only; independent of the oracle's composition)."""
    edges = edge_index(P)
    V = vo.size - 1
    out = np.zeros(V, dtype=bool)
    for v in range(V):
        out[v] = vo[v + 1] > vo[v] and py_walk(P, edges, q, stack, vb[vo[v]:vo[v + 1]]) is not None
    return out


def bits(mask_row, V):
    return np.unpackbits(mask_row.view(np.uint8), bitorder="little")[:V].astype(bool)


def small_json_vocab():
    toks = [bytes([c]) for c in range(256)]
    toks += [b"]]", b"]]]", b"}]", b"]}", b'"]', b'"}', b'":', b'": ', b", ", b',"', b"[[", b"[{",
             b'{"', b"true", b"tru", b"null,", b"1]", b"12", b"-1", b"0]", b"01", b'""', b'"a"',
             b'a"]', b"}}", b"],", b"], ", b"] ,", b"]]]]", b"", b"[]", b"{}", b"[]]", b"{}]"]
    return vocab_from_strings(toks)


def test_allowed_set_against_direct_byte_walk():
    P = json_pda(space=True)
    vb, vo = small_json_vocab()
    V = vo.size - 1
    sym = {n: i for i, n in enumerate(P.symbol_names)}
    st = {n: i for i, n in enumerate(P.state_names)}
    A0, O0, A, O = sym["ARR0"], sym["OBJ0"], sym["ARR"], sym["OBJ"]
    cases = [("start", []), ("arr_first", [A0]), ("after_value", [A0, A, A]),
             ("after_value", [O0, A]), ("num_int", [A0, O, A, A, A]), ("str", [O0]),
             ("after_value", [A0]), ("obj_first", [A0, O]), ("colon", [O0]), ("done", []),
             ("after_value", [O0, O, A, O]), ("num_zero", [A0, A])]
    states = [st[c[0]] for c in cases]
    stacks = [c[1] for c in cases]
    got = op.allowed(P, vb, vo, states, stacks)
    for i, (q, s) in enumerate(zip(states, stacks)):
        assert np.array_equal(bits(got[i], V), py_allowed(P, vb, vo, q, s)), cases[i]
    # ]]] closes three arrays only when three are open (the third being the outermost)
    v3 = V - 1 - [bytes(vb[vo[v]:vo[v + 1]]) for v in range(V)][::-1].index(b"]]]")
    assert bits(got[2], V)[v3] and not bits(got[3], V)[v3] and not bits(got[6], V)[v3]


def test_stackless_pda_reduces_to_the_finite_state_oracle():
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    V = vo.size - 1
    P = stackless_pda(*dfa)
    S = dfa[0].shape[0]
    _, mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
    got = op.allowed(P, vb, vo, np.arange(S), [[] for _ in range(S)])
    assert np.array_equal(got, mask)
    B = 8
    rng = np.random.default_rng(5)
    states = rng.integers(0, S, size=B).astype(np.int32)
    logits = normal_logits(9, 0, range(B), V)
    noise = gumbel_noise(1, 0, range(B), V)
    ref = oracle.step([dfa], vb, vo, logits, states, noise=noise)
    res = op.step(P, vb, vo, logits, states, np.zeros((B, 4), np.int32), np.zeros(B, np.int32),
                  noise=noise)
    for k in ("tokens", "states", "accept"):
        assert np.array_equal(res[k], ref[k]), k
    assert np.array_equal(res["masked"].view(np.uint32), ref["masked"].view(np.uint32))
    assert not res["depth"].any()


def test_step_penalise_select_traverse():
    P = json_pda(space=True)
    vb, vo = small_json_vocab()
    V = vo.size - 1
    toks = [bytes(vb[vo[v]:vo[v + 1]]) for v in range(V)]
    B, cap = 16, 3
    states = np.full(B, P.start, dtype=np.int32)
    stacks = np.zeros((B, cap), dtype=np.int32)
    depth = np.zeros(B, dtype=np.int32)
    texts = [b""] * B
    alive = np.ones(B, dtype=bool)
    saw_overflow = False
    edges = edge_index(P)
    for t in range(40):
        logits = normal_logits(21, t, range(B), V)
        for name in (b"[", b"[[", b"[{"):          # the last rows dig deeper than cap
            logits[B - 4:, toks.index(name)] += np.float32(6.0)
        noise = gumbel_noise(2, t, range(B), V) if t % 2 else None
        res = op.step(P, vb, vo, logits, states, stacks, depth, noise=noise, threads=2)
        score = logits if noise is None else (logits + noise).astype(np.float32)
        for r in range(B):
            if not alive[r]:
                assert res["tokens"][r] == -1 and res["states"][r] == -1
                assert (res["masked"][r].view(np.uint32) == NEG_INF_BITS).all()
                continue
            ok = py_allowed(P, vb, vo, int(states[r]), list(stacks[r, :depth[r]]))
            m = res["masked"][r].view(np.uint32)
            assert (m[ok] == logits[r].view(np.uint32)[ok]).all() and (m[~ok] == NEG_INF_BITS).all()
            if not ok.any():
                assert res["tokens"][r] == -1 and res["states"][r] == -1
                assert P.accept[states[r]]          # only "done" has no way on
                alive[r] = False
                continue
            tok = int(res["tokens"][r])
            assert tok == int(np.argmax(np.where(ok, score[r], -np.inf)))
            if res["states"][r] < 0:               # the edge would outgrow the stack array
                saw_overflow = True
                alive[r] = False
                assert np.array_equal(res["stacks"][r], stacks[r]) and res["depth"][r] == depth[r]
                continue
            texts[r] += toks[tok]
            # the bytes so far, run through the byte PDA, give the reported situation
            want_q, want_s = py_walk(P, edges, P.start, [], texts[r])
            assert res["states"][r] == want_q
            assert list(res["stacks"][r, :res["depth"][r]]) == want_s
            assert res["accept"][r] == P.accept[want_q]
        states, stacks, depth = res["states"], res["stacks"], res["depth"]
    assert saw_overflow and alive.any() and max(len(t) for t in texts) > 20


def test_inactive_rows_overflow_and_eos_by_hand():
    P = anbn_pda()
    vb, vo = vocab_from_strings([b"a", b"b", b"bb", b"aaab", b"<eos>"])
    st = {n: i for i, n in enumerate(P.state_names)}
    Z, A = P.symbol_names.index("Z"), P.symbol_names.index("A")
    V, cap = 5, 3
    logits = np.array([[0.0, 1.0, 2.0, 3.0, 0.5]] * 7, dtype=np.float32)
    states = np.array([st["start"], st["as"], st["bs"], -1, 9, st["as"], st["done"]], np.int32)
    stacks = np.array([[0, 0, 0], [Z, A, 0], [Z, A, 0], [0, 0, 0], [0, 0, 0], [Z, 7, 0],
                       [0, 0, 0]], np.int32)
    depth = np.array([0, 2, 2, 0, 0, 2, 0], np.int32)
    res = op.step(P, vb, vo, logits, states, stacks, depth, eos_id=4)
    # row 0: aaab wins and leaves Z A; row 1: aaab would need 4 cells of 3: emitted, row ends
    assert list(res["tokens"]) == [3, 3, 2, -1, -1, -1, 4]
    assert list(res["states"]) == [st["bs"], -1, st["done"], -1, -1, -1, -1]
    assert list(res["depth"]) == [2, 2, 0, 0, 0, 2, 0]
    assert list(res["stacks"][0, :2]) == [Z, A]
    assert (res["bad_state_rows"], res["empty_mask_rows"], res["overflow_rows"]) == (2, 0, 1)
    m = res["masked"]
    assert np.isneginf(m[3]).all() and np.isneginf(m[4]).all() and np.isneginf(m[5]).all()
    assert list(np.isneginf(m[0])) == [False, True, True, False, True]
    assert list(np.isneginf(m[2])) == [True, False, False, True, True]
    assert list(np.isneginf(m[6])) == [True, True, True, True, False]   # only EOS in "done"
    assert list(res["accept"]) == [0, 0, 1, 0, 0, 0, 0]


@pytest.mark.parametrize("seed", range(6))
def test_random_pdas_allowed_set_and_traversal_against_direct_walk(seed):
    # multi-symbol pushes, edges that push back what they popped, pops reaching several
    # symbols down: the composed edges must agree with running the bytes one by one
    from synth import random_pda
    rng = np.random.default_rng(100 + seed)
    P = random_pda(seed, n_states=int(rng.choice([3, 6])), n_symbols=int(rng.choice([1, 2, 3])))
    toks = [bytes(t) for n in range(0, 5) for t in itertools.product(b"abcd", repeat=n)]
    toks = [toks[i] for i in rng.permutation(len(toks))][:120]
    vb, vo = vocab_from_strings(toks)
    V = vo.size - 1
    edges = edge_index(P)
    states = rng.integers(0, P.n_states, size=10)
    stacks = [list(rng.integers(0, P.n_symbols, size=int(rng.integers(0, 6)))) for _ in range(10)]
    got = op.allowed(P, vb, vo, states, stacks)
    for i in range(10):
        want = py_allowed(P, vb, vo, int(states[i]), [int(x) for x in stacks[i]])
        assert np.array_equal(bits(got[i], V), want)
    cap = 16
    sk = np.zeros((10, cap), dtype=np.int32)
    dp = np.array([len(s) for s in stacks], dtype=np.int32)
    for i, s in enumerate(stacks):
        sk[i, :len(s)] = s
    logits = normal_logits(5, seed, range(10), V)
    res = op.step(P, vb, vo, logits, states.astype(np.int32), sk, dp)
    for i in range(10):
        tok = int(res["tokens"][i])
        if tok < 0:
            assert not bits(got[i], V).any()
            continue
        q2, s2 = py_walk(P, edges, int(states[i]), [int(x) for x in stacks[i]], toks[tok])
        if len(s2) > cap:
            assert res["states"][i] == -1
        else:
            assert res["states"][i] == q2 and list(res["stacks"][i, :res["depth"][i]]) == s2


# ------------------------------------------------ grammar front-end (input generator)

def test_bracketed_grammar_front_end():
    # The PDAs it builds are inputs of both sides; here they are checked as languages:
    # Figure 6's grammar against the closed form, nested JSON against the json module and
    # against the hand-built PDA, and ambiguous grammars are refused.
    from synth import GrammarError, anbn_grammar_pda, grammar_to_pda, json_grammar_pda
    P = anbn_grammar_pda()
    words = list(all_words(b"abc", 9))
    assert np.array_equal(op.accepts(P, words, threads=4),
                          np.array([is_anbn(w) for w in words], dtype=np.uint8))
    assert all(P.pop_off[j + 1] - P.pop_off[j] <= 1 and P.push_off[j + 1] - P.push_off[j] <= 1
               for j in range(P.n_edges))

    def deterministic(A):          # at most one edge per (state, byte, popped symbol or none)
        keys = [(int(A.src[j]), int(A.inp[j]), tuple(A.pops[A.pop_off[j]:A.pop_off[j + 1]]))
                for j in range(A.n_edges)]
        plain = {k[:2] for k in keys if not k[2]}
        return len(set(keys)) == len(keys) and not any(k[:2] in plain for k in keys if k[2])
    assert deterministic(P) and deterministic(json_grammar_pda())
    J, H = json_grammar_pda(), json_pda(space=True)
    words = list(all_words(b'[]{}"a:, 1', 6)) + list(all_words(b"[]-01,tru", 6))
    got = op.accepts(J, words, threads=8)
    assert np.array_equal(got, op.accepts(H, words, threads=8))

    def valid(w):
        if w[:1] not in (b"[", b"{"):
            return False
        try:
            json.loads(w.decode("ascii"))
            return b" " not in w        # blanks are only allowed after ':' and ',' here
        except ValueError:
            return False
    no_blank = [i for i, w in enumerate(words) if b" " not in w]
    assert all(bool(got[i]) == valid(words[i]) for i in no_blank)
    assert got.sum() > 100
    with pytest.raises(GrammarError):            # a byte edge and a call start with the same byte
        grammar_to_pda(r"<B>|\(x", {}, {"B": ("(", "y", ")")})
    with pytest.raises(GrammarError):            # the body may read its own closing byte
        grammar_to_pda(r"<B>", {}, {"B": ("(", r"[a)]*", ")")})
    with pytest.raises(GrammarError):            # recursion outside a bracket
        grammar_to_pda(r"<m>", {"m": "a<m>?"}, {})


# ------------------------------------------------ rewindable push-down constraint

def pda_target_only(P, vb, vo, seed, row, n_tokens, cap):
    from synth.models import target_logits
    V = vo.size - 1
    q, s, d, out = P.start, np.zeros((1, cap), np.int32), np.zeros(1, np.int32), []
    while len(out) < n_tokens and q >= 0:
        res = op.step(P, vb, vo, target_logits(seed, row, out, V)[None, :], [q], s, d)
        tok = int(res["tokens"][0])
        if tok < 0:
            break
        out.append(tok)
        q, s, d = int(res["states"][0]), res["stacks"], res["depth"]
    return out


def pda_speculative(P, vb, vo, seed, row, n_tokens, k, cap):
    """Draft k tokens keeping the history of situations, verify all k + 1 positions in
    one batched step over the history, accept and rewind; repeat."""
    from synth.models import draft_logits, target_logits
    V = vo.size - 1
    q, s, d, out, kept = P.start, np.zeros(cap, np.int32), 0, [], 0
    while len(out) < n_tokens and q >= 0:
        hq, hs, hd, draft = [q], [s], [d], []
        for i in range(k):
            res = op.step(P, vb, vo, draft_logits(seed, row, out + draft, V)[None, :], [hq[-1]],
                          hs[-1][None, :], [hd[-1]])
            draft.append(int(res["tokens"][0]))
            hq.append(int(res["states"][0]))
            hs.append(res["stacks"][0])
            hd.append(int(res["depth"][0]))
        tl = np.stack([target_logits(seed, row, out + draft[:i], V) for i in range(k + 1)])
        res = op.step(P, vb, vo, tl, hq, np.stack(hs), hd)
        n, toks, st, sk, dp = op.accept_draft(np.array([draft]), res["tokens"][None, :],
                                              res["states"][None, :], res["stacks"][None, :, :],
                                              res["depth"][None, :])
        emitted = [int(t) for t in toks[0] if t >= 0]
        out += emitted
        q, s, d = int(st[0]), sk[0], int(dp[0])
        kept += int(n[0])
        if not emitted:
            break
    return out[:n_tokens], kept


@pytest.mark.parametrize("k", [1, 3])
def test_pda_speculative_equals_target_only(k):
    # with greedy selection, draft / verify / rewind emits exactly what constrained
    # decoding with the target model alone emits - stacks included in the rewind
    P = json_pda(space=True)
    vb, vo = small_json_vocab()
    total_kept = 0
    for row in range(3):
        want = pda_target_only(P, vb, vo, 77, row, 12, cap=8)
        got, kept = pda_speculative(P, vb, vo, 77, row, 12, k, cap=8)
        assert got == want[:len(got)] and len(got) == len(want)
        total_kept += kept
    assert total_kept > 0
