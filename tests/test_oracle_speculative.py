"""Pins for the rewindable constraint / speculative decoding logic (CPU only).

The defining property: with greedy selection, drafting k tokens with a
constrained approximation model, verifying them against the penalised target
model, and rewinding the constraint emits exactly the sequence that constrained
greedy decoding with the target model alone emits."""
import numpy as np
import pytest

import oracle
from oracle import regex_dfa as rd
from synth import vocab_from_strings
from synth.configs import config_dfas, config_vocab
from synth.models import draft_logits, target_logits


def target_only(dfa, vb, vo, seed, row, n_tokens):
    V = vo.size - 1
    q, out = dfa[2], []
    while len(out) < n_tokens and q >= 0:
        res = oracle.step([dfa], vb, vo, target_logits(seed, row, out, V)[None, :], [q])
        tok = int(res["tokens"][0])
        if tok < 0:
            break
        out.append(tok)
        q = int(res["states"][0])
    return out


def speculative(dfa, vb, vo, seed, row, n_tokens, k):
    """Draft k tokens keeping the state history, verify at all k + 1 positions in
    one batched step over the history, accept / rewind; repeat."""
    V = vo.size - 1
    q, out, rounds, kept = dfa[2], [], 0, 0
    while len(out) < n_tokens and q >= 0:
        hist, draft = [q], []
        for i in range(k):                           # approximation model, constrained
            res = oracle.step([dfa], vb, vo, draft_logits(seed, row, out + draft, V)[None, :], [hist[-1]])
            draft.append(int(res["tokens"][0]))
            hist.append(int(res["states"][0]))
        prefixes = [out + [t for t in draft[:i]] for i in range(k + 1)]
        tl = np.stack([target_logits(seed, row, p, V) for p in prefixes])
        res = oracle.step([dfa], vb, vo, tl, hist)   # penalties shared: same masks, history states
        n, toks, st = oracle.accept_draft(np.array([draft]), res["tokens"][None, :], res["states"][None, :])
        emitted = [int(t) for t in toks[0] if t >= 0]
        assert len(emitted) == min(int(n[0]) + 1, len(emitted))
        out += emitted
        q = int(st[0])
        rounds += 1
        kept += int(n[0])
        if not emitted:
            break
    return out[:n_tokens], rounds, kept


@pytest.mark.parametrize("k", [1, 3, 5])
def test_speculative_equals_target_only(k):
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    total_kept = 0
    for row in range(3):
        want = target_only(dfa, vb, vo, 31, row, 14)
        got, rounds, kept = speculative(dfa, vb, vo, 31, row, 14, k)
        assert got == want[:len(got)] and len(got) == len(want)
        total_kept += kept
    assert total_kept > 0                      # the draft is right often enough to matter


def test_accept_draft_by_hand():
    draft = np.array([[5, 6, 7], [5, 6, 7], [5, 6, 7], [-1, -1, -1]], dtype=np.int32)
    tgt = np.array([[5, 6, 7, 8], [5, 9, 7, 8], [4, 6, 7, 8], [-1, -1, -1, -1]], dtype=np.int32)
    st = np.array([[10, 11, 12, 13], [10, 14, 12, 13], [15, 11, 12, 13], [-1, -1, -1, -1]], dtype=np.int32)
    n, out, s = oracle.accept_draft(draft, tgt, st)
    assert n.tolist() == [3, 1, 0, 3]
    assert out.tolist() == [[5, 6, 7, 8], [5, 9, -1, -1], [4, -1, -1, -1], [-1, -1, -1, -1]]
    assert s.tolist() == [13, 14, 15, -1]
    n, out, s = oracle.accept_draft(np.zeros((2, 0), dtype=np.int32), np.array([[3], [4]]), np.array([[7], [8]]))
    assert n.tolist() == [0, 0] and out.tolist() == [[3], [4]] and s.tolist() == [7, 8]


def test_rewound_state_is_the_dfa_state_of_the_emitted_text():
    dfa = rd.compile_regex("(ab|c)*d")
    toks = [b"a", b"b", b"ab", b"c", b"cd", b"abc", b"d"]
    vb, vo = vocab_from_strings(toks)
    got, _, _ = speculative(dfa, vb, vo, 5, 0, 6, 3)
    q = dfa[2]
    for t in got:
        for byte in toks[t]:
            q = int(dfa[0][q, byte])
            assert q >= 0
