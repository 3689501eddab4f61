"""GPU parity for terminal-label (wildcard) edges: table and decoding step vs the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import regex_dfa as rd
from paper_2407_08103_b200 import cstr
from synth import normal_logits, vocab_from_strings
from synth.configs import config_vocab
from synth.regex_frontend import regex_to_dfa

from gpu_common import check_table, gpu_tables, run_step_both
from test_gpu_table import random_vocab

pytestmark = pytest.mark.gpu


def split(full):
    trans, term = rd.split_terminals(full[0])
    return (trans, full[1], full[2]), term


@pytest.mark.parametrize("seed", range(8))
def test_random_small(seed):
    rng = np.random.default_rng(300 + seed)
    S = int(rng.choice([1, 5, 40, 300, 600]))
    T = int(rng.choice([1, 2, 5, 32]))
    V = int(rng.choice([7, 33, 1000, 4097]))
    trans = rng.integers(0, S, size=(S, 256)).astype(np.int32)
    trans[rng.random((S, 256)) < 0.6] = -1
    term = rng.integers(0, S, size=(S, T)).astype(np.int32)
    term[rng.random((S, T)) < float(rng.choice([0.3, 0.9]))] = -1
    dfa = (trans, (rng.random(S) < 0.3).astype(np.uint8), int(rng.integers(S)))
    vb, vo = random_vocab(rng, V, max_len=5)
    sets = rng.integers(0, 2 ** 32, size=V, dtype=np.uint64).astype(np.uint32)
    if T < 32:
        sets &= np.uint32((1 << T) - 1)
    sets[rng.random(V) < 0.5] = 0
    eos = int(rng.integers(0, V)) if seed % 2 else -1
    tables = gpu_tables([dfa], vb, vo, eos_id=eos, term_trans=[term], token_sets=sets)
    check_table(tables[0], dfa, vb, vo, eos_id=eos, term_trans=term, token_sets=sets)
    B = 9
    logits = rng.standard_normal((B, V)).astype(np.float32)
    states = rng.integers(-1, S, size=B).astype(np.int32)
    run_step_both([dfa], tables, vb, vo, logits, states, eos_id=eos, term_trans=[term],
                  token_sets=sets)


def test_summary_bullets_decode():
    # Section 2.5.1's bulleted-list constraint over the 32k vocabulary, decoded
    # for 40 steps; PARAGRAPH_TOKEN = newline-free tokens.
    dfa, term = split(regex_to_dfa(r"Summary:(\n\* (?P<PARAGRAPH_TOKEN>)+){3,5}", ["PARAGRAPH_TOKEN"]))
    vb, vo = config_vocab("json_32k")
    V = vo.size - 1
    has_nl = np.zeros(V, dtype=bool)
    pos = np.nonzero(vb == 0x0A)[0]
    has_nl[np.searchsorted(vo, pos, side="right") - 1] = True
    sets = (~has_nl).astype(np.uint32)
    tables = gpu_tables([dfa], vb, vo, term_trans=[term], token_sets=sets)
    check_table(tables[0], dfa, vb, vo, term_trans=term, token_sets=sets)
    B = 16
    states = np.full(B, dfa[2], dtype=np.int32)
    finished = 0
    for t in range(40):
        logits = normal_logits(55, t, range(B), V)
        ref = run_step_both([dfa], tables, vb, vo, logits, states, term_trans=[term], token_sets=sets)
        states = ref["states"]
        finished = int((states < 0).sum())
    assert finished < B          # bullets of wildcard tokens keep most rows alive


def test_summary_bullets_table_over_the_256k_vocabulary():
    # The wildcard build the benchmark times: the same constraint, 256,000 tokens, whole table.
    dfa, term = split(regex_to_dfa(r"Summary:(\n\* (?P<PARAGRAPH_TOKEN>)+){3,5}", ["PARAGRAPH_TOKEN"]))
    vb, vo = config_vocab("string_256k")
    V = vo.size - 1
    has_nl = np.zeros(V, dtype=bool)
    pos = np.nonzero(vb == 0x0A)[0]
    has_nl[np.searchsorted(vo, pos, side="right") - 1] = True
    sets = (~has_nl).astype(np.uint32)
    tables = gpu_tables([dfa], vb, vo, term_trans=[term], token_sets=sets)
    check_table(tables[0], dfa, vb, vo, term_trans=term, token_sets=sets)


def test_mixed_tables_with_and_without_labels():
    rng = np.random.default_rng(9)
    vb, vo = random_vocab(rng, 3000, max_len=4)
    V = vo.size - 1
    plain = regex_to_dfa("[a-z]+")
    wild, term = split(regex_to_dfa(r"<(?P<ANY>)+>", ["ANY"]))
    sets = (rng.random(V) < 0.8).astype(np.uint32)
    vocab = cstr.cstr_load_vocab(vb, vo)
    cstr.cstr_vocab_set_token_sets(vocab, sets, 1)
    h0 = cstr.cstr_load_dfa(*plain)
    h1 = cstr.cstr_load_dfa_terminals(wild[0], term, wild[1], wild[2])
    t0 = cstr.cstr_table_create(vocab, plain[0].shape[0])
    t1 = cstr.cstr_table_create(vocab, wild[0].shape[0])
    cstr.cstr_table_build(t0, h0)
    cstr.cstr_table_build(t1, h1)
    check_table(t0, plain, vb, vo)
    check_table(t1, wild, vb, vo, term_trans=term, token_sets=sets)
    B = 12
    row_table = (np.arange(B) % 2).astype(np.int32)
    states = np.array([plain[2] if r % 2 == 0 else wild[2] for r in range(B)], dtype=np.int32)
    no_labels = np.full((plain[0].shape[0], 1), -1, dtype=np.int32)
    for step in range(3):
        logits = rng.standard_normal((B, V)).astype(np.float32)
        ref = run_step_both([plain, wild], [t0, t1], vb, vo, logits, states, row_table=row_table,
                            term_trans=[no_labels, term], token_sets=sets)
        states = ref["states"]


def test_missing_token_sets_is_an_error():
    wild, term = split(regex_to_dfa(r"(?P<ANY>)*", ["ANY"]))
    vb, vo = vocab_from_strings([b"a", b"b"])
    vocab = cstr.cstr_load_vocab(vb, vo)
    h = cstr.cstr_load_dfa_terminals(wild[0], term, wild[1], wild[2])
    t = cstr.cstr_table_create(vocab, wild[0].shape[0])
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_table_build(t, h)
    assert e.value.code == -6
    cstr.cstr_vocab_set_token_sets(vocab, np.array([1, 0], dtype=np.uint32), 1)
    cstr.cstr_table_build(t, h)
    sets = np.array([1, 0], dtype=np.uint32)
    check_table(t, wild, vb, vo, term_trans=term, token_sets=sets)
