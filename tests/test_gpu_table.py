"""GPU parity: token table built by libcstr vs the CPU oracle, bit exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_08103_b200 import cstr
from synth import random_range_dfa, vocab_from_strings
from synth.configs import config_dfas, config_vocab
from synth.regex_frontend import regex_to_dfa

from gpu_common import check_table, gpu_tables

pytestmark = pytest.mark.gpu


def random_vocab(rng, V, max_len=20, alphabet=None, empty_prob=0.02):
    alphabet = np.arange(256, dtype=np.uint8) if alphabet is None else np.frombuffer(alphabet, dtype=np.uint8)
    toks = []
    for _ in range(V):
        n = 0 if rng.random() < empty_prob else int(min(rng.geometric(0.3), max_len))
        toks.append(bytes(alphabet[rng.integers(0, alphabet.size, size=n)]))
    return vocab_from_strings(toks)


def dense_random_dfa(rng, S, live=0.7):
    trans = rng.integers(0, S, size=(S, 256)).astype(np.int32)
    trans[rng.random((S, 256)) > live] = -1
    return trans, (rng.random(S) < 0.3).astype(np.uint8), int(rng.integers(S))


@pytest.mark.parametrize("seed", range(12))
def test_random_small(seed):
    rng = np.random.default_rng(seed)
    S = int(rng.choice([1, 2, 3, 17, 64, 100, 257]))
    V = int(rng.choice([1, 5, 31, 32, 33, 255, 256, 257, 1000, 2049]))
    dfa = dense_random_dfa(rng, S, live=float(rng.choice([0.2, 0.7, 1.0])))
    vb, vo = random_vocab(rng, V)
    eos = int(rng.integers(-1, V)) if seed % 3 == 0 else -1
    (table,) = gpu_tables([dfa], vb, vo, eos_id=eos)
    check_table(table, dfa, vb, vo, eos_id=eos)


def test_degenerate_cases():
    # a single state with no edges; all-dead and all-live DFAs; only empty tokens; 16/17-byte tokens
    dead = (np.full((1, 256), -1, dtype=np.int32), np.zeros(1, dtype=np.uint8), 0)
    loop = (np.zeros((1, 256), dtype=np.int32), np.ones(1, dtype=np.uint8), 0)
    toks = [b"", b"a", b"x" * 15, b"y" * 16, b"z" * 17, b"w" * 40, b"", bytes(range(256))]
    vb, vo = vocab_from_strings(toks)
    for dfa in (dead, loop):
        (table,) = gpu_tables([dfa], vb, vo)
        check_table(table, dfa, vb, vo)
    vb, vo = vocab_from_strings([b"", b"", b""])
    (table,) = gpu_tables([loop], vb, vo)
    check_table(table, loop, vb, vo)
    # long tokens walking a chain DFA: dies exactly at position 20
    S = 21
    trans = np.full((S, 256), -1, dtype=np.int32)
    for q in range(S - 1):
        trans[q, 0x61] = q + 1
    chain = (trans, np.eye(1, S, S - 1, dtype=np.uint8)[0], 0)
    vb, vo = vocab_from_strings([b"a" * n for n in range(0, 30)])
    (table,) = gpu_tables([chain], vb, vo)
    check_table(table, chain, vb, vo)


def test_rebuild_reuses_the_table_and_wide_capacity():
    rng = np.random.default_rng(5)
    vb, vo = random_vocab(rng, 700)
    vocab = cstr.cstr_load_vocab(vb, vo)
    table = cstr.cstr_table_create(vocab, 300)
    for S in (300, 7, 120):
        dfa = dense_random_dfa(rng, S)
        h = cstr.cstr_load_dfa(*dfa)
        cstr.cstr_table_build(table, h, -1)
        check_table(table, dfa, vb, vo)
    too_big = cstr.cstr_load_dfa(*dense_random_dfa(rng, 301))
    with pytest.raises(cstr.CstrError):
        cstr.cstr_table_build(table, too_big, -1)
    # capacity above 32767 states stores 32-bit entries; a small DFA still fits
    vb2, vo2 = random_vocab(rng, 40)
    vocab2 = cstr.cstr_load_vocab(vb2, vo2)
    wide = cstr.cstr_table_create(vocab2, 40000)
    dfa = dense_random_dfa(rng, 50)
    h_small = cstr.cstr_load_dfa(*dfa)
    cstr.cstr_table_build(wide, h_small, -1)
    check_table(wide, dfa, vb2, vo2)
    big = random_range_dfa(33000, seed=9)
    h_big = cstr.cstr_load_dfa(*big)
    cstr.cstr_table_build(wide, h_big, -1)
    check_table(wide, big, vb2, vo2, states=[0, 1, 32767, 32768, 32999])


def test_one_call_form():
    dfa = regex_to_dfa("(ab|c)*d")
    vb, vo = vocab_from_strings([b"a", b"b", b"ab", b"c", b"cd", b"abc", b"d"])
    h = cstr.cstr_load_dfa(*dfa)
    table = cstr.cstr_build_token_table(h, vb, vo, eos_id=-1)
    check_table(table, dfa, vb, vo)


@pytest.mark.parametrize("name", ["api_1k", "json_32k"])
def test_config_full(name):
    dfa = config_dfas(name)[0]
    vb, vo = config_vocab(name)
    (table,) = gpu_tables([dfa], vb, vo)
    check_table(table, dfa, vb, vo)


def test_config_schema40_128k():
    dfa = config_dfas("schema40_128k")[0]
    vb, vo = config_vocab("schema40_128k")
    (table,) = gpu_tables([dfa], vb, vo)
    check_table(table, dfa, vb, vo, slab=123)


def whole_table_parity(table, dfa, vb, vo, slab=256):
    """Every state of a full-size table against the oracle, streamed in slabs of states so
    that neither side ever holds the table on the host; returns the number of live edges."""
    S = dfa[0].shape[0]
    threads = min(oracle.max_threads(), 32)
    live_total = 0
    for lo in range(0, S, slab):
        hi = min(S, lo + slab)
        nxt, mask = cstr.cstr_table_download(table, lo, hi)
        o_next, o_mask = oracle.token_table(dfa[0], dfa[1], vb, vo, q_lo=lo, q_hi=hi, threads=threads)
        assert np.array_equal(nxt, o_next), "next-state rows %d..%d differ" % (lo, hi)
        assert np.array_equal(mask, o_mask), "mask rows %d..%d differ" % (lo, hi)
        live_total += int((o_next >= 0).sum())
    return live_total


def test_config_string_256k_whole_table():
    # all 8,195 x 256,000 transitions and all mask words
    dfa = config_dfas("string_256k")[0]
    vb, vo = config_vocab("string_256k")
    (table,) = gpu_tables([dfa], vb, vo)
    check_table(table, dfa, vb, vo, states=[0])          # shape information, first row
    assert whole_table_parity(table, dfa, vb, vo) > 0
    # popcount of every mask row equals the count of live entries, for a slab of rows
    nxt, mask = cstr.cstr_table_download(table, 100, 132)
    live = (nxt >= 0).sum(axis=1)
    pop = np.unpackbits(mask.view(np.uint8), axis=1).sum(axis=1)
    assert np.array_equal(live, pop)


def test_config_random10k_256k_whole_tables_of_all_eight_dfas():
    # 8 x 10,000 x 256,000 transitions: each automaton is built into the same table storage
    # (a rebuild) and compared completely before the next one is built
    dfas = config_dfas("random10k_256k")
    assert len(dfas) == 8
    vb, vo = config_vocab("random10k_256k")
    vocab = cstr.cstr_load_vocab(vb, vo)
    table = cstr.cstr_table_create(vocab, 10000)
    for dfa in dfas:
        cstr.cstr_table_build(table, cstr.cstr_load_dfa(*dfa))
        torch.cuda.synchronize()
        assert cstr.cstr_table_info(table)["start_state"] == dfa[2]
        assert whole_table_parity(table, dfa, vb, vo) > 0


def test_download_slabs_of_any_alignment():
    # the download decodes on the device in tiles of 32 states: ranges that start and end
    # anywhere, single rows, the last partial tile, and 32-bit entries
    rng = np.random.default_rng(31)
    vb, vo = random_vocab(rng, 1000)
    for S in (70, 300):
        dfa = dense_random_dfa(rng, S, live=0.8)
        (table,) = gpu_tables([dfa], vb, vo)
        full_next, full_mask = oracle.token_table(dfa[0], dfa[1], vb, vo)
        for lo, hi in [(0, S), (1, 2), (31, 33), (S - 1, S), (5, 69), (33, 64), (7, 7)]:
            nxt, mask = cstr.cstr_table_download(table, lo, hi)
            assert np.array_equal(nxt, full_next[lo:hi]) and np.array_equal(mask, full_mask[lo:hi])
        nxt, _ = cstr.cstr_table_download(table, 3, 40, want_mask=False)
        assert np.array_equal(nxt, full_next[3:40])


def test_small_constraints_over_the_256k_vocabulary():
    # The small-constraint compiles the benchmark times (2 to 56 states over 256,000 tokens:
    # the lane = token kernels and the smallest trie-walker variant), whole tables.
    from synth import constraints
    vb, vo = config_vocab("string_256k")
    pats = dict(constraints.SMALL_CONSTRAINTS)
    pats["api_call"] = constraints.API_CALL_REGEX
    pats["flat_json"] = constraints.FLAT_JSON_REGEX
    dfas = [regex_to_dfa(p) for p in pats.values()]
    assert sorted(d[0].shape[0] for d in dfas) == [2, 11, 24, 26, 56]
    tables = gpu_tables(dfas, vb, vo)
    for table, dfa in zip(tables, dfas):
        check_table(table, dfa, vb, vo)


def test_long_shared_prefixes_and_long_suffixes():
    # Tokens that share far more than the 8 bytes the walk keeps on its stack,
    # suffixes longer than the 8 bytes carried inline, exact duplicates, and a
    # vocabulary order that is the reverse of the trie order.
    rng = np.random.default_rng(77)
    base = bytes(rng.integers(97, 100, size=60).astype(np.uint8))
    toks = []
    for _ in range(1500):
        p = int(rng.integers(0, 60))
        s = bytes(rng.integers(97, 100, size=int(rng.integers(0, 25))).astype(np.uint8))
        toks.append(base[:p] + s)
    toks += toks[:100]                                   # duplicates
    toks = sorted(toks, reverse=True)
    vb, vo = vocab_from_strings(toks)
    S = 700
    trans = rng.integers(0, S, size=(S, 256)).astype(np.int32)
    trans[:, :97] = -1
    trans[:, 100:] = -1
    trans[rng.random((S, 256)) < 0.03] = -1              # long walks mostly survive
    dfa = (trans, (rng.random(S) < 0.3).astype(np.uint8), 0)
    (table,) = gpu_tables([dfa], vb, vo)
    check_table(table, dfa, vb, vo)
    # the same vocabulary against a counter-like chain (neighbouring states stay neighbours)
    S = 300
    chain = np.full((S, 256), -1, dtype=np.int32)
    for q in range(S):
        chain[q, 97] = (q + 1) % S
        chain[q, 98] = q
        chain[q, 99] = (q * 7 + 3) % S
    dfa = (chain, np.ones(S, dtype=np.uint8), 5)
    (table,) = gpu_tables([dfa], vb, vo)
    check_table(table, dfa, vb, vo)


@pytest.mark.parametrize("case", ["string", "two_classes", "one_class", "eos_and_terminals"])
def test_few_byte_classes_take_the_duplicate_column_pass(case):
    # Automata of >= 2,048 states with at most 16 byte classes over >= 8,192 tokens share
    # one walk per class string; every column must still be the oracle's, copies included.
    from synth import make_vocab_geometric
    rng = np.random.default_rng(11)
    vb, vo = make_vocab_geometric(9000 if case != "string" else 20000, seed=5)
    V = vo.size - 1
    eos, term, sets = -1, None, None
    if case == "string":
        dfa = regex_to_dfa(r'"([^"\\]|\\.){0,1100}"')        # 3 classes, 2,203 states
    elif case == "two_classes":
        dfa = regex_to_dfa(r"([a-z ]{3}[^a-z ]){0,600}")
    elif case == "one_class":
        dfa = regex_to_dfa(r".{0,2100}")
    else:
        full = regex_to_dfa(r'x(?P<WORD>)+"[^"]{0,2050}"', ["WORD"])
        dfa = (np.ascontiguousarray(full[0][:, :256]), full[1], full[2])
        term = [np.ascontiguousarray(full[0][:, 256:])]
        sets = (rng.random(V) < 0.3).astype(np.uint32)
        eos = 4242                                             # a token equal to many others
    toks = [bytes(vb[vo[v]:vo[v + 1]]) for v in range(V)]
    assert len(set(toks)) < V                                  # the vocabulary repeats strings
    (table,) = gpu_tables([dfa], vb, vo, eos_id=eos, term_trans=term, token_sets=sets)
    S = dfa[0].shape[0]
    assert S >= 2048
    sample = sorted(set([0, 1, 2, 255, 256, 257, S - 3, S - 2, S - 1] + rng.integers(0, S, 40).tolist()))
    check_table(table, dfa, vb, vo, eos_id=eos, states=sample,
                term_trans=None if term is None else term[0], token_sets=sets)
    # rebuilding into the same table reuses the grouping scratch
    h = (cstr.cstr_load_dfa_terminals(dfa[0], term[0], dfa[1], dfa[2]) if term is not None
         else cstr.cstr_load_dfa(*dfa))
    cstr.cstr_table_build(table, h, eos)
    torch.cuda.synchronize()
    check_table(table, dfa, vb, vo, eos_id=eos, states=[0, dfa[0].shape[0] - 1],
                term_trans=None if term is None else term[0], token_sets=sets)


def test_duplicate_column_pass_wide_entries_and_table_reuse():
    # 32-bit next entries (more than 32,766 states) through the duplicate-column pass, then the
    # same table rebuilt for automata that take the plain walk (many byte classes; few states).
    from synth import make_vocab_geometric
    vb, vo = make_vocab_geometric(8200, seed=9)
    vocab = cstr.cstr_load_vocab(vb, vo)
    wide = regex_to_dfa(r"[a-z ]{0,33000}")
    S = wide[0].shape[0]
    assert S > 32767
    table = cstr.cstr_table_create(vocab, S)
    cstr.cstr_table_build(table, cstr.cstr_load_dfa(*wide))
    torch.cuda.synchronize()
    check_table(table, wide, vb, vo, states=[0, 1, 255, 256, 12345, 32766, 32767, 32768, S - 2, S - 1])
    rng = np.random.default_rng(4)
    many = dense_random_dfa(rng, 300, live=0.6)                      # 256 byte classes
    cstr.cstr_table_build(table, cstr.cstr_load_dfa(*many))
    torch.cuda.synchronize()
    check_table(table, many, vb, vo, states=[0, 1, 150, 299])
    small = regex_to_dfa(r'"[^"]{0,40}"')                            # few classes, few states
    cstr.cstr_table_build(table, cstr.cstr_load_dfa(*small))
    torch.cuda.synchronize()
    check_table(table, small, vb, vo)
    cstr.cstr_table_build(table, cstr.cstr_load_dfa(*wide), 300)      # and back, with an EOS token
    torch.cuda.synchronize()
    check_table(table, wide, vb, vo, eos_id=300, states=[0, 77, S - 1])


def test_load_dfa_reports_bad_targets_and_reuses_its_scratch():
    # the target check runs on the device; the message still names the first bad entry,
    # and loads of different sizes in a row (the per-thread scratch shrinks and grows) stay exact
    trans = np.full((300, 256), -1, dtype=np.int32)
    acc = np.zeros(300, dtype=np.uint8)
    trans[299, 255] = 300
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_load_dfa(trans, acc, 0)
    assert e.value.code == -3 and "state 299 byte 255" in str(e.value)
    trans[299, 255] = -2
    with pytest.raises(cstr.CstrError) as e:
        cstr.cstr_load_dfa(trans, acc, 0)
    assert e.value.code == -3
    rng = np.random.default_rng(8)
    vb, vo = random_vocab(rng, 700)
    for S in (5, 900, 40, 2000, 3):
        dfa = dense_random_dfa(rng, S, live=0.8)
        (table,) = gpu_tables([dfa], vb, vo)
        check_table(table, dfa, vb, vo, states=sorted(set([0, S // 2, S - 1])))


@pytest.fixture
def check_build():
    """Route the test through the checking build (bounds-checked kernels, test setters); the
    bounds record must be clean before and after."""
    cstr.use_check_library(True)
    try:
        cstr.cstr_debug_bounds_status(reset=True)
        yield
        torch.cuda.synchronize()
        record = cstr.cstr_debug_bounds_status(reset=True)
        cstr.cstr_test_set_group_hash_bits(0)
        assert record[0] == 0, "out-of-range index: site %d, index %d, extent %d" % record[1:]
    finally:
        cstr.use_check_library(False)


@pytest.mark.parametrize("bits", [3, 12])
def test_duplicate_column_pass_survives_hash_collisions(check_build, bits):
    # with only a few hash bits kept, tokens of different class strings land in the same group;
    # the exact comparison must then leave them on their own, and the table stays the oracle's
    from synth import make_vocab_geometric
    cstr.cstr_test_set_group_hash_bits(bits)
    vb, vo = make_vocab_geometric(9000, seed=5)
    dfa = regex_to_dfa(r'"([^"\\]|\\.){0,1100}"')
    (table,) = gpu_tables([dfa], vb, vo, eos_id=17)
    S = dfa[0].shape[0]
    rng = np.random.default_rng(bits)
    check_table(table, dfa, vb, vo, eos_id=17,
                states=sorted(set([0, 1, S - 1] + rng.integers(0, S, 20).tolist())))


@pytest.mark.parametrize("n_states", [32766, 32767])
def test_entry_width_boundary(n_states):
    # 32,766 states are the most that 16-bit entries hold (the sink takes one more code);
    # one state more switches the DFA and the table to 32-bit entries
    trans = np.full((n_states, 256), -1, dtype=np.int32)
    q = np.arange(n_states - 1)
    trans[q, 0x61] = q + 1                          # a chain on 'a' ...
    trans[:, 0x62] = np.arange(n_states)[::-1]      # ... and 'b' jumps to the mirrored state
    acc = np.zeros(n_states, dtype=np.uint8)
    acc[-1] = 1
    dfa = (trans, acc, 0)
    toks = [b"a", b"aa", b"b", b"ab", b"ba", b"bab", b"c", b"", b"a" * 40, b"aba" * 5] + \
           [bytes([c]) for c in range(256)]
    vb, vo = vocab_from_strings(toks)
    (table,) = gpu_tables([dfa], vb, vo, eos_id=6)
    S = n_states
    check_table(table, dfa, vb, vo, eos_id=6,
                states=[0, 1, 2, 255, 256, 16383, 16384, S - 42, S - 41, S - 3, S - 2, S - 1])
    nxt, _ = cstr.cstr_table_download(table, S - 2, S)
    assert nxt[0, 0] == S - 1 and nxt[1, 0] == -1 and nxt[1, 2] == 0


@pytest.mark.parametrize("S", [4, 16, 17, 25, 32, 33, 64, 65])
def test_small_automaton_kernels(S):
    # up to 16 states: lane = token with ballots; 17..64: lane = token over tokens of equal
    # length + transpose; 65: the trie walker.  Long tokens, empty tokens, an EOS token.
    rng = np.random.default_rng(S)
    dfa = dense_random_dfa(rng, S, live=0.85)
    vb, vo = random_vocab(rng, 1500 + S, max_len=40)
    eos = int(rng.integers(vo.size - 1))
    (table,) = gpu_tables([dfa], vb, vo, eos_id=eos)
    check_table(table, dfa, vb, vo, eos_id=eos)
    (table,) = gpu_tables([dfa], vb, vo)
    check_table(table, dfa, vb, vo)


@pytest.mark.parametrize("case", ["small", "eos_long_tokens", "json_32k", "wide"])
def test_dense_walker_baseline_gives_the_same_table(case):
    # cstr_table_build_dense (every token from its first byte, no trie) exists to measure
    # what the trie walk saves; it must produce the oracle's table too
    rng = np.random.default_rng(61)
    eos, states = -1, None
    if case == "small":
        dfa = dense_random_dfa(rng, 70, live=0.7)
        vb, vo = random_vocab(rng, 1500, max_len=20)
    elif case == "eos_long_tokens":
        dfa = dense_random_dfa(rng, 300, live=0.95)
        vb, vo = random_vocab(rng, 700, max_len=40)
        eos = 33
    elif case == "json_32k":
        dfa = config_dfas("json_32k")[0]
        vb, vo = config_vocab("json_32k")
    else:
        dfa = random_range_dfa(33000, seed=9)
        vb, vo = random_vocab(rng, 200, max_len=4)
        states = [0, 1, 255, 256, 32766, 32767, 32768, 32999]
    vocab = cstr.cstr_load_vocab(vb, vo)
    table = cstr.cstr_table_create(vocab, dfa[0].shape[0])
    cstr.cstr_table_build_dense(table, cstr.cstr_load_dfa(*dfa), eos)
    torch.cuda.synchronize()
    check_table(table, dfa, vb, vo, eos_id=eos, states=states)


def sparse_dfa(rng, S, many_every=37):
    """Mostly picky states (1-3 edges each) with a state that allows nearly every byte now and
    then: the shape of a schema constraint (fixed keys and punctuation around free text)."""
    trans = np.full((S, 256), -1, dtype=np.int32)
    for q in range(S):
        if q % many_every == 3:
            trans[q] = rng.integers(0, S, size=256)
            trans[q, rng.random(256) < 0.1] = -1
        else:
            for b in rng.choice(np.arange(97, 123), size=int(rng.integers(1, 4)), replace=False):
                trans[q, b] = int(rng.integers(0, S))
    return trans, (rng.random(S) < 0.3).astype(np.uint8), int(rng.integers(S))


@pytest.mark.parametrize("case", ["plain", "eos", "terminals", "wide", "dense_walker"])
def test_sparse_automata_are_renumbered_and_pruned(case):
    # More than 512 states, at least 256 of them picky, the states that allow many bytes
    # scattered among them: the library numbers those first internally and prunes dead trie
    # subtrees per warp.  Whole tables, then steps from random states (the step maps state
    # ids into and out of the internal numbering).
    from gpu_common import run_step_both
    rng = np.random.default_rng(91)
    S = 33100 if case == "wide" else 1300
    dfa = sparse_dfa(rng, S)
    V = 3000
    vb, vo = random_vocab(rng, V, max_len=12, alphabet=b"abcdefghijklmnopqrstuvwxyz ", empty_prob=0.01)
    eos = 77 if case in ("eos", "terminals") else -1
    term, sets = None, None
    if case == "terminals":
        term = np.full((S, 2), -1, dtype=np.int32)
        for q in range(0, S, 11):
            term[q, int(rng.integers(2))] = int(rng.integers(S))
        sets = rng.integers(0, 4, size=V).astype(np.uint32)
    if case == "dense_walker":
        vocab = cstr.cstr_load_vocab(vb, vo)
        table = cstr.cstr_table_create(vocab, S)
        cstr.cstr_table_build_dense(table, cstr.cstr_load_dfa(*dfa), eos)
        torch.cuda.synchronize()
        tables = [table]
    else:
        tables = gpu_tables([dfa], vb, vo, eos_id=eos, term_trans=None if term is None else [term],
                            token_sets=sets)
    states = None
    if case == "wide":
        states = sorted(set([0, 1, 2, 3, 40, 255, 256, 32767, 32768, S - 1] +
                            rng.integers(0, S, 30).tolist()))
    check_table(tables[0], dfa, vb, vo, eos_id=eos, states=states, term_trans=term, token_sets=sets)
    B = 64
    logits = rng.standard_normal((B, V)).astype(np.float32)
    st = rng.integers(-1, S, size=B).astype(np.int32)
    st[:8] = [3, 40, 77, 0, 1, S - 1, -1, S]            # many-byte states, picky ones, bad ones
    for _ in range(3):
        ref = run_step_both([dfa], tables, vb, vo, logits, st, eos_id=eos,
                            term_trans=None if term is None else [term], token_sets=sets)
        st = ref["states"]
        logits = rng.standard_normal((B, V)).astype(np.float32)


@pytest.mark.parametrize("block", range(6))
def test_randomised_automaton_and_vocabulary_shapes(block):
    # Many shapes in one go: automata that are dense, byte-range, sparse (with and without
    # scattered many-byte states) or of a few byte classes, of 1 to 9,300 states (every builder
    # kernel and both sides of each threshold), against vocabularies over 256 / 27 / 2 symbols
    # with many repeated strings, in sorted, reverse-sorted or random order, with and without EOS.
    for case in range(25):
        rng = np.random.default_rng(7000 + 25 * block + case)
        kind = str(rng.choice(["dense", "range", "sparse", "fewclass"]))
        S = int(rng.choice([1, 2, 15, 16, 17, 63, 64, 65, 200, 255, 256, 257, 511, 512, 513, 700, 1300,
                            2049, 2500, 9000, 9300]))
        if kind == "fewclass" and rng.random() < 0.5:
            S = int(rng.choice([2048, 2300, 4100]))
        V = int(rng.choice([1, 31, 33, 700, 2049, 8200, 9000]))
        alphabet = [None, b"abcdefghijklmnopqrstuvwxyz ", b"ab"][int(rng.integers(3))]
        vb, vo = random_vocab(rng, V, max_len=int(rng.choice([3, 12, 40])), alphabet=alphabet,
                              empty_prob=0.01)
        toks = [bytes(vb[vo[v]:vo[v + 1]]) for v in range(V)]
        dup = float(rng.choice([0.0, 0.3, 0.7]))
        for v in range(1, V):                            # repeated strings
            if rng.random() < dup:
                toks[v] = toks[int(rng.integers(v))]
        if rng.random() < 0.5:
            toks.sort(reverse=bool(rng.random() < 0.5))
        vb, vo = vocab_from_strings(toks)
        if kind == "dense":
            dfa = dense_random_dfa(rng, S, live=float(rng.choice([0.3, 0.7, 1.0])))
        elif kind == "range":
            dfa = random_range_dfa(S, seed=int(rng.integers(1 << 30)))
        elif kind == "sparse":
            dfa = sparse_dfa(rng, S, many_every=int(rng.choice([7, 37, 101, 10 ** 9])))
        else:
            k = int(rng.integers(1, 5))
            cls = rng.integers(0, k, size=256)
            base = rng.integers(-1, S, size=(S, k)).astype(np.int32)
            dfa = (np.ascontiguousarray(base[:, cls]), (rng.random(S) < 0.3).astype(np.uint8),
                   int(rng.integers(S)))
        eos = int(rng.integers(-1, V)) if rng.random() < 0.4 else -1
        (table,) = gpu_tables([dfa], vb, vo, eos_id=eos)
        states = None
        if S * V > 6_000_000:
            states = sorted(set([0, 1, S - 1] + rng.integers(0, S, 40).tolist()))
        check_table(table, dfa, vb, vo, eos_id=eos, states=states, slab=max(S, 1))
