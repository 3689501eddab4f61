"""Pins for the oracle's constrained decoding step (CPU only)."""
import numpy as np
import pytest

import oracle
from oracle import regex_dfa as rd
from synth import (bf16_bits_to_f32, f32_to_bf16_bits, gumbel_noise, normal_logits,
                   vocab_from_strings)
from synth.configs import CONFIGS, config_dfas, config_vocab

NEG_INF_BITS = np.uint32(0xFF800000)


def allowed_matrix(dfa, vb, vo, states):
    """Brute-force validity by walking bytes in Python (independent of the C code)."""
    trans = dfa[0]
    V = vo.size - 1
    out = np.zeros((len(states), V), dtype=bool)
    for r, q in enumerate(states):
        if q < 0 or q >= trans.shape[0]:
            continue
        for v in range(V):
            s = int(q)
            if vo[v + 1] == vo[v]:
                continue
            for b in vb[vo[v]:vo[v + 1]]:
                s = int(trans[s, b])
                if s < 0:
                    break
            out[r, v] = s >= 0
    return out


def test_penalise_and_select_against_numpy():
    # Valid positions are bit copies, invalid ones exactly -inf, and
    # the selected token is numpy's first-occurrence argmax over the masked values.
    w = CONFIGS["api_1k"]
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    V = vo.size - 1
    rng = np.random.default_rng(3)
    states = rng.integers(0, dfa[0].shape[0], size=16).astype(np.int32)
    logits = normal_logits(7, 0, range(16), V)
    for noise in (None, gumbel_noise(1, 0, range(16), V)):
        res = oracle.step([dfa], vb, vo, logits, states, noise=noise)
        ok = allowed_matrix(dfa, vb, vo, states)
        m = res["masked"]
        assert (m.view(np.uint32)[ok] == logits.view(np.uint32)[ok]).all()
        assert (m.view(np.uint32)[~ok] == NEG_INF_BITS).all()
        score = logits if noise is None else (logits + noise).astype(np.float32)
        for r in range(16):
            if ok[r].any():
                want = int(np.argmax(np.where(ok[r], score[r], -np.inf)))
                assert res["tokens"][r] == want
            else:
                assert res["tokens"][r] == -1 and res["states"][r] == -1


def test_decode_loop_tracks_the_byte_dfa():
    # After every step, the bytes emitted so far, run through the byte DFA from
    # its start state, land on the reported state.
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    V = vo.size - 1
    B = 8
    states = np.full(B, dfa[2], dtype=np.int32)
    texts = [bytearray() for _ in range(B)]
    finished = np.zeros(B, dtype=bool)
    for t in range(32):
        logits = normal_logits(11, t, range(B), V)
        res = oracle.step([dfa], vb, vo, logits, states, threads=2)
        for r in range(B):
            tok = int(res["tokens"][r])
            if finished[r]:
                assert tok == -1 and res["states"][r] == -1
                continue
            if tok < 0:
                finished[r] = True
                # only a state without outgoing tokens may stall; it must accept
                q = dfa[2]
                for b in texts[r]:
                    q = int(dfa[0][q, b])
                assert (dfa[0][q] < 0).all() and dfa[1][q]
                continue
            texts[r] += bytes(vb[vo[tok]:vo[tok + 1]])
            q = dfa[2]
            for b in texts[r]:
                q = int(dfa[0][q, b])
                assert q >= 0
            assert q == res["states"][r]
            assert res["accept"][r] == dfa[1][q]
        states = res["states"]


def tiny():
    dfa = rd.compile_regex("(a|b)*c")
    toks = [b"a", b"b", b"c", b"ab", b"zz", b"bc", b"ca"]
    return dfa, toks, vocab_from_strings(toks)


def test_ties_go_to_the_lowest_index():
    dfa, toks, (vb, vo) = tiny()
    logits = np.array([[1.0, 1.0, 1.0, 1.0, 9.0, 1.0, 9.0],
                       [0.0, -0.0, 0.0, -0.0, 9.0, 0.0, 9.0],
                       [-0.0, 0.0, 0.0, 0.0, 9.0, 0.0, 9.0]], dtype=np.float32)
    res = oracle.step([dfa], vb, vo, logits, [dfa[2]] * 3)
    assert res["tokens"].tolist() == [0, 0, 0]         # zz and ca are not allowed
    logits[:, 0] = -5
    res = oracle.step([dfa], vb, vo, logits, [dfa[2]] * 3)
    assert res["tokens"].tolist() == [1, 1, 1]


def test_nan_inf_rules():
    dfa, toks, (vb, vo) = tiny()
    nan, inf = np.float32(np.nan), np.float32(np.inf)
    logits = np.array([[nan, nan, -inf, -inf, inf, -inf, inf],     # -inf valid still wins over nothing
                       [nan, nan, nan, nan, 1, nan, 1],            # all valid are NaN: no token
                       [nan, 2, inf, 1, 0, inf, 0],                # +inf, first occurrence
                       [3, nan, 1, 1, 0, 1, 0]], dtype=np.float32)
    res = oracle.step([dfa], vb, vo, logits, [dfa[2]] * 4)
    assert res["tokens"].tolist() == [2, -1, 2, 0]
    assert res["states"][1] == -1 and res["empty_mask_rows"] == 1
    # NaN payloads of allowed positions pass through untouched
    assert res["masked"].view(np.uint32)[1, 0] == logits.view(np.uint32)[1, 0]
    # noise can create the NaN (inf + -inf) and it must lose too
    logits = np.array([[inf, 0, 0, 0, 0, 0, 0]], dtype=np.float32)
    noise = np.array([[-inf, 0, 1, 0, 0, 0, 0]], dtype=np.float32)
    res = oracle.step([dfa], vb, vo, logits, [dfa[2]], noise=noise)
    assert res["tokens"].tolist() == [2]


def test_inactive_and_bad_rows():
    dfa, toks, (vb, vo) = tiny()
    S = dfa[0].shape[0]
    logits = normal_logits(5, 0, range(4), 7)
    res = oracle.step([dfa], vb, vo, logits, [-1, S, -7, dfa[2]])
    assert res["tokens"][:3].tolist() == [-1, -1, -1]
    assert res["states"][:3].tolist() == [-1, -1, -1]
    assert (res["masked"].view(np.uint32)[:3] == NEG_INF_BITS).all()
    assert res["bad_state_rows"] == 2 and res["empty_mask_rows"] == 0
    assert res["tokens"][3] >= 0
    # accepting state of (a|b)*c has no outgoing token: active row, empty mask
    acc_state = int(np.nonzero(dfa[1])[0][0])
    res = oracle.step([dfa], vb, vo, logits[:1], [acc_state])
    assert res["tokens"][0] == -1 and res["empty_mask_rows"] == 1


def test_eos_allowed_only_in_accepting_states():
    dfa = rd.compile_regex("ab?")
    toks = [b"a", b"b", b"<eos>"]
    vb, vo = vocab_from_strings(toks)
    big = np.array([[0.0, 0.0, 5.0]], dtype=np.float32)
    res = oracle.step([dfa], vb, vo, big, [dfa[2]], eos_id=2)
    assert res["tokens"][0] == 0                       # start state does not accept
    q1 = int(res["states"][0])
    res = oracle.step([dfa], vb, vo, big, [q1], eos_id=2)
    assert res["tokens"][0] == 2 and res["states"][0] == -1 and res["accept"][0] == 0


def test_bf16_path():
    dfa = config_dfas("api_1k")[0]
    vb, vo = config_vocab("api_1k")
    V = vo.size - 1
    lb = normal_logits(9, 0, range(6), V, sigma=2.0, dtype="bf16")
    states = np.array([0, 1, 2, 3, 4, 5], dtype=np.int32)
    res = oracle.step([dfa], vb, vo, lb, states)
    ok = allowed_matrix(dfa, vb, vo, states)
    assert (res["masked"][ok] == lb[ok]).all() and (res["masked"][~ok] == 0xFF80).all()
    wide = bf16_bits_to_f32(lb)
    for r in range(6):
        if ok[r].any():
            assert res["tokens"][r] == int(np.argmax(np.where(ok[r], wide[r], -np.inf)))
    # bf16 rounding helper: round-to-nearest-even on a few hand values
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.0e38], dtype=np.float32)
    assert f32_to_bf16_bits(x).tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x7F62]


def test_mixed_tables_and_padding_columns():
    d0 = rd.compile_regex("a*b")
    d1 = rd.compile_regex("[bc]+")
    toks = [b"a", b"b", b"c", b"ab", b"cc"]
    vb, vo = vocab_from_strings(toks)
    ld = 8
    logits = np.zeros((4, ld), dtype=np.float32)
    logits[:, :5] = [0.1, 0.2, 0.3, 0.9, 0.5]
    logits[:, 5:] = 77.0                                # padding must be ignored
    res = oracle.step([d0, d1], vb, vo, logits, [0, 0, 0, 0],
                      row_table=np.array([0, 1, 1, 0], dtype=np.int32), vocab_size=5)
    assert res["tokens"].tolist() == [3, 4, 4, 3]
    assert (res["masked"][:, 5:] == 77.0).all()
    res_t = oracle.step([d0, d1], vb, vo, logits, [0, 0, 0, 0],
                        row_table=np.array([0, 1, 1, 0], dtype=np.int32), vocab_size=5, threads=4)
    assert (res_t["tokens"] == res["tokens"]).all()
