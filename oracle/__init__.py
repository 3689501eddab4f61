"""ORACLE (test infrastructure, not product code).

A plain, slow CPU statement of the path the CUDA library implements:

* ``regex_dfa``     regex -> Thompson NFA -> subset construction -> trim
                    (Algorithm 2, automaton construction; Section 2.1);
* ``token_table``   T[q][v] = delta*(q, bytes(v)) and the per-state allowed-token
                    bitmask (Algorithm 1 composed with the DFA, Theorem 2);
* ``step``          mask, penalise with -inf, select, advance for a batch of
                    rows (Algorithm 2, loop body);
* ``pda``           push-down constraints (Section 3): PDA acceptance, the
                    token-level PDA's edges, Algorithm 3's allowed set and step.

All but the first are plain C (``cstr_oracle.c``, ``pda_oracle.c``), compiled
with gcc on first use.
Nothing here shares code with the CUDA path and the product never calls it:
only tests, the smoke check and the benchmark's CPU-baseline leg do.
"""

from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import pda, regex_dfa  # noqa: F401

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cstr_oracle.c")
_LIB = os.path.join(_HERE, "_cstr_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    pda.build(force)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_max_threads.restype = ctypes.c_int
        _lib.oracle_token_table.restype = None
        _lib.oracle_step.restype = None
        _lib.oracle_accept_draft.restype = None
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_dfa(trans, accept):
    trans = np.ascontiguousarray(trans, dtype=np.int32)
    accept = np.ascontiguousarray(accept, dtype=np.uint8)
    assert trans.ndim == 2 and trans.shape[1] == 256 and accept.shape == (trans.shape[0],)
    return trans, accept


def _check_terminals(term_trans, token_sets, S, V):
    if term_trans is None:
        return None, 0, None
    term_trans = np.ascontiguousarray(term_trans, dtype=np.int32)
    assert term_trans.ndim == 2 and term_trans.shape[0] == S and term_trans.shape[1] <= 32
    token_sets = np.ascontiguousarray(token_sets, dtype=np.uint32)
    assert token_sets.shape == (V,)
    return term_trans, term_trans.shape[1], token_sets


def token_table(trans, accept, vocab_bytes, offsets, eos_id: int = -1,
                q_lo: int = 0, q_hi: int | None = None, threads: int = 1,
                term_trans=None, token_sets=None):
    """Returns (next int32 [q_hi-q_lo][V], mask uint32 [q_hi-q_lo][ceil(V/32)]).

    ``term_trans`` int32 ``[S][T]`` (terminal-label edges, -1 = none) and
    ``token_sets`` uint32 ``[V]`` (bit t: token belongs to label t) are optional."""
    lib = _load()
    trans, accept = _check_dfa(trans, accept)
    vocab_bytes = np.ascontiguousarray(vocab_bytes, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    S = trans.shape[0]
    V = offsets.size - 1
    q_hi = S if q_hi is None else q_hi
    assert 0 <= q_lo <= q_hi <= S
    W = (V + 31) // 32
    nxt = np.empty((q_hi - q_lo, V), dtype=np.int32)
    mask = np.empty((q_hi - q_lo, W), dtype=np.uint32)
    term_trans, n_term, token_sets = _check_terminals(term_trans, token_sets, S, V)
    lib.oracle_token_table(_ptr(trans), _ptr(accept), ctypes.c_int32(S), _ptr(term_trans),
                           ctypes.c_int32(n_term), _ptr(token_sets), _ptr(vocab_bytes),
                           _ptr(offsets), ctypes.c_int32(V), ctypes.c_int32(eos_id),
                           ctypes.c_int32(q_lo), ctypes.c_int32(q_hi), _ptr(nxt), _ptr(mask),
                           ctypes.c_int32(threads))
    return nxt, mask


def step(dfas, vocab_bytes, offsets, logits, states, noise=None, row_table=None,
         eos_id: int = -1, vocab_size: int | None = None, threads: int = 1,
         term_trans=None, token_sets=None):
    """One constrained decoding step on the CPU.

    dfas: list of (trans, accept[, start]); ``term_trans``: matching list of
    terminal-edge tables (or None), ``token_sets`` uint32 ``[V]``.  logits: float32 ``[B][ld]`` or uint16
    (bfloat16 bit patterns) ``[B][ld]``.  states: int32 ``[B]`` (not modified).
    Returns dict(tokens, states, masked, accept, bad_state_rows, empty_mask_rows);
    ``masked`` columns past the vocabulary keep the input values.
    """
    lib = _load()
    pairs = [_check_dfa(d[0], d[1]) for d in dfas]
    n = len(pairs)
    TransArr = ctypes.c_void_p * n
    trans_ptrs = TransArr(*[p[0].ctypes.data for p in pairs])
    acc_ptrs = TransArr(*[p[1].ctypes.data for p in pairs])
    n_states = np.array([p[0].shape[0] for p in pairs], dtype=np.int32)
    vocab_bytes = np.ascontiguousarray(vocab_bytes, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    V = offsets.size - 1 if vocab_size is None else vocab_size
    logits = np.ascontiguousarray(logits)
    if logits.dtype == np.float32:
        dtype = 0
    elif logits.dtype == np.uint16:
        dtype = 1
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits)")
    B, ld = logits.shape
    assert ld >= V
    if noise is not None:
        noise = np.ascontiguousarray(noise, dtype=np.float32)
        assert noise.shape == logits.shape
    if row_table is not None:
        row_table = np.ascontiguousarray(row_table, dtype=np.int32)
    term_ptrs, n_term, sets = None, None, None
    if term_trans is not None:
        terms = [np.ascontiguousarray(t, dtype=np.int32) for t in term_trans]
        term_ptrs = TransArr(*[t.ctypes.data for t in terms])
        n_term = np.array([t.shape[1] for t in terms], dtype=np.int32)
        sets = np.ascontiguousarray(token_sets, dtype=np.uint32)
        assert sets.shape == (offsets.size - 1,)
    st = np.array(states, dtype=np.int32, copy=True)
    tokens = np.empty(B, dtype=np.int32)
    masked = logits.copy()
    acc_out = np.empty(B, dtype=np.uint8)
    counters = np.zeros(2, dtype=np.int64)
    lib.oracle_step(trans_ptrs, acc_ptrs, _ptr(n_states), term_ptrs, _ptr(n_term), _ptr(sets),
                    ctypes.c_int32(n), _ptr(row_table),
                    _ptr(vocab_bytes), _ptr(offsets), ctypes.c_int32(V), ctypes.c_int32(eos_id),
                    _ptr(logits), ctypes.c_int32(dtype), ctypes.c_int64(ld), _ptr(noise),
                    _ptr(st), _ptr(tokens), _ptr(masked), _ptr(acc_out), ctypes.c_int32(B),
                    _ptr(counters), ctypes.c_int32(threads))
    return dict(tokens=tokens, states=st, masked=masked, accept=acc_out,
                bad_state_rows=int(counters[0]), empty_mask_rows=int(counters[1]))


def accept_draft(draft_tokens, target_tokens, target_states):
    """Greedy verification + rewind.  int32 arrays ``[B][k]``, ``[B][k+1]``, ``[B][k+1]``;
    returns (n_accepted [B], out_tokens [B][k+1], states [B])."""
    lib = _load()
    target_tokens = np.ascontiguousarray(target_tokens, dtype=np.int32)
    target_states = np.ascontiguousarray(target_states, dtype=np.int32)
    B, k1 = target_tokens.shape
    draft_tokens = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, k1 - 1)
    assert target_states.shape == (B, k1)
    n_acc = np.empty(B, dtype=np.int32)
    out = np.empty((B, k1), dtype=np.int32)
    st = np.empty(B, dtype=np.int32)
    lib.oracle_accept_draft(_ptr(draft_tokens), _ptr(target_tokens), _ptr(target_states),
                            ctypes.c_int32(k1 - 1), ctypes.c_int32(B), _ptr(n_acc), _ptr(out),
                            _ptr(st))
    return n_acc, out, st
