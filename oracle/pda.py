"""ORACLE (test infrastructure, not product code): push-down constraints.

Python access to ``pda_oracle.c``, the plain CPU statement of Section 3 of the
paper: PDA acceptance by the definition, the edges of the token-level PDA
P_{G o V} (composition with the detokenizing transducer), the allowed set A of
Algorithm 3 for a given state and stack, and the loop body of Algorithm 3 for a
batch of rows.  A PDA is any object with the flat edge arrays of
``synth.pda.Pda``.  Nothing here is used by the product.
"""

from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pda_oracle.c")
_LIB = os.path.join(_HERE, "_pda_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_pda_accepts.restype = None
        _lib.oracle_pda_token_edges.restype = ctypes.c_int32
        _lib.oracle_pda_allowed.restype = ctypes.c_int32
        _lib.oracle_pda_step.restype = None
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _pda_args(pda):
    """The eleven leading arguments every C entry point takes; keeps the arrays alive."""
    arrs = [np.ascontiguousarray(getattr(pda, n), dtype=np.int32)
            for n in ("src", "inp", "tgt", "pop_off", "pops", "push_off", "pushes")]
    accept = np.ascontiguousarray(pda.accept, dtype=np.uint8)
    n_edges = arrs[0].size
    assert arrs[3].size == n_edges + 1 and arrs[5].size == n_edges + 1
    assert accept.size == pda.n_states
    if n_edges:
        assert 0 <= arrs[0].min() and arrs[0].max() < pda.n_states
        assert 0 <= arrs[2].min() and arrs[2].max() < pda.n_states
        assert 0 <= arrs[1].min() and arrs[1].max() < 256
    args = [ctypes.c_int32(pda.n_states), ctypes.c_int32(pda.n_symbols), ctypes.c_int32(n_edges)]
    args += [_ptr(a) for a in arrs] + [_ptr(accept)]
    return args, arrs + [accept]


def accepts(pda, words, init_stack=(), threads: int = 1) -> np.ndarray:
    """``words``: list of byte strings.  Returns uint8 flags: accepted by the
    definition of Section 3.1, starting at ``pda.start`` with ``init_stack``."""
    args, keep = _pda_args(pda)
    words = [bytes(w) for w in words]
    woff = np.zeros(len(words) + 1, dtype=np.int64)
    np.cumsum([len(w) for w in words], out=woff[1:])
    data = np.frombuffer(b"".join(words) + b"\0", dtype=np.uint8).copy()
    init = np.ascontiguousarray(list(init_stack) + [0], dtype=np.int32)
    out = np.zeros(len(words), dtype=np.uint8)
    _load().oracle_pda_accepts(*args, ctypes.c_int32(pda.start), _ptr(init),
                               ctypes.c_int32(len(init_stack)), _ptr(data), _ptr(woff),
                               ctypes.c_int64(len(words)), _ptr(out), ctypes.c_int32(threads))
    return out


def token_edges(pda, q: int, token: bytes, max_edges: int = 256):
    """Edges of the token-level PDA leaving ``q`` on ``token``:
    list of (target, pops tuple (top last), pushes tuple)."""
    args, keep = _pda_args(pda)
    stride = 3 + 80 + 400
    out = np.zeros((max_edges, stride), dtype=np.int32)
    data = np.frombuffer(bytes(token) + b"\0", dtype=np.uint8).copy()
    n = _load().oracle_pda_token_edges(*args, ctypes.c_int32(q), _ptr(data),
                                       ctypes.c_int64(len(token)), _ptr(out),
                                       ctypes.c_int32(stride), ctypes.c_int32(max_edges))
    if n < 0:
        raise RuntimeError("token edge enumeration exceeded its bounds")
    res = []
    for i in range(n):
        t, npop, npush = (int(x) for x in out[i, :3])
        res.append((t, tuple(int(x) for x in out[i, 3:3 + npop]),
                    tuple(int(x) for x in out[i, 3 + npop:3 + npop + npush])))
    return res


def _pack_stacks(stacks, cap):
    n = len(stacks)
    arr = np.zeros((n, max(cap, 1)), dtype=np.int32)
    depth = np.zeros(n, dtype=np.int32)
    for i, s in enumerate(stacks):
        depth[i] = len(s)
        arr[i, :len(s)] = list(s)
    return arr, depth


def allowed(pda, vocab_bytes, offsets, states, stacks, eos_id: int = -1, threads: int = 1):
    """Allowed-token bitmasks (uint32 ``[n][ceil(V/32)]``, LSB = lowest id) for
    the situations ``(states[i], stacks[i])``; a stack is a sequence, top last."""
    args, keep = _pda_args(pda)
    vocab_bytes = np.ascontiguousarray(vocab_bytes, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    V = offsets.size - 1
    states = np.ascontiguousarray(states, dtype=np.int32)
    assert states.min() >= 0 and states.max() < pda.n_states
    cap = max([len(s) for s in stacks] + [1])
    arr, depth = _pack_stacks(stacks, cap)
    mask = np.zeros((len(stacks), (V + 31) // 32), dtype=np.uint32)
    rc = _load().oracle_pda_allowed(*args, _ptr(vocab_bytes), _ptr(offsets), ctypes.c_int32(V),
                                    ctypes.c_int32(eos_id), _ptr(states), _ptr(arr), _ptr(depth),
                                    ctypes.c_int32(cap), ctypes.c_int32(len(stacks)), _ptr(mask),
                                    ctypes.c_int32(threads))
    if rc:
        raise RuntimeError("token edge enumeration exceeded its bounds")
    return mask


def step(pda, vocab_bytes, offsets, logits, states, stacks, depth, noise=None, eos_id: int = -1,
         vocab_size: int | None = None, threads: int = 1):
    """One step of Algorithm 3 on the CPU.  ``stacks`` int32 ``[B][cap]`` and
    ``depth`` int32 ``[B]`` (inputs are not modified).  Returns dict(tokens,
    states, stacks, depth, masked, accept, bad_state_rows, empty_mask_rows,
    overflow_rows)."""
    args, keep = _pda_args(pda)
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
    st = np.array(states, dtype=np.int32, copy=True)
    sk = np.array(stacks, dtype=np.int32, copy=True, order="C")
    dp = np.array(depth, dtype=np.int32, copy=True)
    assert sk.ndim == 2 and sk.shape[0] == B and st.shape == (B,) and dp.shape == (B,)
    cap = sk.shape[1]
    tokens = np.empty(B, dtype=np.int32)
    masked = logits.copy()
    acc_out = np.empty(B, dtype=np.uint8)
    counters = np.zeros(4, dtype=np.int64)
    _load().oracle_pda_step(*args, _ptr(vocab_bytes), _ptr(offsets), ctypes.c_int32(V),
                            ctypes.c_int32(eos_id), _ptr(logits), ctypes.c_int32(dtype),
                            ctypes.c_int64(ld), _ptr(noise), _ptr(st), _ptr(sk), _ptr(dp),
                            ctypes.c_int32(cap), _ptr(tokens), _ptr(masked), _ptr(acc_out),
                            ctypes.c_int32(B), _ptr(counters), ctypes.c_int32(threads))
    if counters[3]:
        raise RuntimeError("token edge enumeration exceeded its bounds")
    return dict(tokens=tokens, states=st, stacks=sk, depth=dp, masked=masked, accept=acc_out,
                bad_state_rows=int(counters[0]), empty_mask_rows=int(counters[1]),
                overflow_rows=int(counters[2]))


def accept_draft(draft_tokens, target_tokens, target_states, target_stacks, target_depths):
    """Greedy verification and rewind under a push-down constraint (Section 4): the
    kept prefix and the emitted tokens are those of the finite-state rule
    (``oracle.accept_draft``); the constraint goes back to the whole situation
    - state, stack and depth - that followed the last token kept.
    ``target_stacks`` int32 ``[B][k+1][cap]``, the others ``[B][k+1]`` / ``[B][k]``.
    Returns (n_accepted, out_tokens, states, stacks [B][cap], depths)."""
    import oracle
    n, out, states = oracle.accept_draft(draft_tokens, target_tokens, target_states)
    target_stacks = np.asarray(target_stacks, dtype=np.int32)
    target_depths = np.asarray(target_depths, dtype=np.int32)
    rows = np.arange(n.size)
    return n, out, states, target_stacks[rows, n].copy(), target_depths[rows, n].copy()
