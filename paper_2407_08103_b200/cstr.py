"""Thin ctypes binding of libcstr (argument marshalling only).

Functions carry the names of the C entry points in ``include/cstr.h``; device
arrays are ``torch`` CUDA tensors (used here only as owners of device memory)
and streams are ``torch.cuda`` streams.  There is no CPU path: importing works
anywhere, but any call raises if ``libcstr.so`` cannot be loaded.
"""

from __future__ import annotations

import ctypes
import os

import numpy as np

from .build import CHECK_LIB_PATH, LIB_PATH

CSTR_F32 = 0
CSTR_BF16 = 1
CSTR_MAX_TABLES = 16
CSTR_STATIC_MAX_BATCH = 4096

EXPORTS = [
    "cstr_load_dfa", "cstr_load_dfa_terminals", "cstr_free_dfa", "cstr_load_vocab",
    "cstr_vocab_set_token_sets", "cstr_free_vocab",
    "cstr_table_create", "cstr_table_build", "cstr_table_build_dense", "cstr_build_token_table", "cstr_table_info",
    "cstr_table_download", "cstr_free_table", "cstr_workspace_create", "cstr_free_workspace",
    "cstr_step", "cstr_step_host", "cstr_step_history", "cstr_accept_draft", "cstr_step_status",
    "cstr_step_static", "cstr_last_error",
    "cstr_load_pda", "cstr_free_pda", "cstr_build_pda_table", "cstr_free_pda_table",
    "cstr_pda_table_rebuild", "cstr_pda_table_info", "cstr_pda_table_download",
    "cstr_pda_workspace_create",
    "cstr_free_pda_workspace", "cstr_pda_step", "cstr_pda_step_history",
    "cstr_pda_accept_draft", "cstr_pda_step_status",
]

# entry points of the checking build only (include/cstr_debug.h)
DEBUG_EXPORTS = ["cstr_debug_bounds_status", "cstr_test_set_group_hash_bits"]

_lib = None
_libs = {}            # path -> loaded library
_active_path = None   # None: the release library at LIB_PATH


class CstrError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("libcstr error %d: %s" % (code, message))
        self.code = code


def _load(path, debug):
    if path not in _libs:
        if not os.path.exists(path):
            raise RuntimeError(
                "%s is missing at %s: build it with `python -m paper_2407_08103_b200.build%s` "
                "(needs nvcc); there is no fallback path"
                % (os.path.basename(path), path, " --check" if debug else ""))
        L = ctypes.CDLL(path)
        for name in EXPORTS + (DEBUG_EXPORTS if debug else []):
            fn = getattr(L, name)
            fn.restype = ctypes.c_int
        L.cstr_last_error.restype = ctypes.c_char_p
        for name in ("cstr_free_dfa", "cstr_free_vocab", "cstr_free_table", "cstr_free_workspace",
                     "cstr_free_pda", "cstr_free_pda_table", "cstr_free_pda_workspace"):
            getattr(L, name).restype = None
        L.is_check_build = debug
        _libs[path] = L
    return _libs[path]


def lib():
    """The active library: libcstr.so (built in-tree by ``build.build_library``) unless
    ``use_check_library(True)`` selected the checking build.  Fails loudly if absent."""
    global _lib
    if _lib is None:
        _lib = _load(LIB_PATH, False) if _active_path is None else _load(_active_path, True)
    return _lib


def use_check_library(on: bool) -> None:
    """Route every later call through ``libcstr_check.so`` (bounds-checked kernels, test
    setters) or back through the release library.  Handles stay bound to the library that
    made them; do not mix handles of the two in one call."""
    global _lib, _active_path
    _active_path = CHECK_LIB_PATH if on else None
    _lib = None


def cstr_debug_bounds_status(reset: bool = True):
    """Checking build only: (violations, site, index, extent) of the device's bounds record."""
    L = lib()
    if not getattr(L, "is_check_build", False):
        raise RuntimeError("cstr_debug_bounds_status needs the checking build (use_check_library)")
    out = (ctypes.c_uint64 * 4)()
    _check(L.cstr_debug_bounds_status(out, ctypes.c_int32(1 if reset else 0)))
    return tuple(int(x) for x in out)


def cstr_test_set_group_hash_bits(bits: int) -> None:
    """Checking build only: keep ``bits`` bits of the duplicate-column pass's hash (0 = all)."""
    L = lib()
    if not getattr(L, "is_check_build", False):
        raise RuntimeError("cstr_test_set_group_hash_bits needs the checking build")
    _check(L.cstr_test_set_group_hash_bits(ctypes.c_int32(bits)))


def _check(rc):
    if rc != 0:
        raise CstrError(rc, lib().cstr_last_error().decode("utf-8", "replace"))


def _np_ptr(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _dev_ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class _Handle:
    _free = None

    def __init__(self, ptr):
        self.ptr = ptr
        self._owner = lib() if ptr else None      # freed by the library that made it

    def close(self):
        if self.ptr:
            getattr(self._owner, self._free)(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Dfa(_Handle):
    _free = "cstr_free_dfa"


class Vocab(_Handle):
    _free = "cstr_free_vocab"


class Table(_Handle):
    _free = "cstr_free_table"
    vocab = None  # keeps the vocabulary handle alive


class Workspace(_Handle):
    _free = "cstr_free_workspace"


class Pda(_Handle):
    _free = "cstr_free_pda"


class PdaTable(_Handle):
    _free = "cstr_free_pda_table"
    pda = None    # keep the handles the table refers to alive
    vocab = None


class PdaWorkspace(_Handle):
    _free = "cstr_free_pda_workspace"


def cstr_load_dfa(trans, accept, start_state=0) -> Dfa:
    trans = np.ascontiguousarray(trans, dtype=np.int32)
    accept = np.ascontiguousarray(accept, dtype=np.uint8)
    if trans.ndim != 2 or trans.shape[1] != 256 or accept.shape != (trans.shape[0],):
        raise ValueError("trans must be [S][256] and accept [S]")
    out = ctypes.c_void_p()
    _check(lib().cstr_load_dfa(_np_ptr(trans), _np_ptr(accept), ctypes.c_int32(trans.shape[0]),
                               ctypes.c_int32(start_state), ctypes.byref(out)))
    return Dfa(out)


def cstr_load_dfa_terminals(trans, term_trans, accept, start_state=0) -> Dfa:
    """``trans`` int32 ``[S][256]``, ``term_trans`` int32 ``[S][n_labels]`` (terminal-label edges)."""
    trans = np.ascontiguousarray(trans, dtype=np.int32)
    term_trans = np.ascontiguousarray(term_trans, dtype=np.int32)
    accept = np.ascontiguousarray(accept, dtype=np.uint8)
    if trans.ndim != 2 or trans.shape[1] != 256 or accept.shape != (trans.shape[0],):
        raise ValueError("trans must be [S][256] and accept [S]")
    if term_trans.ndim != 2 or term_trans.shape[0] != trans.shape[0]:
        raise ValueError("term_trans must be [S][n_labels]")
    out = ctypes.c_void_p()
    _check(lib().cstr_load_dfa_terminals(_np_ptr(trans), _np_ptr(term_trans),
                                         ctypes.c_int32(term_trans.shape[1]), _np_ptr(accept),
                                         ctypes.c_int32(trans.shape[0]),
                                         ctypes.c_int32(start_state), ctypes.byref(out)))
    return Dfa(out)


def cstr_vocab_set_token_sets(vocab: Vocab, token_sets, n_labels: int) -> None:
    """``token_sets`` uint32 ``[V]``: bit t set iff the token belongs to terminal label t's set."""
    token_sets = np.ascontiguousarray(token_sets, dtype=np.uint32)
    if token_sets.shape != (vocab.size,):
        raise ValueError("token_sets must have one uint32 per token")
    _check(lib().cstr_vocab_set_token_sets(vocab.ptr, _np_ptr(token_sets), ctypes.c_int32(n_labels)))


def cstr_load_vocab(vocab_bytes, offsets) -> Vocab:
    vocab_bytes = np.ascontiguousarray(vocab_bytes, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    out = ctypes.c_void_p()
    _check(lib().cstr_load_vocab(_np_ptr(vocab_bytes), _np_ptr(offsets),
                                 ctypes.c_int32(offsets.size - 1), ctypes.byref(out)))
    v = Vocab(out)
    v.size = int(offsets.size - 1)
    return v


def cstr_table_create(vocab: Vocab, max_states: int) -> Table:
    out = ctypes.c_void_p()
    _check(lib().cstr_table_create(vocab.ptr, ctypes.c_int32(max_states), ctypes.byref(out)))
    t = Table(out)
    t.vocab = vocab
    return t


def cstr_table_build(table: Table, dfa: Dfa, eos_id: int = -1, stream=None) -> None:
    _check(lib().cstr_table_build(table.ptr, dfa.ptr, ctypes.c_int32(eos_id), _stream_ptr(stream)))


def cstr_table_build_dense(table: Table, dfa: Dfa, eos_id: int = -1, stream=None) -> None:
    """The same table by the per-token walk without shared prefixes (measurement baseline)."""
    _check(lib().cstr_table_build_dense(table.ptr, dfa.ptr, ctypes.c_int32(eos_id),
                                        _stream_ptr(stream)))


def cstr_build_token_table(dfa: Dfa, vocab_bytes, offsets, eos_id: int = -1, stream=None) -> Table:
    vocab_bytes = np.ascontiguousarray(vocab_bytes, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    out = ctypes.c_void_p()
    _check(lib().cstr_build_token_table(dfa.ptr, _np_ptr(vocab_bytes), _np_ptr(offsets),
                                        ctypes.c_int32(offsets.size - 1), ctypes.c_int32(eos_id),
                                        _stream_ptr(stream), ctypes.byref(out)))
    return Table(out)


def cstr_table_info(table: Table):
    vals = [ctypes.c_int32() for _ in range(4)]
    _check(lib().cstr_table_info(table.ptr, *[ctypes.byref(v) for v in vals]))
    n_states, vocab_size, words, start = (int(v.value) for v in vals)
    return dict(n_states=n_states, vocab_size=vocab_size, mask_words=words, start_state=start)


def cstr_table_download(table: Table, state_lo: int = 0, state_hi: int | None = None,
                        want_mask: bool = True, want_next: bool = True, stream=None):
    info = cstr_table_info(table)
    state_hi = info["n_states"] if state_hi is None else state_hi
    rows = max(state_hi - state_lo, 0)
    mask = np.empty((rows, info["mask_words"]), dtype=np.uint32) if want_mask else None
    nxt = np.empty((rows, info["vocab_size"]), dtype=np.int32) if want_next else None
    _check(lib().cstr_table_download(table.ptr, ctypes.c_int32(state_lo), ctypes.c_int32(state_hi),
                                     _np_ptr(mask), _np_ptr(nxt), _stream_ptr(stream)))
    return nxt, mask


def cstr_workspace_create(max_batch: int) -> Workspace:
    out = ctypes.c_void_p()
    _check(lib().cstr_workspace_create(ctypes.c_int32(max_batch), ctypes.byref(out)))
    return Workspace(out)


def _step_tensor_checks(logits, masked_out, noise, per_row, vocab_ld=None):
    """Argument checks shared by the step wrappers; returns ``(dtype code, ld, batch)``.

    ``per_row`` lists ``(name, tensor or None, torch dtype)`` for the arrays that hold
    one entry per row.  Every check runs before anything is handed to the library: a
    short or wrongly typed per-row tensor would otherwise become an out-of-bounds
    device write."""
    import torch
    if logits.dtype == torch.float32:
        dtype = CSTR_F32
    elif logits.dtype == torch.bfloat16:
        dtype = CSTR_BF16
    else:
        raise TypeError("logits must be float32 or bfloat16")
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [B][ld] with unit inner stride")
    ld = logits.stride(0) if vocab_ld is None else vocab_ld
    batch = logits.shape[0]
    if masked_out is None:
        raise ValueError("masked_out is required")
    for name, t in (("masked_out", masked_out), ("noise", noise)):
        if t is not None and (t.dim() != 2 or t.stride(1) != 1 or t.stride(0) != logits.stride(0)
                              or t.shape[0] != batch):
            raise ValueError("%s must have the layout of logits" % name)
    if masked_out.dtype != logits.dtype:
        raise TypeError("masked_out must have the dtype of logits")
    if noise is not None and noise.dtype != torch.float32:
        raise TypeError("noise must be float32")
    for name, t, dt in per_row:
        if t is not None and (t.dtype != dt or t.numel() < batch or not t.is_contiguous()):
            raise ValueError("%s must be a contiguous %s tensor with one entry per row" % (name, dt))
    tensors = [("logits", logits), ("masked_out", masked_out), ("noise", noise)]
    tensors += [(name, t) for name, t, _ in per_row]
    for name, t in tensors:
        if t is not None and (not t.is_cuda or t.device != logits.device):
            raise ValueError("%s must be a CUDA tensor on the device of logits" % name)
    return dtype, ld, batch


def cstr_step(tables, logits, states, tokens_out, masked_out, ws: Workspace, noise=None,
              row_table=None, accept_out=None, vocab_ld: int | None = None, stream=None,
              states_out=None) -> None:
    """Enqueue one constrained decoding step (``cstr_step``; with ``states_out`` given,
    ``cstr_step_history``: ``states`` is left untouched).  All tensors are CUDA tensors:
    ``logits``/``masked_out`` ``[B][ld]`` float32 or bfloat16, ``noise`` float32
    ``[B][ld]`` or None, ``states``/``tokens_out``/``row_table`` int32 ``[B]``,
    ``accept_out`` uint8 ``[B]`` or None."""
    import torch
    if isinstance(tables, Table):
        tables = [tables]
    if states is None or tokens_out is None:
        raise ValueError("states and tokens_out are required")
    dtype, ld, batch = _step_tensor_checks(
        logits, masked_out, noise,
        (("states", states, torch.int32), ("states_out", states_out, torch.int32),
         ("tokens_out", tokens_out, torch.int32), ("row_table", row_table, torch.int32),
         ("accept_out", accept_out, torch.uint8)), vocab_ld)
    arr = (ctypes.c_void_p * len(tables))(*[t.ptr.value for t in tables])
    if states_out is None:
        _check(lib().cstr_step(arr, ctypes.c_int32(len(tables)), _dev_ptr(row_table),
                               _dev_ptr(logits), ctypes.c_int32(dtype), ctypes.c_int64(ld),
                               _dev_ptr(noise), _dev_ptr(states), _dev_ptr(tokens_out),
                               _dev_ptr(masked_out), _dev_ptr(accept_out), ctypes.c_int32(batch),
                               ws.ptr, _stream_ptr(stream)))
    else:
        _check(lib().cstr_step_history(arr, ctypes.c_int32(len(tables)), _dev_ptr(row_table),
                                       _dev_ptr(logits), ctypes.c_int32(dtype), ctypes.c_int64(ld),
                                       _dev_ptr(noise), _dev_ptr(states), _dev_ptr(states_out),
                                       _dev_ptr(tokens_out), _dev_ptr(masked_out),
                                       _dev_ptr(accept_out), ctypes.c_int32(batch), ws.ptr,
                                       _stream_ptr(stream)))


def cstr_step_host(tables, logits_host, states, tokens_host, logits_dev, masked_out, tokens_dev,
                   ws: Workspace, states_host=None, noise_host=None, noise_dev=None, row_table=None,
                   accept_out=None, masked_host=None, stream=None) -> None:
    """``cstr_step`` for logits in host memory (synchronous).  ``logits_host`` /
    ``noise_host`` / ``tokens_host`` / ``states_host`` are CPU tensors (pinned for speed),
    ``logits_dev`` / ``noise_dev`` device staging tensors of the same shapes, ``masked_host``
    an optional CPU tensor that receives the penalised logits, the rest as in ``cstr_step``."""
    import torch
    if isinstance(tables, Table):
        tables = [tables]
    if logits_host.dtype == torch.float32:
        dtype = CSTR_F32
    elif logits_host.dtype == torch.bfloat16:
        dtype = CSTR_BF16
    else:
        raise TypeError("logits must be float32 or bfloat16")
    if logits_host.is_cuda or logits_host.dim() != 2 or not logits_host.is_contiguous():
        raise ValueError("logits_host must be a contiguous CPU tensor [B][ld]")
    batch, ld = logits_host.shape
    for name, t in (("logits_dev", logits_dev), ("masked_out", masked_out)):
        if not t.is_cuda or t.dtype != logits_host.dtype or tuple(t.shape) != (batch, ld) \
                or not t.is_contiguous():
            raise ValueError("%s must be a contiguous CUDA tensor shaped like logits_host" % name)
    if masked_host is not None and (masked_host.is_cuda or masked_host.dtype != logits_host.dtype
                                    or tuple(masked_host.shape) != (batch, ld)
                                    or not masked_host.is_contiguous()):
        raise ValueError("masked_host must be a contiguous CPU tensor shaped like logits_host")
    if (noise_host is None) != (noise_dev is None):
        raise ValueError("noise_host and noise_dev go together")
    if noise_host is not None:
        for name, t, cuda in (("noise_host", noise_host, False), ("noise_dev", noise_dev, True)):
            if t.is_cuda != cuda or t.dtype != torch.float32 or tuple(t.shape) != (batch, ld) \
                    or not t.is_contiguous():
                raise ValueError("%s must be a contiguous float32 tensor [B][ld]" % name)
    for name, t, cuda in (("states", states, True), ("tokens_dev", tokens_dev, True),
                          ("tokens_host", tokens_host, False), ("states_host", states_host, False),
                          ("row_table", row_table, True)):
        if t is not None and (t.is_cuda != cuda or t.dtype != torch.int32 or t.numel() < batch
                              or not t.is_contiguous()):
            raise ValueError("%s must be a contiguous int32 tensor with one entry per row" % name)
    arr = (ctypes.c_void_p * len(tables))(*[t.ptr.value for t in tables])
    _check(lib().cstr_step_host(arr, ctypes.c_int32(len(tables)), _dev_ptr(row_table),
                                _dev_ptr(logits_host), ctypes.c_int32(dtype), ctypes.c_int64(ld),
                                _dev_ptr(noise_host), _dev_ptr(states), _dev_ptr(tokens_host),
                                _dev_ptr(states_host), _dev_ptr(logits_dev), _dev_ptr(noise_dev),
                                _dev_ptr(masked_out), _dev_ptr(masked_host), _dev_ptr(tokens_dev),
                                _dev_ptr(accept_out), ctypes.c_int32(batch), ws.ptr,
                                _stream_ptr(stream)))


def cstr_step_history(tables, logits, states_in, states_out, tokens_out, masked_out, ws: Workspace,
                      **kw) -> None:
    """``cstr_step`` with separate input and output state arrays (state history)."""
    cstr_step(tables, logits, states_in, tokens_out, masked_out, ws, states_out=states_out, **kw)


def cstr_accept_draft(draft_tokens, target_tokens, target_states, n_accepted, out_tokens, states,
                      stream=None) -> None:
    """Greedy verification + rewind.  CUDA int32 tensors: ``draft_tokens`` ``[B][k]``,
    ``target_tokens`` / ``target_states`` / ``out_tokens`` ``[B][k+1]``, ``n_accepted`` / ``states`` ``[B]``."""
    import torch
    B, k1 = target_tokens.shape
    k = k1 - 1
    for name, t, shape in (("draft_tokens", draft_tokens, (B, k)), ("target_states", target_states, (B, k1)),
                           ("out_tokens", out_tokens, (B, k1)), ("n_accepted", n_accepted, (B,)),
                           ("states", states, (B,)), ("target_tokens", target_tokens, (B, k1))):
        if t.dtype != torch.int32 or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError("%s must be a contiguous int32 tensor of shape %s" % (name, shape))
    _check(lib().cstr_accept_draft(_dev_ptr(draft_tokens), _dev_ptr(target_tokens),
                                   _dev_ptr(target_states), ctypes.c_int32(k), ctypes.c_int32(B),
                                   _dev_ptr(n_accepted), _dev_ptr(out_tokens), _dev_ptr(states),
                                   _stream_ptr(stream)))


def cstr_step_static(tables, logits, states, tokens_out, masked_out, noise=None, row_table=None,
                     accept_out=None, stream=None) -> None:
    """``cstr_step`` for callers that must not allocate: no workspace, the scratch
    is a fixed array inside the library (at most ``CSTR_STATIC_MAX_BATCH`` rows;
    calls that may overlap on the GPU must be ordered by the caller).  Same
    tensors, argument checks and results as ``cstr_step``."""
    import torch
    if isinstance(tables, Table):
        tables = [tables]
    if states is None or tokens_out is None:
        raise ValueError("states and tokens_out are required")
    dtype, ld, batch = _step_tensor_checks(
        logits, masked_out, noise,
        (("states", states, torch.int32), ("tokens_out", tokens_out, torch.int32),
         ("row_table", row_table, torch.int32), ("accept_out", accept_out, torch.uint8)))
    arr = (ctypes.c_void_p * len(tables))(*[t.ptr.value for t in tables])
    _check(lib().cstr_step_static(arr, ctypes.c_int32(len(tables)), _dev_ptr(row_table),
                                  _dev_ptr(logits), ctypes.c_int32(dtype), ctypes.c_int64(ld),
                                  _dev_ptr(noise), _dev_ptr(states), _dev_ptr(tokens_out),
                                  _dev_ptr(masked_out), _dev_ptr(accept_out), ctypes.c_int32(batch),
                                  _stream_ptr(stream)))


def cstr_step_status(ws: Workspace, stream=None):
    bad, empty = ctypes.c_int64(), ctypes.c_int64()
    _check(lib().cstr_step_status(ws.ptr, _stream_ptr(stream), ctypes.byref(bad), ctypes.byref(empty)))
    return int(bad.value), int(empty.value)


def cstr_load_pda(edge_src, edge_byte, edge_tgt, pop_off, pops, push_off, pushes, accept,
                  n_symbols: int, start_state: int = 0) -> Pda:
    """Byte-level PDA from flat int32 edge arrays (see ``cstr_load_pda`` in cstr.h)."""
    arrs = [np.ascontiguousarray(a, dtype=np.int32)
            for a in (edge_src, edge_byte, edge_tgt, pop_off, pops, push_off, pushes)]
    accept = np.ascontiguousarray(accept, dtype=np.uint8)
    n_edges = arrs[0].size
    if arrs[1].size != n_edges or arrs[2].size != n_edges or arrs[3].size != n_edges + 1 \
            or arrs[5].size != n_edges + 1:
        raise ValueError("edge arrays must have n_edges entries, offsets n_edges + 1")
    if n_edges and (arrs[4].size < arrs[3][-1] or arrs[6].size < arrs[5][-1]):
        raise ValueError("pops / pushes shorter than their offsets say")
    out = ctypes.c_void_p()
    _check(lib().cstr_load_pda(*[_np_ptr(a) for a in arrs], ctypes.c_int32(n_edges),
                               _np_ptr(accept), ctypes.c_int32(accept.size),
                               ctypes.c_int32(n_symbols), ctypes.c_int32(start_state),
                               ctypes.byref(out)))
    return Pda(out)


def cstr_build_pda_table(pda: Pda, vocab: Vocab, eos_id: int = -1, stream=None) -> PdaTable:
    out = ctypes.c_void_p()
    _check(lib().cstr_build_pda_table(pda.ptr, vocab.ptr, ctypes.c_int32(eos_id),
                                      _stream_ptr(stream), ctypes.byref(out)))
    t = PdaTable(out)
    t.pda, t.vocab = pda, vocab
    return t


def cstr_pda_table_rebuild(table: PdaTable, eos_id: int = -1, stream=None) -> None:
    _check(lib().cstr_pda_table_rebuild(table.ptr, ctypes.c_int32(eos_id), _stream_ptr(stream)))


def cstr_pda_table_info(table: PdaTable):
    vals = [ctypes.c_int32() for _ in range(5)]
    _check(lib().cstr_pda_table_info(table.ptr, *[ctypes.byref(v) for v in vals]))
    keys = ("n_states", "n_symbols", "vocab_size", "mask_words", "start_state")
    return {k: int(v.value) for k, v in zip(keys, vals)}


def cstr_pda_table_download(table: PdaTable, state: int, top: int = -1, stream=None):
    """(mask, deep) uint32 ``[W]`` rows of one situation; ``top`` = -1 for the empty stack."""
    W = cstr_pda_table_info(table)["mask_words"]
    mask = np.empty(W, dtype=np.uint32)
    deep = np.empty(W, dtype=np.uint32)
    _check(lib().cstr_pda_table_download(table.ptr, ctypes.c_int32(state), ctypes.c_int32(top),
                                         _np_ptr(mask), _np_ptr(deep), _stream_ptr(stream)))
    return mask, deep


def cstr_pda_workspace_create(table: PdaTable, max_batch: int) -> PdaWorkspace:
    out = ctypes.c_void_p()
    _check(lib().cstr_pda_workspace_create(table.ptr, ctypes.c_int32(max_batch), ctypes.byref(out)))
    return PdaWorkspace(out)


def cstr_pda_step(table: PdaTable, logits, states, stacks, depths, tokens_out, masked_out,
                  ws: PdaWorkspace, noise=None, accept_out=None, stream=None,
                  states_out=None, stacks_out=None, depths_out=None) -> None:
    """Enqueue one step of Algorithm 3.  CUDA tensors: ``logits`` / ``masked_out`` /
    ``noise`` as in ``cstr_step``; ``states`` / ``depths`` / ``tokens_out`` int32 ``[B]``;
    ``stacks`` int32 ``[B][cap]`` (bottom first).  With ``states_out`` /
    ``stacks_out`` / ``depths_out`` given (all three) the inputs are left untouched
    (``cstr_pda_step_history``)."""
    import torch
    if logits.dtype == torch.float32:
        dtype = CSTR_F32
    elif logits.dtype == torch.bfloat16:
        dtype = CSTR_BF16
    else:
        raise TypeError("logits must be float32 or bfloat16")
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [B][ld] with unit inner stride")
    batch = logits.shape[0]
    for name, t in (("masked_out", masked_out), ("noise", noise)):
        if t is not None and (t.dim() != 2 or t.stride(1) != 1 or t.stride(0) != logits.stride(0)
                              or t.shape[0] != batch):
            raise ValueError("%s must have the layout of logits" % name)
    if masked_out.dtype != logits.dtype:
        raise TypeError("masked_out must have the dtype of logits")
    if noise is not None and noise.dtype != torch.float32:
        raise TypeError("noise must be float32")
    for name, t, dt in (("states", states, torch.int32), ("depths", depths, torch.int32),
                        ("tokens_out", tokens_out, torch.int32),
                        ("accept_out", accept_out, torch.uint8)):
        if t is not None and (t.dtype != dt or t.numel() < batch or not t.is_contiguous()):
            raise ValueError("%s must be a contiguous %s tensor with one entry per row" % (name, dt))
    if stacks.dtype != torch.int32 or stacks.dim() != 2 or stacks.shape[0] < batch \
            or not stacks.is_contiguous():
        raise ValueError("stacks must be a contiguous int32 tensor [B][cap]")
    outs = (states_out, stacks_out, depths_out)
    if any(o is not None for o in outs):
        if any(o is None for o in outs):
            raise ValueError("states_out, stacks_out and depths_out go together")
        for o, i in zip(outs, (states, stacks, depths)):
            if o.dtype != torch.int32 or o.shape != i.shape or not o.is_contiguous():
                raise ValueError("output situation arrays must match the input ones")
        _check(lib().cstr_pda_step_history(
            table.ptr, _dev_ptr(logits), ctypes.c_int32(dtype), ctypes.c_int64(logits.stride(0)),
            _dev_ptr(noise), _dev_ptr(states), _dev_ptr(stacks), _dev_ptr(depths),
            _dev_ptr(states_out), _dev_ptr(stacks_out), _dev_ptr(depths_out),
            ctypes.c_int32(stacks.shape[1]), _dev_ptr(tokens_out), _dev_ptr(masked_out),
            _dev_ptr(accept_out), ctypes.c_int32(batch), ws.ptr, _stream_ptr(stream)))
        return
    _check(lib().cstr_pda_step(table.ptr, _dev_ptr(logits), ctypes.c_int32(dtype),
                               ctypes.c_int64(logits.stride(0)), _dev_ptr(noise), _dev_ptr(states),
                               _dev_ptr(stacks), _dev_ptr(depths), ctypes.c_int32(stacks.shape[1]),
                               _dev_ptr(tokens_out), _dev_ptr(masked_out), _dev_ptr(accept_out),
                               ctypes.c_int32(batch), ws.ptr, _stream_ptr(stream)))


def cstr_pda_step_history(table: PdaTable, logits, states_in, stacks_in, depths_in, states_out,
                          stacks_out, depths_out, tokens_out, masked_out, ws: PdaWorkspace,
                          **kw) -> None:
    """``cstr_pda_step`` with separate input and output situations (state history)."""
    cstr_pda_step(table, logits, states_in, stacks_in, depths_in, tokens_out, masked_out, ws,
                  states_out=states_out, stacks_out=stacks_out, depths_out=depths_out, **kw)


def cstr_pda_accept_draft(draft_tokens, target_tokens, target_states, target_stacks,
                          target_depths, n_accepted, out_tokens, states, stacks, depths,
                          stream=None) -> None:
    """Greedy verification + rewind under a push-down constraint.  CUDA int32 tensors:
    ``draft_tokens`` ``[B][k]``; ``target_tokens`` / ``target_states`` / ``target_depths`` /
    ``out_tokens`` ``[B][k+1]``; ``target_stacks`` ``[B][k+1][cap]``; ``n_accepted`` /
    ``states`` / ``depths`` ``[B]``; ``stacks`` ``[B][cap]``."""
    import torch
    B, k1 = target_tokens.shape
    k = k1 - 1
    cap = target_stacks.shape[2]
    for name, t, shape in (("draft_tokens", draft_tokens, (B, k)), ("target_tokens", target_tokens, (B, k1)),
                           ("target_states", target_states, (B, k1)),
                           ("target_depths", target_depths, (B, k1)),
                           ("target_stacks", target_stacks, (B, k1, cap)),
                           ("out_tokens", out_tokens, (B, k1)), ("n_accepted", n_accepted, (B,)),
                           ("states", states, (B,)), ("depths", depths, (B,)),
                           ("stacks", stacks, (B, cap))):
        if t.dtype != torch.int32 or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError("%s must be a contiguous int32 tensor of shape %s" % (name, shape))
    _check(lib().cstr_pda_accept_draft(_dev_ptr(draft_tokens), _dev_ptr(target_tokens),
                                       _dev_ptr(target_states), _dev_ptr(target_stacks),
                                       _dev_ptr(target_depths), ctypes.c_int32(k), ctypes.c_int32(B),
                                       ctypes.c_int32(cap), _dev_ptr(n_accepted),
                                       _dev_ptr(out_tokens), _dev_ptr(states), _dev_ptr(stacks),
                                       _dev_ptr(depths), _stream_ptr(stream)))


def cstr_pda_step_status(ws: PdaWorkspace, stream=None):
    vals = [ctypes.c_int64() for _ in range(3)]
    _check(lib().cstr_pda_step_status(ws.ptr, _stream_ptr(stream), *[ctypes.byref(v) for v in vals]))
    return tuple(int(v.value) for v in vals)


def cstr_last_error() -> str:
    return lib().cstr_last_error().decode("utf-8", "replace")
