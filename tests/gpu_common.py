"""Helpers for the GPU parity tests: run the CUDA path and the oracle on the
same seeded inputs and compare bit for bit."""
import numpy as np
import torch

import oracle
from paper_2407_08103_b200 import cstr
from synth import gumbel_noise, normal_logits

DEV = "cuda:0"


def to_dev_logits(arr):
    t = torch.from_numpy(arr).to(DEV)
    return t.view(torch.bfloat16) if arr.dtype == np.uint16 else t


def from_dev_logits(t):
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def bits_equal(a, b):
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    if a.dtype == np.float32:
        return np.array_equal(a.view(np.uint32), b.view(np.uint32))
    return np.array_equal(a, b)


def gpu_tables(dfas, vb, vo, eos_id=-1, term_trans=None, token_sets=None):
    vocab = cstr.cstr_load_vocab(vb, vo)
    if token_sets is not None:
        n_labels = max(max(t.shape[1] for t in term_trans), 1)
        cstr.cstr_vocab_set_token_sets(vocab, token_sets, n_labels)
    tables = []
    for i, d in enumerate(dfas):
        if term_trans is not None:
            h = cstr.cstr_load_dfa_terminals(d[0], term_trans[i], d[1], d[2])
        else:
            h = cstr.cstr_load_dfa(d[0], d[1], d[2])
        t = cstr.cstr_table_create(vocab, d[0].shape[0])
        cstr.cstr_table_build(t, h, eos_id)
        tables.append(t)
    torch.cuda.synchronize()
    return tables


def check_table(table, dfa, vb, vo, states=None, eos_id=-1, slab=64, threads=None,
                term_trans=None, token_sets=None):
    """Compare downloaded rows of a built table with the oracle's, slab by slab."""
    threads = threads or min(oracle.max_threads(), 32)
    S = dfa[0].shape[0]
    info = cstr.cstr_table_info(table)
    assert info["n_states"] == S and info["vocab_size"] == vo.size - 1
    assert info["mask_words"] == (vo.size - 1 + 31) // 32 and info["start_state"] == dfa[2]
    if states is None:
        ranges = [(lo, min(S, lo + slab)) for lo in range(0, S, slab)]
    else:
        ranges = [(int(q), int(q) + 1) for q in states]
    for lo, hi in ranges:
        nxt, mask = cstr.cstr_table_download(table, lo, hi)
        o_next, o_mask = oracle.token_table(dfa[0], dfa[1], vb, vo, eos_id=eos_id, q_lo=lo, q_hi=hi,
                                            threads=threads, term_trans=term_trans,
                                            token_sets=token_sets)
        assert np.array_equal(nxt, o_next), "next-state rows %d..%d differ" % (lo, hi)
        assert np.array_equal(mask, o_mask), "mask rows %d..%d differ" % (lo, hi)


def run_step_both(dfas, tables, vb, vo, logits, states, noise=None, row_table=None, eos_id=-1,
                  ws=None, in_place=False, accept=True, term_trans=None, token_sets=None):
    """One step on the GPU and on the oracle; asserts bit equality of every output."""
    B = logits.shape[0]
    ws = ws or cstr.cstr_workspace_create(B)
    d_logits = to_dev_logits(logits)
    d_noise = None if noise is None else torch.from_numpy(noise).to(DEV)
    d_states = torch.from_numpy(np.asarray(states, dtype=np.int32)).to(DEV)
    d_tokens = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    d_acc = torch.full((B,), 9, dtype=torch.uint8, device=DEV) if accept else None
    d_rt = None if row_table is None else torch.from_numpy(np.asarray(row_table, dtype=np.int32)).to(DEV)
    d_out = d_logits if in_place else torch.full_like(d_logits, 123.0)
    cstr.cstr_step(tables, d_logits, d_states, d_tokens, d_out, ws, noise=d_noise,
                   row_table=d_rt, accept_out=d_acc)
    torch.cuda.synchronize()
    bad, empty = cstr.cstr_step_status(ws)
    ref = oracle.step(dfas, vb, vo, logits, states, noise=noise, row_table=row_table,
                      eos_id=eos_id, vocab_size=vo.size - 1,
                      threads=min(oracle.max_threads(), 32), term_trans=term_trans,
                      token_sets=token_sets)
    V = vo.size - 1
    assert np.array_equal(d_tokens.cpu().numpy(), ref["tokens"])
    assert np.array_equal(d_states.cpu().numpy(), ref["states"])
    got = from_dev_logits(d_out)
    assert bits_equal(got[:, :V], ref["masked"][:, :V])
    if not in_place and got.shape[1] > V:       # padding columns are never written
        pad = from_dev_logits(torch.full_like(d_logits, 123.0))[:, V:]
        assert bits_equal(got[:, V:], pad)
    if accept:
        assert np.array_equal(d_acc.cpu().numpy(), ref["accept"])
    assert (bad, empty) == (ref["bad_state_rows"], ref["empty_mask_rows"])
    return ref
